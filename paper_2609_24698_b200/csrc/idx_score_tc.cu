// Indexer scores of long candidate lists on the tensor core (bf16 storage, 128-wide indexer rows).
//
// score(node n, entry e) = sum_h iw[n][h] * relu(iq[n][h] . ik[e])   (the lightning-indexer score of the CSA selection)
//
// For one sequence the inner products of ALL nodes and heads with a tile of entries are one small GEMM:
//   [128 entries x 128 dims] x [128 dims x (D * HI <= 32) query rows]  ->  tcgen05.mma, M = 128, N = 32, K = 128, fp32 in TMEM.
// An entry row is therefore read once per sequence instead of once per node.  A CTA walks kTilesPerCta tiles of 128
// entries: the tile rows arrive by 16-byte cp.async into two 128-byte-swizzled K-major buffers (two tiles in flight: the
// copies of tile t + 2 are issued as soon as the product of tile t is complete), thread 0 issues the eight MMAs of a
// tile, and the four warps read the accumulator (lane = entry, column = node * HI + head), apply relu and the head
// weights and store one fp32 score per ranked node.  Several CTAs share an SM (73 KiB of shared memory, 64 TMEM columns
// each).
#include "tc_common.cuh"

namespace tsv {

namespace {

constexpr int kItThreads = 128;
constexpr int kItRows = 128;               // entries per tile (the M of the MMA)
constexpr int kItN = 32;                   // query rows (node, head), zero rows beyond D * HI
constexpr int kTilesPerCta = 4;
constexpr int kItCtl = 1024, kItB = 2 * kItN * 128, kItA = 2 * kItRows * 128;
constexpr int kItSmem = kItCtl + kItB + 2 * kItA + 1024;     // + slack for the 1024-byte alignment of the tiles

struct ItCtl {
  uint64_t mma_bar[2];
  uint32_t tmem_base;
  uint32_t need_mask;
  float iw[kItN];
  TreeMeta tm;
  TreeStage tstage;
};
static_assert(sizeof(ItCtl) <= kItCtl, "control block");

template <int HI>
__global__ void __launch_bounds__(kItThreads) idx_score_tc_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                                  const tsv_scratch sc, char* __restrict__ ws, int32_t* __restrict__ status) {
  using namespace tc;
  extern __shared__ unsigned char smem_raw[];
  const int b = blockIdx.y, D = s.D, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int e0 = blockIdx.x * kTilesPerCta * kItRows;
  {   // cheap exit: even with every ancestor closing a block, no node of this sequence has more than topk candidates
    const int L0 = c.L[b];
    if (L0 < 0 || L0 / s.m_csa + D <= s.topk || e0 >= L0 / s.m_csa) return;
  }
  unsigned char* base = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  ItCtl& sm = *reinterpret_cast<ItCtl*>(base);
  const uint32_t bq = smem_u32(base + kItCtl), a0 = bq + kItB;
  coop_tree_meta(sm.tm, sm.tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, nullptr, nullptr);
  if (tid == 0) {   // nodes that rank: committed entries + blocks closed at strict ancestors exceed topk
    uint32_t m = 0;
    if (!sm.tm.status)
      for (int n = 0; n < sm.tm.nn; ++n) {
        int extra = 0;
        for (int j = 0; j < n; ++j)
          if (((sm.tm.anc[n] >> j) & 1u) && sc.csa_done[(size_t)b * D + j]) ++extra;
        if (sm.tm.n_csa + extra > s.topk) m |= 1u << n;
      }
    sm.need_mask = m;
  }
  if (tid >= 32 && tid < 32 + kItN) sm.iw[tid - 32] = tid - 32 < D * HI ? nd.iw[(size_t)b * D * HI + tid - 32] : 0.f;
  __syncthreads();
  const uint32_t need = sm.need_mask;
  const int n_csa = sm.tm.n_csa;
  if (!need || e0 >= n_csa) return;                       // taken by the whole CTA alike; nothing allocated yet
  const int nt = min(kTilesPerCta, (n_csa - e0 + kItRows - 1) / kItRows);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.mma_bar[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.mma_bar[1])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 64;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // query rows: row j = node * HI + head, two 64-wide K slices of [32 rows x 128 bytes], rows of absent nodes zero
  {
    const char* iq = reinterpret_cast<const char*>(nd.iq) + (size_t)b * D * HI * 256;
    const int rows_q = sm.tm.nn * HI;
#pragma unroll
    for (int i = 0; i < kItN * 16 / kItThreads; ++i) {
      const int idx = tid + kItThreads * i, row = idx >> 4, c16 = idx & 15;
      const bool v = row < rows_q;
      cp16(bq + (c16 >> 3) * (kItN * 128) + row * 128 + (((c16 & 7) ^ (row & 7)) << 4), iq + (v ? (size_t)row * 256 + c16 * 16 : 0), v);
    }
  }
  const char* ik = reinterpret_cast<const char*>(c.csa_ik);
  const RowAddr ikrow = csa_rows_of(c, s, b);
  auto load_tile = [&](int t) {                           // entries e0 + 128 t ..: two K slices of [128 rows x 128 bytes]
    const uint32_t dst = a0 + (uint32_t)(t & 1) * kItA;
    const int r0 = e0 + t * kItRows;
#pragma unroll
    for (int i = 0; i < kItRows * 16 / kItThreads; ++i) {
      const int idx = tid + kItThreads * i, row = idx >> 4, c16 = idx & 15;
      const bool v = r0 + row < n_csa;
      cp16(dst + (c16 >> 3) * (kItRows * 128) + row * 128 + (((c16 & 7) ^ (row & 7)) << 4), ik + (v ? (size_t)ikrow(r0 + row) * 256 + c16 * 16 : 0), v);
    }
    cp_commit();
  };
  load_tile(0);                                           // one group with the query rows
  if (nt > 1) load_tile(1); else cp_commit();             // two tiles in flight from here on
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tm = sm.tmem_base;
  const uint32_t idesc = make_idesc(kItN, 0);
  const uint32_t tlane = tm + ((uint32_t)(warp * 32) << 16);
  float* scores = reinterpret_cast<float*>(ws + pl.off_scores) + (size_t)b * D * pl.score_ld;
  int fail = 0;

  auto epilogue = [&](int t) {                            // the accumulator of tile t is complete (its barrier has been waited on)
    uint32_t r[32];
    tmem_ld32(tlane + (uint32_t)(t & 1) * kItN, r);
    const int e = e0 + t * kItRows + warp * 32 + lane;
#pragma unroll
    for (int n = 0; n < kItN / HI; ++n) {
      if (n < D && ((need >> n) & 1u)) {
        float tot = 0.f;
#pragma unroll
        for (int h = 0; h < HI; ++h) tot = fmaf(sm.iw[n * HI + h], fmaxf(__uint_as_float(r[n * HI + h]), 0.f), tot);
        if (e < n_csa) scores[(size_t)n * pl.score_ld + e] = tot;
      }
    }
  };

  for (int t = 0; t < nt; ++t) {
    cp_wait<1>();                                         // tile t (and the query rows) have landed: this thread's copies
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    fence_before();
    __syncthreads();                                      // everyone's copies; the accumulator buffer of tile t - 2 has been read
    if (tid == 0) {
      fence_after();
      const uint32_t at = a0 + (uint32_t)(t & 1) * kItA;
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_ss(tm + (uint32_t)(t & 1) * kItN, make_desc(at + j * (kItRows * 128) + ks * 32, 16, 1024),
                 make_desc(bq + j * (kItN * 128) + ks * 32, 16, 1024), idesc, (j | ks) != 0);
      mma_commit(&sm.mma_bar[t & 1]);
    }
    if (!fail && !mbar_wait(&sm.mma_bar[t & 1], (uint32_t)(t >> 1) & 1u)) fail = 1;
    fail = __any_sync(0xffffffffu, fail);                 // warp-uniform: the accumulator loads are warp-collective
    fence_after();
    if (t + 2 < nt) load_tile(t + 2); else cp_commit();   // the tile's buffer is free again; one group per iteration either way
    if (!fail) epilogue(t);
  }
  cp_wait<0>();
  if (fail && lane == 0) atomicOr(status + b, TSV_ST_INTERNAL);
  fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 64;" ::"r"(tm) : "memory");
}

template <int HI>
void launch_hi(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, char* ws,
               int32_t* status, cudaStream_t st) {
  cudaFuncSetAttribute(idx_score_tc_kernel<HI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kItSmem);
  TSV_PREP(idx_score_tc_kernel<HI>);
  const int pref_cap = (int)(s.max_L / s.m_csa);
  const dim3 grid((pref_cap + kTilesPerCta * kItRows - 1) / (kTilesPerCta * kItRows), s.B);
  idx_score_tc_kernel<HI><<<grid, kItThreads, kItSmem, st>>>(s, p, c, nd, sc, ws, status);
  count_launch();
}

}  // namespace

bool idx_score_tc_applies(const tsv_shape& s) {
  return s.dtype == TSV_BF16 && s.di == 128 && s.D * s.HI <= kItN && (s.HI == 1 || s.HI == 2 || s.HI == 4 || s.HI == 8) &&
         s.max_L / s.m_csa > 0;
}

void launch_idx_score_tc(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, char* ws,
                         int32_t* status, cudaStream_t st) {
  switch (s.HI) {
    case 1: launch_hi<1>(s, p, c, nd, sc, ws, status, st); break;
    case 2: launch_hi<2>(s, p, c, nd, sc, ws, status, st); break;
    case 4: launch_hi<4>(s, p, c, nd, sc, ws, status, st); break;
    default: launch_hi<8>(s, p, c, nd, sc, ws, status, st); break;
  }
}

}  // namespace tsv
