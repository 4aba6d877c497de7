// Per-node top-k for short candidate lists (at most kIdxFusedMax committed entries) with 128-wide bf16 indexer rows (the
// benchmark's): one CTA per (sequence, node) that scores, ranks and selects.  Same result as topk_kernel (the exact k
// largest scores, ties to the lower index, ascending output); built so that
//   * nodes that do not rank (nearly all of them) are a short chain and ALL CTAs of the launch are resident at once
//     (four CTAs per SM: 64 registers, shared memory sized by the host for it), and
//   * a node that ranks -- its CTA is the critical path of the whole stage -- overlaps what it can: the first rows are
//     requested as soon as the length is known, the scores come from warp-level tensor-core products (mma.sync: the
//     rows of a round as A, the node's indexer queries as B) so that a round costs its copies only, the radix keys stay
//     in registers, and the selected indices are written after ONE block scan.
#include <mma.h>

#include "select_common.cuh"

namespace tsv {

namespace fsel {

constexpr int DI = 128;                       // indexer width (bf16: 256-byte rows)
// candidates per thread (keys in registers): 3 for lists of up to 768 candidates, else 9 (9 x 256 >= kIdxFusedMax + TSV_MAX_D);
// two instantiations, so that the short lists of the common shapes do not step through the predicated code of nine
constexpr int KPT_SHORT = 3, KPT_LONG = 9;
static_assert(kIdxFusedMax + TSV_MAX_D <= KPT_LONG * 256, "candidate lists must fit the in-register keys");

__device__ __forceinline__ void cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace fsel

// Dynamic shared memory: [4][128] bf16 queries (heads beyond HI zero) | scores [score_cap] fp32 | two buffers of `rows`
// staged indexer rows of 256 bytes (16-byte pieces XOR-swizzled by the row, so that ldmatrix reads without conflicts).
template <bool PAGED, int KPT>
__global__ void __launch_bounds__(256, 4) topk_fused_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                            const tsv_scratch sc, int32_t* __restrict__ topk_user, char* __restrict__ ws,
                                                            int32_t* __restrict__ status, const int rows, const int score_cap) {
  using namespace fsel;
  extern __shared__ __align__(128) unsigned char dsm[];
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ PathEntries pe;
  __shared__ float extra[TSV_MAX_D];
  __shared__ uint32_t hist[3][128];                    // radix histogram, two 16-bit bins per word (a list has < 65536 candidates); the buffers rotate between passes
  __shared__ int wsum[9];
  __shared__ int64_t row0_sm;
  bf16* iqs = reinterpret_cast<bf16*>(dsm);
  float* ssm = reinterpret_cast<float*>(dsm + 4 * DI * 2);
  unsigned char* stage = dsm + 4 * DI * 2 + (size_t)score_cap * 4;
  const int t = threadIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the tile plan may start its selection-independent part
  const int n = blockIdx.x, b = blockIdx.y, D = s.D, k = s.topk, HI = s.HI;
  const bool anchor = blockIdx.x == 0 && blockIdx.y == 0;
  int32_t* sel = reinterpret_cast<int32_t*>(ws + pl.off_sel) + ((size_t)b * D + n) * k;
  int32_t* selcnt = reinterpret_cast<int32_t*>(ws + pl.off_selcnt) + (size_t)b * D + n;
  int32_t* usr = topk_user ? topk_user + ((size_t)b * D + n) * k : nullptr;
  // The tensor-core attention path reads mask rows of ranking nodes only, never the index lists: when the caller does not
  // ask for the lists either, the CTA of a node that cannot rank (the sequence's committed entries plus one per node
  // of the tree stay within k) has nothing to do.  One load decides it; node 0 of every sequence still goes on, to
  // validate the sequence's inputs.  (A CTA takes up the registers of a ranking one while it lives, and the plan kernel
  // starts when the last CTA of this kernel has: the sooner it leaves the better.)
  if (pl.tc && !topk_user && n != 0) {
    const int L0 = c.L[b];
    if (L0 >= 0 && L0 / s.m_csa + D <= k) return;
  }
  // Everything the CTA may need that depends on (b, n) alone is requested together with the tree's loads (one memory
  // latency for all): the slab offset and -- used only if the node ranks -- its indexer queries and head weights.  The
  // kernel is launched as a programmatic dependent of the state build and reads nothing that kernel writes until a node
  // that ranks scores the entries closed inside the tree (the done flags are worked out from the positions).  A CTA that
  // does not rank leaves without waiting, except CTA (0, 0): through it this kernel's completion implies that one's.
  if (!PAGED && t == 64) row0_sm = c.csa_row0[b];
  const int lane = t & 31, w = t >> 5, g = lane >> 2, tq = lane & 3;
  const bf16* iq = reinterpret_cast<const bf16*>(nd.iq) + ((size_t)b * D + n) * HI * DI;
  const float* iwp = nd.iw + ((size_t)b * D + n) * HI;
  uint4 qv = make_uint4(0u, 0u, 0u, 0u);
  if (t < HI * 16) qv = __ldg(reinterpret_cast<const uint4*>(iq) + t);
  const float iw0 = 2 * tq < HI ? __ldg(iwp + 2 * tq) : 0.f, iw1 = 2 * tq + 1 < HI ? __ldg(iwp + 2 * tq + 1) : 0.f;
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
  if (t < 64) reinterpret_cast<uint4*>(iqs)[t] = qv;   // (read after the next barrier)
  const bool live = !tm.status && n < tm.nn;
  const int n_csa = tm.n_csa;
  // A node ranks iff its committed entries plus the blocks closed at its strict ancestors exceed k; at most depth(n)
  // ancestors can have closed one, so the rows are requested now where that bound allows ranking (the done flags
  // arrive two memory latencies later).
  const bool may_rank = live && n_csa + tm.depth[n] > k;
  RowAddr ikr;
  if (PAGED) ikr = csa_rows_of(c, s, b); else { ikr.pt = nullptr; ikr.per_page = 1; ikr.row0 = row0_sm; }
  const char* ikb = reinterpret_cast<const char*>(c.csa_ik) + (size_t)ikr.row0 * (DI * 2);
  const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
  const int nrd = (n_csa + rows - 1) / rows;
  auto issue = [&](int rd) {                           // rows [rd * rows, ..) into buffer rd & 1; one copy group per call
    const int base = rd * rows, nrow = min(rows, n_csa - base);
    const uint32_t dst = stage_s + (uint32_t)(rd & 1) * (uint32_t)(rows * 256);
    for (int idx = t; idx < nrow * 16; idx += 256) {
      const int row = idx >> 4, c16 = idx & 15;
      cp16(dst + row * 256 + ((c16 ^ (row & 7)) << 4), ikb + (size_t)(PAGED ? ikr.rel(base + row) : (int64_t)(base + row)) * 256 + c16 * 16);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (may_rank) issue(0);
  if (t < 32) {
    // Warp 0, lane j = node j: which nodes close a block (from their positions), and from that the entries on this node's
    // path -- the strict ancestors that closed a CSA / HCA block, root first -- by ballots instead of a loop of one thread.
    const bool valid = !tm.status && t < tm.nn;
    const uint32_t strict = live ? tm.anc[n] & ~(1u << n) : 0u;
    const uint32_t cm = __ballot_sync(0xffffffffu, valid && node_closes(tm.L, tm.depth[t], s.m_csa)) & strict;
    const uint32_t hm = __ballot_sync(0xffffffffu, valid && node_closes(tm.L, tm.depth[t], s.m_hca)) & strict;
    const uint32_t lower = (1u << t) - 1u;
    if ((cm >> t) & 1u) { const int o = __popc(cm & lower); pe.newc[o] = t; pe.newc_blk[o] = (tm.L + tm.depth[t]) / s.m_csa; }
    if ((hm >> t) & 1u) pe.newh[__popc(hm & lower)] = t;
    if (t == 0) {
      pe.n_newc = __popc(cm); pe.n_newh = __popc(hm);
      if (tm.status && n == 0) atomicOr(status + b, tm.status);
    }
  }
  __syncthreads();
  if (!live) {
    for (int i = t; i < k; i += 256) { sel[i] = -1; if (usr) usr[i] = -1; }
    if (t == 0) *selcnt = 0;
    if (anchor) asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
  const int n_cand = n_csa + pe.n_newc;
  if (n_cand <= k) {                                   // everything is selected: no ranking
    for (int i = t; i < k; i += 256) {
      const int v = i < n_csa ? i : (i < n_cand ? pe.newc_blk[i - n_csa] : -1);
      sel[i] = v; if (usr) usr[i] = v;
    }
    if (t == 0) *selcnt = n_cand;
    if (may_rank) asm volatile("cp.async.wait_group 0;" ::: "memory");     // (requested in vain: the bound was not reached)
    if (anchor) asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
  // ---------------------------------------------------------------------------------------------- the node ranks
  if (nrd > 1) issue(1); else asm volatile("cp.async.commit_group;" ::: "memory");
  if (t < 128) hist[0][t] = 0;
  // B fragments of the eight k-steps: column g = head g (zero beyond HI), k = 16 ks + 2 tq (+ 8)
  uint32_t bq[8][2];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    bq[ks][0] = g < 4 ? *reinterpret_cast<const uint32_t*>(iqs + g * DI + ks * 16 + 2 * tq) : 0u;
    bq[ks][1] = g < 4 ? *reinterpret_cast<const uint32_t*>(iqs + g * DI + ks * 16 + 2 * tq + 8) : 0u;
  }
  // Rounds of `rows` rows in two buffers: the copies of the next round run under the products of the current one.
  for (int rd = 0; rd < nrd; ++rd) {                   // uniform trip count: barriers and shuffles below
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // round rd has landed (this thread's copies)
    __syncthreads();
    const int base = rd * rows, nrow = min(rows, n_csa - base);
    const uint32_t buf = stage_s + (uint32_t)(rd & 1) * (uint32_t)(rows * 256);
    for (int r0 = 16 * w; r0 < nrow; r0 += 128) {       // a warp scores 16 rows per step
      float acc[4] = {0.f, 0.f, 0.f, 0.f}, acd[4] = {0.f, 0.f, 0.f, 0.f};     // two chains: even and odd k-steps
      const int row = r0 + (lane & 15);
#pragma unroll
      for (int ks = 0; ks < 8; ks += 2) {
        uint32_t a[4], a2[4];
        ldmatrix_x4(buf + row * 256 + (((ks * 2 + (lane >> 4)) ^ (row & 7)) << 4), a);
        ldmatrix_x4(buf + row * 256 + (((ks * 2 + 2 + (lane >> 4)) ^ (row & 7)) << 4), a2);
        mma_bf16_16816(acc, a, bq[ks][0], bq[ks][1]);
        mma_bf16_16816(acd, a2, bq[ks + 1][0], bq[ks + 1][1]);
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) acc[x] += acd[x];
      // C: rows g and g + 8 of the step, columns (heads) 2 tq and 2 tq + 1
      float lo = fmaf(iw1, fmaxf(acc[1], 0.f), iw0 * fmaxf(acc[0], 0.f)), hi = fmaf(iw1, fmaxf(acc[3], 0.f), iw0 * fmaxf(acc[2], 0.f));
      lo += __shfl_xor_sync(0xffffffffu, lo, 1);
      hi += __shfl_xor_sync(0xffffffffu, hi, 1);
      if (tq == 0) {
        if (r0 + g < nrow) ssm[base + r0 + g] = lo;
        if (r0 + g + 8 < nrow) ssm[base + r0 + g + 8] = hi;
      }
    }
    __syncthreads();                                   // the buffer is refilled; the scores are visible
    if (rd + 2 < nrd) issue(rd + 2); else asm volatile("cp.async.commit_group;" ::: "memory");
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  // Scores of the in-tree entries on this node's path: the state build's results, the first thing of that kernel this
  // CTA reads (all of the committed entries' scoring above may run under its tail).  Warp w takes entries w, w + 8, ...
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int i = w; i < pe.n_newc; i += 8) {
    const bf16* ik = reinterpret_cast<const bf16*>(sc.new_csa_ik) + ((size_t)b * D + pe.newc[i]) * DI;
    float tot = 0.f;
    for (int h = 0; h < HI; ++h) {
      float p = 0.f;
      for (int x = lane; x < DI; x += 32) p = fmaf(to_f(iqs[h * DI + x]), to_f(ik[x]), p);
      p = warp_sum(p);
      tot = fmaf(iwp[h], fmaxf(p, 0.f), tot);
    }
    if (lane == 0) extra[i] = tot;
  }
  __syncthreads();                                     // (the in-tree entries' scores, the cleared histogram)
  // order-preserving keys: candidate t + 256 j is key j of thread t (all warps take part in every pass)
  uint32_t key[KPT];
  const int nj = (n_cand + 255) >> 8;
#pragma unroll
  for (int j = 0; j < KPT; ++j) {
    const int i = t + 256 * j;
    key[j] = (j < nj && i < n_cand) ? order_key(i < n_csa ? ssm[i] : extra[i - n_csa]) : 0u;
  }
  // Four radix passes of 8 bits.  ONE barrier per pass: after it the histogram is complete and EVERY warp finds the bin of
  // the rem-th largest key for itself (lane l owns bins 255 - 8 l .. 248 - 8 l); the histogram buffers rotate, the one for
  // the next pass is cleared at the start of a pass (its last readers passed the previous pass's barrier before).
  uint32_t mask = 0, prefix = 0;
  int rem = k;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    uint32_t* hcur = hist[pass % 3];
    if (t < 128) hist[(pass + 1) % 3][t] = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      if (j < nj) {
        const bool in = t + 256 * j < n_cand && (key[j] & mask) == prefix;
        const uint32_t bin = in ? (key[j] >> shift) & 255u : 256u;
        // the scores of one list share their high digits: when the whole warp hits one bin, one lane adds for all
        int uniform;
        __match_all_sync(0xffffffffu, bin, &uniform);
        if (uniform) { if (in && lane == 0) atomicAdd(&hcur[bin >> 1], 32u << (16 * (bin & 1))); }
        else if (in) atomicAdd(&hcur[bin >> 1], 1u << (16 * (bin & 1)));
      }
    }
    __syncthreads();
    int h[8], tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { const int bj = 255 - (lane * 8 + j); h[j] = (hcur[bj >> 1] >> (16 * (bj & 1))) & 0xFFFF; tot += h[j]; }
    int incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
    const int excl = incl - tot;
    const bool owner = excl < rem && incl >= rem;      // exactly one lane
    int cum = excl, bin = 255 - lane * 8;
    if (owner) {
#pragma unroll
      for (int j = 0; j < 8; ++j) { if (cum + h[j] >= rem) { bin = 255 - (lane * 8 + j); break; } cum += h[j]; }
    }
    const int src = __ffs(__ballot_sync(0xffffffffu, owner)) - 1;
    prefix |= (uint32_t)__shfl_sync(0xffffffffu, bin, src) << shift;
    rem -= __shfl_sync(0xffffffffu, cum, src);
    mask |= 0xFFu << shift;
  }
  const uint32_t thr = prefix;          // key of the k-th largest score
  const int r_take = rem;               // how many of the scores equal to it are taken (lowest indices)
  // Ordered compaction: warp w owns the candidates [w * share, (w + 1) * share) (whole rows of 32; their keys are derived
  // again from the scores), counts its keys above and equal to the threshold with ballots, the warps exchange their
  // counts once, then each writes its selected indices row by row.
  uint8_t* selmask = pl.tc ? reinterpret_cast<uint8_t*>(ws + pl.off_selmask) + ((size_t)b * D + n) * pl.mask_ld : nullptr;   // (for the tile plan)
  const int share = ((n_cand + 7) / 8 + 31) & ~31, beg = w * share;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t ckey[(KPT * 256 / 8 + 31) / 32 + 1];        // rows of the warp's share: at most 10
  constexpr int CR = (KPT * 256 / 8 + 31) / 32 + 1;
  int cgt = 0, ceq = 0;
#pragma unroll
  for (int r = 0; r < CR; ++r) {
    const int i = beg + 32 * r + lane;
    const bool v = 32 * r < share && i < n_cand;
    ckey[r] = v ? order_key(i < n_csa ? ssm[i] : extra[i - n_csa]) : 0u;
    cgt += __popc(__ballot_sync(0xffffffffu, v && ckey[r] > thr));
    ceq += __popc(__ballot_sync(0xffffffffu, v && ckey[r] == thr));
  }
  if (lane == 0) wsum[w] = cgt | (ceq << 16);
  __syncthreads();
  int eq_base = 0, out_base = 0;
  for (int x = 0; x < w; ++x) { const int v = wsum[x]; out_base += v & 0xFFFF; eq_base += v >> 16; }
  out_base += min(r_take, eq_base);                    // of the equal keys before this share, the first r_take are taken
#pragma unroll
  for (int r = 0; r < CR; ++r) {
    const int i = beg + 32 * r + lane;
    const bool v = 32 * r < share && i < n_cand, eq = v && ckey[r] == thr;
    const uint32_t eqm = __ballot_sync(0xffffffffu, eq);
    const bool take = (v && ckey[r] > thr) || (eq && eq_base + __popc(eqm & lt) < r_take);
    const uint32_t tkm = __ballot_sync(0xffffffffu, take);
    if (v && selmask) selmask[i] = (uint8_t)take;
    if (take) {
      const int pos = out_base + __popc(tkm & lt), val = i < n_csa ? i : pe.newc_blk[i - n_csa];
      sel[pos] = val; if (usr) usr[pos] = val;
    }
    eq_base += __popc(eqm); out_base += __popc(tkm);
  }
  if (t == 0) *selcnt = k;
}

// The kernel serves: bf16, 128-wide indexer rows, at most four indexer heads, lists the selection scores itself.
bool topk_fused_applies(const tsv_shape& s, const TvaPlan& p) {
  return p.need_scores && p.idx_fused && s.dtype == TSV_BF16 && s.di == fsel::DI && s.HI <= 4;
}

// Rows per staging buffer (two buffers) and dynamic shared memory: as many rows (<= 128, a multiple of 16) as let four
// CTAs share an SM.
static void fused_smem(const TvaPlan& p, int& rows, int& score_cap, size_t& bytes) {
  score_cap = p.score_ld;
  const size_t fixed = 4 * fsel::DI * 2 + (size_t)score_cap * 4;
  const size_t budget = 52 * 1024;                     // of 57 KiB per CTA at four per SM: static shared memory and the per-CTA reserve come on top
  rows = 128;
  while (rows > 16 && fixed + (size_t)2 * rows * 256 > budget) rows -= 16;
  bytes = fixed + (size_t)2 * rows * 256;
}

int launch_topk_fused(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                      int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st) {
  int rows, score_cap;
  size_t bytes;
  fused_smem(p, rows, score_cap, bytes);
  const dim3 grid(s.D, s.B);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(256, 1, 1); cfg.dynamicSmemBytes = bytes; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;          // may start under the state build's tail (it waits inside)
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
#define TSV_FUSED_LAUNCH(PG_, KPT_)                                                                                                     \
  do {                                                                                                                                 \
    TSV_PREP((topk_fused_kernel<PG_, KPT_>));                                                                                          \
    if (bytes > 40 * 1024) cudaFuncSetAttribute(topk_fused_kernel<PG_, KPT_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); \
    cudaLaunchKernelEx(&cfg, topk_fused_kernel<PG_, KPT_>, s, p, c, nd, sc, topk_idx, ws, status, rows, score_cap);                     \
  } while (0)
  const bool shortl = p.cand_cap <= fsel::KPT_SHORT * 256;
  if (c.page_table) { if (shortl) TSV_FUSED_LAUNCH(true, fsel::KPT_SHORT); else TSV_FUSED_LAUNCH(true, fsel::KPT_LONG); }
  else { if (shortl) TSV_FUSED_LAUNCH(false, fsel::KPT_SHORT); else TSV_FUSED_LAUNCH(false, fsel::KPT_LONG); }
#undef TSV_FUSED_LAUNCH
  count_launch();
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
