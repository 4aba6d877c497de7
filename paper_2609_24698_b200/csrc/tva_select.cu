// CSA selection for tree_verify_attn: indexer scores of the committed entries and the exact
// per-node top-k (ties to the lower block index, ascending output).
//
//   idx_score_kernel  thread-per-entry; the entry's indexer key stays in flight in registers
//                     16 bytes at a time, the indexer queries of a group of nodes sit in shared
//                     memory (broadcast reads).  Skipped (early exit) for sequences where every
//                     node has at most topk candidates -- then the selection is "everything".
//   topk_kernel       one CTA per (sequence, node): 4-pass 8-bit radix select on the order-
//                     preserving integer image of the fp32 score, then one ordered compaction
//                     pass.  In-tree entries (closed at strict ancestors) are scored here.
#include "select_common.cuh"

namespace tsv {

template <typename T>
__global__ void __launch_bounds__(256) idx_score_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                        const tsv_scratch sc, char* __restrict__ ws) {
  extern __shared__ float iq_s[];                 // [<=32 (node, head) pairs][di]
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ int need_any;
  __shared__ uint32_t need_mask;
  const int b = blockIdx.y, D = s.D, di = s.di, HI = s.HI;
  {   // cheap exit: even with every ancestor closing a block, no node of this sequence has more than topk candidates
    const int L0 = c.L[b];
    if (L0 < 0 || L0 / s.m_csa + D <= s.topk || (int)(blockIdx.x * blockDim.x) >= L0 / s.m_csa) return;
  }
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, nullptr, nullptr);
  if (threadIdx.x == 0) {
    uint32_t m = 0;
    if (!tm.status)
      for (int n = 0; n < tm.nn; ++n) {
        int extra = 0;
        for (int j = 0; j < n; ++j)
          if (((tm.anc[n] >> j) & 1u) && sc.csa_done[(size_t)b * D + j]) ++extra;
        if (tm.n_csa + extra > s.topk) m |= 1u << n;
      }
    need_mask = m; need_any = m != 0;
  }
  __syncthreads();
  if (!need_any || (int)(blockIdx.x * blockDim.x) >= tm.n_csa) return;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const bool live = e < tm.n_csa;
  const T* ikrow = reinterpret_cast<const T*>(c.csa_ik) + (size_t)csa_rows_of(c, s, b)(live ? e : 0) * di;
  float* scores = reinterpret_cast<float*>(ws + pl.off_scores) + (size_t)b * D * pl.score_ld;
  constexpr int V = Vec<T>::N;
  const int npg = min(32 / HI, (D + (int)gridDim.z - 1) / (int)gridDim.z);   // nodes per group; blockIdx.z owns a slab of nodes
  const int nz0 = blockIdx.z * ((D + (int)gridDim.z - 1) / (int)gridDim.z), nz1 = min(tm.nn, nz0 + (D + (int)gridDim.z - 1) / (int)gridDim.z);
  for (int n0 = nz0; n0 < nz1; n0 += npg) {
    const int gn = min(npg, nz1 - n0), G = gn * HI;
    __syncthreads();
    for (int i = threadIdx.x; i < G * di; i += blockDim.x)
      iq_s[i] = to_f(reinterpret_cast<const T*>(nd.iq)[((size_t)b * D + n0) * HI * di + i]);
    __syncthreads();
    if (!((need_mask >> n0) & ((gn >= 32 ? 0xffffffffu : ((1u << gn) - 1u))))) continue;
    float acc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
    for (int cidx = 0; cidx < di / V; ++cidx) {
      float kk[V];
      ld16(ikrow + cidx * V, kk);
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        if (j < G) {
          const float* qv = iq_s + j * di + cidx * V;
#pragma unroll
          for (int t = 0; t < V; ++t) acc[j] = fmaf(qv[t], kk[t], acc[j]);
        }
      }
    }
    if (live) {
      for (int g = 0; g < gn; ++g) {
        float sc_ = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if (j / HI == g && j < G) sc_ = fmaf(nd.iw[((size_t)b * D + n0 + g) * HI + (j % HI)], fmaxf(acc[j], 0.f), sc_);
        }
        scores[(size_t)(n0 + g) * pl.score_ld + e] = sc_;
      }
    }
  }
}

// 16 raw bytes of storage elements widened to fp32 (the tag argument selects the storage type)
__device__ __forceinline__ void unpack16(const uint4& v, float* o, const float*) {
  o[0] = __uint_as_float(v.x); o[1] = __uint_as_float(v.y); o[2] = __uint_as_float(v.z); o[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4& v, float* o, const bf16*) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { o[2 * i] = __uint_as_float(w[i] << 16); o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}

// Indexer scores for long candidate lists with 256-byte key rows (the benchmark's indexer width), one node per CTA in z:
// eight lanes share an entry, each holding its 32-byte slice of the node's queries in registers, so the inner product runs
// from registers (the thread-per-entry kernel above reads a query value from shared memory for every multiply-add and is
// bound by that); a CTA covers kRows256PerCta entries (the set-up of a CTA is amortised over them), four entries of a
// lane group in flight.  grid (ceil(entries / kRows256PerCta), B, D).
constexpr int kRows256PerCta = 2048;
template <typename T>
__global__ void __launch_bounds__(256) idx_score_rows256_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                                const tsv_scratch sc, char* __restrict__ ws) {
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  const int b = blockIdx.y, n = blockIdx.z, D = s.D, di = s.di, HI = s.HI;
  constexpr int V = Vec<T>::N, EL = 2 * V;
  {   // cheap exit: even with every ancestor closing a block, no node of this sequence has more than topk candidates
    const int L0 = c.L[b];
    if (L0 < 0 || L0 / s.m_csa + D <= s.topk || (int)(blockIdx.x * kRows256PerCta) >= L0 / s.m_csa) return;
  }
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, nullptr, nullptr);
  if (tm.status || n >= tm.nn || (int)(blockIdx.x * kRows256PerCta) >= tm.n_csa) return;
  {   // does this node rank?  candidates = committed entries + blocks closed at its strict ancestors
    int extra = 0;
    for (int j = 0; j < n; ++j) if (((tm.anc[n] >> j) & 1u) && sc.csa_done[(size_t)b * D + j]) ++extra;
    if (tm.n_csa + extra <= s.topk) return;
  }
  const int grp = threadIdx.x >> 3, gl = threadIdx.x & 7;
  const T* iq = reinterpret_cast<const T*>(nd.iq) + ((size_t)b * D + n) * HI * di;
  float q[4][EL], iwreg[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    iwreg[h] = h < HI ? nd.iw[((size_t)b * D + n) * HI + h] : 0.f;
    float t0[V], t1[V];
    if (h < HI) { ld16(iq + h * di + gl * EL, t0); ld16(iq + h * di + gl * EL + V, t1); }
#pragma unroll
    for (int j = 0; j < V; ++j) { q[h][j] = h < HI ? t0[j] : 0.f; q[h][V + j] = h < HI ? t1[j] : 0.f; }
  }
  const RowAddr ikr = csa_rows_of(c, s, b);
  const T* ik0 = reinterpret_cast<const T*>(c.csa_ik) + (size_t)ikr.row0 * di;
  float* sw = reinterpret_cast<float*>(ws + pl.off_scores) + ((size_t)b * D + n) * pl.score_ld;
  const int n_csa = tm.n_csa, e_base = blockIdx.x * kRows256PerCta, e_end = min(n_csa, e_base + kRows256PerCta);
#pragma unroll 1
  for (int base = e_base; base < e_end; base += 128) {          // uniform trip count: the shuffles need the whole warp
    uint4 raw[4][2];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = base + grp + 32 * u;
      const uint4* rowp = reinterpret_cast<const uint4*>(ik0 + (size_t)ikr.rel(e < n_csa ? e : 0) * di) + gl * 2;
      raw[u][0] = __ldg(rowp); raw[u][1] = __ldg(rowp + 1);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float kk[EL];
      unpack16(raw[u][0], kk, (const T*)nullptr);
      unpack16(raw[u][1], kk + V, (const T*)nullptr);
      float tot = 0.f;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        float pp = 0.f;
#pragma unroll
        for (int j = 0; j < EL; ++j) pp = fmaf(q[h][j], kk[j], pp);
        pp += __shfl_xor_sync(0xffffffffu, pp, 1);
        pp += __shfl_xor_sync(0xffffffffu, pp, 2);
        pp += __shfl_xor_sync(0xffffffffu, pp, 4);
        tot = fmaf(iwreg[h], fmaxf(pp, 0.f), tot);
      }
      const int e = base + grp + 32 * u;
      if (gl == 0 && e < n_csa) sw[e] = tot;
    }
  }
}

// staging area of the rows a ranking CTA scores itself (256-byte indexer rows, padded in shared memory)
constexpr int kStageRows = 128, kStagePitch = 272;   // two buffers of kStageRows rows

// PAGED: the caches live in a paged pool (a separate instantiation: the flat layout's ranking path is a tuned latency
// chain and keeps exactly its code)
template <typename T, bool PAGED>
__global__ void __launch_bounds__(256) topk_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                   const tsv_scratch sc, int32_t* __restrict__ topk_user, char* __restrict__ ws,
                                                   int32_t* __restrict__ status) {
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ PathEntries pe;
  __shared__ float extra[TSV_MAX_D];
  __shared__ int hist[256];
  __shared__ int wsum[9];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the tile plan may start its selection-independent part
  const int n = blockIdx.x, b = blockIdx.y, D = s.D, k = s.topk;
  int32_t* sel = reinterpret_cast<int32_t*>(ws + pl.off_sel) + ((size_t)b * D + n) * k;
  int32_t* selcnt = reinterpret_cast<int32_t*>(ws + pl.off_selcnt) + (size_t)b * D + n;
  int32_t* usr = topk_user ? topk_user + ((size_t)b * D + n) * k : nullptr;
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
  if (threadIdx.x == 0) {
    if (tm.status && n == 0) atomicOr(status + b, tm.status);
    if (!tm.status && n < tm.nn) path_entries(pe, tm, s, n, sc.csa_done + (size_t)b * D, sc.hca_done + (size_t)b * D);
  }
  __syncthreads();
  if (tm.status || n >= tm.nn) {
    for (int i = threadIdx.x; i < k; i += blockDim.x) { sel[i] = -1; if (usr) usr[i] = -1; }
    if (threadIdx.x == 0) *selcnt = 0;
    return;
  }
  const int n_csa = tm.n_csa, n_cand = n_csa + pe.n_newc;
  if (n_cand <= k) {                                           // everything is selected: no ranking
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
      const int v = i < n_csa ? i : (i < n_cand ? pe.newc_blk[i - n_csa] : -1);
      sel[i] = v; if (usr) usr[i] = v;
    }
    if (threadIdx.x == 0) *selcnt = n_cand;
    return;
  }
  // scores of the in-tree entries on this node's path: warp w takes entries w, w+8, ...
  {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const T* iq = reinterpret_cast<const T*>(nd.iq) + ((size_t)b * D + n) * s.HI * s.di;
    for (int i = w; i < pe.n_newc; i += 8) {
      const T* ik = reinterpret_cast<const T*>(sc.new_csa_ik) + ((size_t)b * D + pe.newc[i]) * s.di;
      float tot = 0.f;
      for (int h = 0; h < s.HI; ++h) {
        float p = 0.f;
        for (int t = lane; t < s.di; t += 32) p = fmaf(to_f(iq[h * s.di + t]), to_f(ik[t]), p);
        p = warp_sum(p);
        tot = fmaf(nd.iw[((size_t)b * D + n) * s.HI + h], fmaxf(p, 0.f), tot);
      }
      if (lane == 0) extra[i] = tot;
    }
  }
  const float* score_sm = nullptr;                    // scores of the committed entries in shared memory (set below), else in the workspace
  if (pl.idx_fused) {
    // short candidate lists: the committed entries are scored here as well (same formula as idx_score_kernel: thread per
    // entry, the node's indexer queries in shared memory), into the score array the radix passes read
    extern __shared__ __align__(16) float iq_sm[];    // [HI][di], then the staged rows
    const int HI = s.HI, di = s.di;
    constexpr int V = Vec<T>::N;
    const T* iq = reinterpret_cast<const T*>(nd.iq) + ((size_t)b * D + n) * HI * di;
    for (int i = threadIdx.x; i < HI * di; i += blockDim.x) iq_sm[i] = to_f(iq[i]);
    __syncthreads();
    RowAddr ikr;
    if (PAGED) ikr = csa_rows_of(c, s, b); else { ikr.pt = nullptr; ikr.per_page = 1; ikr.row0 = c.csa_row0[b]; }
    const T* ik0 = reinterpret_cast<const T*>(c.csa_ik) + (size_t)ikr.row0 * di;
    float* sw = reinterpret_cast<float*>(ws + pl.off_scores) + ((size_t)b * D + n) * pl.score_ld;
    if ((size_t)di * sizeof(T) == 256 && HI <= 4 && blockDim.x == 256) {
      // Rows of 256 bytes (the benchmark's indexer width).  Few CTAs rank and each is a chain of its own, so load latency
      // and arithmetic must not follow each other: the rows are staged in shared memory by 16-byte asynchronous copies,
      // kStageRows rows per round in two buffers, the copies of the next round under the arithmetic of the current one.
      // Eight lanes share an entry, lane l holding bytes [16 l, 16 l + 16) of both 128-byte halves of the node's
      // queries in registers; the per-head dot products are completed by three shuffles.
      constexpr int EL = 2 * V;                        // row elements per lane
      const int grp = threadIdx.x >> 3, gl = threadIdx.x & 7;
      float q[4][EL], iwreg[4];
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        iwreg[h] = h < HI ? nd.iw[((size_t)b * D + n) * HI + h] : 0.f;
#pragma unroll
        for (int j = 0; j < EL; ++j) q[h][j] = h < HI ? iq_sm[h * di + (j < V ? gl * V + j : di / 2 + gl * V + (j - V))] : 0.f;
      }
      unsigned char* stage = reinterpret_cast<unsigned char*>(iq_sm + HI * di);
      // the scores stay in shared memory: such a list has at most kIdxFusedMax + D candidates, which the radix passes
      // below keep in registers, so nothing else reads them (written to and read back from global memory they cost a
      // round trip of the chain)
      float* ssm = reinterpret_cast<float*>(stage + 2 * kStageRows * kStagePitch);
      score_sm = ssm;
      const uint32_t stage_s = (uint32_t)__cvta_generic_to_shared(stage);
      const char* ikb = reinterpret_cast<const char*>(ik0);
      auto issue = [&](int rd) {                         // rows [rd kStageRows, ..) into buffer rd & 1; one group per call
        const int base = rd * kStageRows, nrow = min(kStageRows, n_csa - base);
        const uint32_t dst = stage_s + (uint32_t)(rd & 1) * (kStageRows * kStagePitch);
        if (PAGED) {                                       // paged pool: a page-table look-up per row
#pragma unroll
          for (int i = 0; i < kStageRows * 16 / 256; ++i) {
            const int idx = threadIdx.x + 256 * i, row = idx >> 4, c16 = idx & 15;
            if (row < nrow)
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + row * kStagePitch + c16 * 16),
                           "l"(ikb + (size_t)ikr.rel(base + row) * 256 + c16 * 16) : "memory");
          }
        } else {
#pragma unroll
          for (int i = 0; i < kStageRows * 16 / 256; ++i) {
            const int idx = threadIdx.x + 256 * i, row = idx >> 4, c16 = idx & 15;
            if (row < nrow)
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + row * kStagePitch + c16 * 16),
                           "l"(ikb + (size_t)(base + row) * 256 + c16 * 16) : "memory");
          }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      const int nrd = (n_csa + kStageRows - 1) / kStageRows;
      issue(0);
      for (int rd = 0; rd < nrd; ++rd) {                 // uniform trip count: barriers and shuffles below
        if (rd + 1 < nrd) issue(rd + 1); else asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // round rd has landed (this thread's copies)
        __syncthreads();
        const int base = rd * kStageRows, nrow = min(kStageRows, n_csa - base);
        const unsigned char* buf = stage + (size_t)(rd & 1) * (kStageRows * kStagePitch);
#pragma unroll
        for (int r0 = 0; r0 < kStageRows; r0 += 32) {
          const int row = r0 + grp;
          const unsigned char* rp = buf + (row < nrow ? row : 0) * kStagePitch + gl * 16;
          const uint4 lo = *reinterpret_cast<const uint4*>(rp), hi = *reinterpret_cast<const uint4*>(rp + 128);
          float kk[EL];
          unpack16(lo, kk, (const T*)nullptr);
          unpack16(hi, kk + V, (const T*)nullptr);
          float tot = 0.f;
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            float pp = 0.f;
#pragma unroll
            for (int j = 0; j < EL; ++j) pp = fmaf(q[h][j], kk[j], pp);
            pp += __shfl_xor_sync(0xffffffffu, pp, 1);
            pp += __shfl_xor_sync(0xffffffffu, pp, 2);
            pp += __shfl_xor_sync(0xffffffffu, pp, 4);
            tot = fmaf(iwreg[h], fmaxf(pp, 0.f), tot);
          }
          if (gl == 0 && row < nrow) ssm[base + row] = tot;
        }
        __syncthreads();                                 // the buffer is refilled two rounds on
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else
    for (int e = threadIdx.x; e < n_csa; e += blockDim.x) {
      float acc[8];
#pragma unroll
      for (int h = 0; h < 8; ++h) acc[h] = 0.f;
      // the key row is fetched 8 x 16 bytes at a time, all loads of a batch in flight before the first use (few CTAs
      // rank, so a thread cannot count on other warps to hide its load latency)
      for (int c0 = 0; c0 < di / V; c0 += 8) {
        uint4 raw[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          raw[u] = (c0 + u < di / V) ? __ldg(reinterpret_cast<const uint4*>(ik0 + (size_t)(PAGED ? ikr.rel(e) : (int64_t)e) * di + (c0 + u) * V)) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (c0 + u < di / V) {
            float kk[V];
            unpack16(raw[u], kk, (const T*)nullptr);
#pragma unroll
            for (int h = 0; h < 8; ++h) {
              if (h < HI) {
                const float* qv = iq_sm + h * di + (c0 + u) * V;
#pragma unroll
                for (int t = 0; t < V; ++t) acc[h] = fmaf(qv[t], kk[t], acc[h]);
              }
            }
          }
        }
      }
      float tot = 0.f;
#pragma unroll
      for (int h = 0; h < 8; ++h)
        if (h < HI) tot = fmaf(nd.iw[((size_t)b * D + n) * HI + h], fmaxf(acc[h], 0.f), tot);
      sw[e] = tot;
    }
  }
  if (threadIdx.x == 0) { sh_prefix = 0; sh_remaining = k; }
  __syncthreads();
  const float* scores = reinterpret_cast<const float*>(ws + pl.off_scores) + ((size_t)b * D + n) * pl.score_ld;
  // order-preserving keys; lists of up to 9 x 256 candidates keep them in registers for the five passes below (candidate
  // i = threadIdx.x + 256 j is key j of its thread), longer lists read the scores again
  constexpr int KREG = 9;
  static_assert(kIdxFusedMax + TSV_MAX_D <= KREG * 256, "lists scored in shared memory must fit the in-register key path");
  const bool in_regs = n_cand <= KREG * 256;
  uint32_t kreg[KREG];
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < KREG; ++j) {
      const int i = threadIdx.x + 256 * j;
      kreg[j] = i < n_cand ? order_key(i < n_csa ? (score_sm ? score_sm[i] : __ldcg(scores + i)) : extra[i - n_csa]) : 0u;
    }
  }
  auto key_of = [&](int i) { return order_key(i < n_csa ? __ldcg(scores + i) : extra[i - n_csa]); };
  // Long lists are scanned in rounds: per round a thread takes eight groups of four consecutive candidates (groups g0,
  // g0 + gstride, ...; key 4u + j is candidate 4 (g0 + gstride u) + j; a round of all threads covers 4 ground candidates
  // from i_lo on).  A node's list is scanned by one CTA, so latency has to be covered inside the thread: the eight
  // 16-byte loads of a round are issued unconditionally (group index clamped to the row; rows are padded to whole
  // groups) and before anything that branches, and the next round's loads are issued before the current round's keys are
  // used.  `full` (uniform over the threads that share i_lo, i_hi) says that every candidate of the round is a committed
  // entry below i_hi, so that the body needs no range checks.
  auto scan32 = [&](int first_g, int gstride, int ground, int i_lo, int i_hi, auto&& body) {
    const float4* s4 = reinterpret_cast<const float4*>(scores);
    const int gmax = pl.score_ld / 4 - 1;
    const int nround = i_hi > i_lo ? (i_hi - i_lo + 4 * ground - 1) / (4 * ground) : 0;
    const int i_full = min(i_hi, n_csa);
    float4 va[8], vb[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) va[u] = __ldg(s4 + min(first_g + gstride * u, gmax));
    for (int rd = 0; rd < nround; ++rd) {
      const int g0 = first_g + rd * ground;
      if (rd + 1 < nround) {
#pragma unroll
        for (int u = 0; u < 8; ++u) vb[u] = __ldg(s4 + min(g0 + ground + gstride * u, gmax));
      }
      const bool full = i_lo + (rd + 1) * 4 * ground <= i_full;
      uint32_t kk[32];
      if (full) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          kk[4 * u] = order_key(va[u].x); kk[4 * u + 1] = order_key(va[u].y);
          kk[4 * u + 2] = order_key(va[u].z); kk[4 * u + 3] = order_key(va[u].w);
        }
      } else {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float f[4] = {va[u].x, va[u].y, va[u].z, va[u].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int i = 4 * (g0 + gstride * u) + j;
            kk[4 * u + j] = i < i_hi ? order_key(i < n_csa ? f[j] : extra[i - n_csa]) : 0u;
          }
        }
      }
      body(kk, g0, full);
#pragma unroll
      for (int u = 0; u < 8; ++u) va[u] = vb[u];
    }
  };
  uint32_t mask = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    if (in_regs) {
#pragma unroll
      for (int j = 0; j < KREG; ++j) {
        const uint32_t key = kreg[j];
        if (threadIdx.x + 256 * j < n_cand && (key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
      }
    } else {
      scan32(threadIdx.x, 256, 2048, 0, n_cand, [&](const uint32_t (&kk)[32], int g0, bool full) {
#pragma unroll
        for (int q = 0; q < 32; ++q)
          if ((full || 4 * (g0 + 256 * (q >> 2)) + (q & 3) < n_cand) && (kk[q] & mask) == prefix)
            atomicAdd(&hist[(kk[q] >> shift) & 255u], 1);
      });
    }
    __syncthreads();
    if (threadIdx.x < 32) {                           // warp 0 finds the bin holding the rem-th largest key: lane l owns bins 255-8l .. 248-8l
      const int lane = threadIdx.x, rem = sh_remaining;
      int h[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { h[j] = hist[255 - (lane * 8 + j)]; tot += h[j]; }
      int incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
      const int excl = incl - tot;
      if (excl < rem && incl >= rem) {
        int cum = excl, bin = 255 - lane * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) { if (cum + h[j] >= rem) { bin = 255 - (lane * 8 + j); break; } cum += h[j]; }
        sh_prefix = prefix | ((uint32_t)bin << shift);
        sh_remaining = rem - cum;
      }
    }
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  const uint32_t thr = sh_prefix;       // key of the k-th largest score
  const int r = sh_remaining;           // how many of the scores equal to it are taken (lowest indices)
  uint8_t* selmask = pl.tc ? reinterpret_cast<uint8_t*>(ws + pl.off_selmask) + ((size_t)b * D + n) * pl.mask_ld : nullptr;   // the selection as a byte per candidate (for the tile plan)
  if (!in_regs) {
    // Long lists: warp w owns a contiguous share of the candidates (whole 128-candidate steps: a lane holds four
    // consecutive candidates of a step) and walks it twice, eight steps per round: first counting the
    // keys above and equal to the threshold, then (after one exchange of the warps' counts) writing the selected indices
    // in ascending order at positions found with ballots.
    __shared__ int wgt[8], weq[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int share = ((n_cand + 7) / 8 + 127) & ~127;
    const int beg = w * share, end = min(n_cand, beg + share);
    int cg = 0, ce = 0;
    scan32(beg / 4 + lane, 32, 256, beg, end, [&](const uint32_t (&kk)[32], int g0, bool full) {
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const bool in = full || 4 * (g0 + 32 * (q >> 2)) + (q & 3) < end;
        cg += in && kk[q] > thr; ce += in && kk[q] == thr;
      }
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { cg += __shfl_xor_sync(0xffffffffu, cg, o); ce += __shfl_xor_sync(0xffffffffu, ce, o); }
    if (lane == 0) { wgt[w] = cg; weq[w] = ce; }
    __syncthreads();
    int eq_base = 0, out_base = 0;
    for (int x = 0; x < w; ++x) { eq_base += weq[x]; out_base += wgt[x]; }
    out_base += min(r, eq_base);                       // of the equal keys before this share, the first r are taken
    const uint32_t lt = (1u << lane) - 1u;
    scan32(beg / 4 + lane, 32, 256, beg, end, [&](const uint32_t (&kk)[32], int g0, bool full) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int ib = 4 * (g0 + 32 * u);              // this lane's four candidates of the step
        bool eq[4], take[4];
        uint32_t eqm[4], tkm[4];
        int run = eq_base, neq = 0, ntk = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          eq[j] = (full || ib + j < end) && kk[4 * u + j] == thr;
          eqm[j] = __ballot_sync(0xffffffffu, eq[j]);
          run += __popc(eqm[j] & lt); neq += __popc(eqm[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          take[j] = ((full || ib + j < end) && kk[4 * u + j] > thr) || (eq[j] && run < r);
          run += eq[j];
          tkm[j] = __ballot_sync(0xffffffffu, take[j]);
        }
        int pos = out_base;
#pragma unroll
        for (int j = 0; j < 4; ++j) { pos += __popc(tkm[j] & lt); ntk += __popc(tkm[j]); }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (selmask && (full || ib + j < end)) selmask[ib + j] = (uint8_t)take[j];
          if (take[j]) {
            const int i = ib + j, v = i < n_csa ? i : pe.newc_blk[i - n_csa];
            sel[pos] = v; if (usr) usr[pos] = v;
            ++pos;
          }
        }
        eq_base += neq; out_base += ntk;
      }
    });
    if (threadIdx.x == 0) *selcnt = k;
    return;
  }
  int eq_base = 0, out_base = 0;
  for (int i0 = 0, j0 = 0; i0 < n_cand; i0 += blockDim.x, ++j0) {
    const int i = i0 + threadIdx.x;
    uint32_t key = 0;
    if (i < n_cand) {
      if (in_regs) {
#pragma unroll
        for (int j = 0; j < KREG; ++j) if (j == j0) key = kreg[j];
      } else key = key_of(i);
    }
    const int eq = (i < n_cand) && key == thr, gt = (i < n_cand) && key > thr;
    int tot_eq, tot_take;
    const int eq_rank = eq_base + block_excl_scan_256(eq, wsum, tot_eq);
    const int take = gt || (eq && eq_rank < r);
    const int pos = out_base + block_excl_scan_256(take, wsum, tot_take);
    if (selmask && i < n_cand) selmask[i] = (uint8_t)take;
    if (take) {
      const int v = i < n_csa ? i : pe.newc_blk[i - n_csa];
      sel[pos] = v; if (usr) usr[pos] = v;
    }
    eq_base += tot_eq; out_base += tot_take;
  }
  if (threadIdx.x == 0) *selcnt = k;
}

int launch_tva_select(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                      int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st) {
  const bool bf = s.dtype == TSV_BF16;
  if (p.need_scores && !p.idx_fused) {
    const int pref_cap = (int)(s.max_L / s.m_csa);
    dim3 grid((pref_cap + 255) / 256, s.B, s.D <= 8 ? s.D : 8);        // z: slabs of nodes, so a ranked sequence is scored by many CTAs
    const size_t sm = (size_t)32 * s.di * sizeof(float);
    if (grid.x > 0 && idx_score_tc_applies(s)) {
      launch_idx_score_tc(s, p, c, nd, sc, ws, status, st);             // all nodes of a sequence at once, on the tensor core
    } else if (grid.x > 0 && (size_t)s.di * (bf ? 2 : 4) == 256 && s.HI <= 4) {
      const dim3 g8((pref_cap + kRows256PerCta - 1) / kRows256PerCta, s.B, s.D);   // one node per CTA: queries in registers
      if (bf) { TSV_PREP(idx_score_rows256_kernel<bf16>); idx_score_rows256_kernel<bf16><<<g8, 256, 0, st>>>(s, p, c, nd, sc, ws); }
      else { TSV_PREP(idx_score_rows256_kernel<float>); idx_score_rows256_kernel<float><<<g8, 256, 0, st>>>(s, p, c, nd, sc, ws); }
      count_launch();
    } else if (grid.x > 0) {
      if (bf) {
        cudaFuncSetAttribute(idx_score_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        TSV_PREP(idx_score_kernel<bf16>);
        idx_score_kernel<bf16><<<grid, 256, sm, st>>>(s, p, c, nd, sc, ws);
      } else {
        cudaFuncSetAttribute(idx_score_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        TSV_PREP(idx_score_kernel<float>);
        idx_score_kernel<float><<<grid, 256, sm, st>>>(s, p, c, nd, sc, ws);
      }
      count_launch();
    }
  }
  if (topk_long_applies(s, p)) return launch_topk_long(s, p, c, nd, sc, topk_idx, ws, status, st);
  if (topk_fused_applies(s, p)) return launch_topk_fused(s, p, c, nd, sc, topk_idx, ws, status, st);
  dim3 g2(s.D, s.B);
  const bool paged = c.page_table != nullptr;
  size_t sm2 = p.idx_fused ? (size_t)s.HI * s.di * sizeof(float) : 0;         // the node's indexer queries ...
  if (p.idx_fused && (size_t)s.di * (bf ? 2 : 4) == 256 && s.HI <= 4) sm2 += (size_t)2 * kStageRows * kStagePitch + (size_t)kIdxFusedMax * sizeof(float);   // ... the staged rows (two buffers), the scores
#define TSV_TOPK_LAUNCH(T_, PG_)                                                                                        \
  do {                                                                                                                  \
    TSV_PREP((topk_kernel<T_, PG_>));                                                                                   \
    if (sm2 > 48 * 1024) cudaFuncSetAttribute(topk_kernel<T_, PG_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2); \
    topk_kernel<T_, PG_><<<g2, 256, sm2, st>>>(s, p, c, nd, sc, topk_idx, ws, status);                                  \
  } while (0)
  if (bf) { if (paged) TSV_TOPK_LAUNCH(bf16, true); else TSV_TOPK_LAUNCH(bf16, false); }
  else { if (paged) TSV_TOPK_LAUNCH(float, true); else TSV_TOPK_LAUNCH(float, false); }
#undef TSV_TOPK_LAUNCH
  count_launch();
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
