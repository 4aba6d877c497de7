// Per-node top-k over LONG candidate lists (more than topk_kernel keeps in registers), by a thread-block cluster per
// node: the list is split over the cluster's CTAs, each thread keeps 16 consecutive candidates' keys in registers for
// the whole selection, and the CTAs exchange only radix histograms and counts: each CTA ADDS its figures into the shared
// memory of its peers before a cluster barrier, so that after the barrier everything a CTA needs is local.
// Same result as topk_kernel: the exact k largest scores, ties to the lower candidate index, ascending output.
#include "select_common.cuh"

namespace tsv {

namespace lsel {

constexpr int THREADS = 512, KEYS = 16, CS = 8;          // threads per CTA, keys per thread, CTAs per cluster
constexpr int MAXC = THREADS * KEYS * CS;                // longest list the cluster path takes

__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// adds v to the same shared variable in CTA `rank` of the cluster (visible there after the next cluster barrier)
__device__ __forceinline__ void add_peer(int* p, uint32_t rank, int v) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
  asm volatile("red.relaxed.cluster.shared::cluster.add.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

}  // namespace lsel

template <typename T>
__global__ void __launch_bounds__(lsel::THREADS, 2) topk_long_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                                  const tsv_scratch sc, int32_t* __restrict__ topk_user,
                                                                  char* __restrict__ ws, int32_t* __restrict__ status) {
  using namespace lsel;
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ PathEntries pe;
  __shared__ float extra[TSV_MAX_D];
  __shared__ int hist[2][256];          // this CTA's histogram of the current digit
  __shared__ int tot[2][256];           // the cluster's histogram: every CTA adds its own into every CTA's copy
  __shared__ int wsum[THREADS / 32 + 1];
  __shared__ int before_sm[2];          // keys above / equal to the threshold in the CTAs of lower rank (added by them)
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int n = blockIdx.x / CS, b = blockIdx.y, D = s.D, k = s.topk;
  // every exit below is taken by all CTAs of a cluster alike (it depends on the node's facts only); after the last
  // cluster barrier no CTA touches a peer's memory, so they leave independently
  int32_t* sel = reinterpret_cast<int32_t*>(ws + pl.off_sel) + ((size_t)b * D + n) * k;
  int32_t* selcnt = reinterpret_cast<int32_t*>(ws + pl.off_selcnt) + (size_t)b * D + n;
  int32_t* usr = topk_user ? topk_user + ((size_t)b * D + n) * k : nullptr;
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
  if (threadIdx.x == 0) {
    if (tm.status && n == 0 && rank == 0) atomicOr(status + b, tm.status);
    if (!tm.status && n < tm.nn) path_entries(pe, tm, s, n, sc.csa_done + (size_t)b * D, sc.hca_done + (size_t)b * D);
  }
  __syncthreads();
  const int t = threadIdx.x, gt = (int)rank * THREADS + t;       // thread index within the cluster
  if (tm.status || n >= tm.nn) {
    for (int i = gt; i < k; i += CS * THREADS) { sel[i] = -1; if (usr) usr[i] = -1; }
    if (gt == 0) *selcnt = 0;
    return;
  }
  const int n_csa = tm.n_csa, n_cand = n_csa + pe.n_newc;
  if (n_cand <= k) {                                             // everything is selected: no ranking
    for (int i = gt; i < k; i += CS * THREADS) {
      const int v = i < n_csa ? i : (i < n_cand ? pe.newc_blk[i - n_csa] : -1);
      sel[i] = v; if (usr) usr[i] = v;
    }
    if (gt == 0) *selcnt = n_cand;
    return;
  }
  // this thread's candidates: 16 consecutive ones of the CTA's share (their committed scores were left in the workspace by
  // the scoring kernel: four 16-byte loads, issued before the in-tree entries are scored)
  const int share = ((n_cand + CS - 1) / CS + KEYS - 1) / KEYS * KEYS;      // <= THREADS * KEYS as n_cand <= MAXC
  const int i0 = (int)rank * share + t * KEYS;
  const bool owner = t * KEYS < share && i0 < n_cand;
  const float* scores = reinterpret_cast<const float*>(ws + pl.off_scores) + ((size_t)b * D + n) * pl.score_ld;
  float4 raw[KEYS / 4];
#pragma unroll
  for (int j = 0; j < KEYS / 4; ++j)
    raw[j] = (owner && i0 + 4 * j < n_csa) ? __ldg(reinterpret_cast<const float4*>(scores + i0) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
  {   // scores of the in-tree entries on this node's path (every CTA: at most D of them): warp w takes entries w, w + 16, ...
    const int lane = t & 31, w = t >> 5;
    const T* iq = reinterpret_cast<const T*>(nd.iq) + ((size_t)b * D + n) * s.HI * s.di;
    for (int i = w; i < pe.n_newc; i += THREADS / 32) {
      const T* ik = reinterpret_cast<const T*>(sc.new_csa_ik) + ((size_t)b * D + pe.newc[i]) * s.di;
      float acc = 0.f;
      for (int h = 0; h < s.HI; ++h) {
        float p = 0.f;
        for (int x = lane; x < s.di; x += 32) p = fmaf(to_f(iq[h * s.di + x]), to_f(ik[x]), p);
        p = warp_sum(p);
        acc = fmaf(nd.iw[((size_t)b * D + n) * s.HI + h], fmaxf(p, 0.f), acc);
      }
      if (lane == 0) extra[i] = acc;
    }
  }
  if (t < 256) { hist[0][t] = 0; tot[0][t] = 0; }
  if (t == 0) { sh_prefix = 0; sh_remaining = k; before_sm[0] = before_sm[1] = 0; }
  __syncthreads();
  cluster_sync();                                                 // every CTA's arrays are cleared before a peer adds to them
  uint32_t key[KEYS];
  uint32_t valid = 0;                                            // bit j: key j is a candidate
#pragma unroll
  for (int j = 0; j < KEYS; ++j) {
    const int i = i0 + j;
    const float f4[4] = {raw[j >> 2].x, raw[j >> 2].y, raw[j >> 2].z, raw[j >> 2].w};
    const bool v = owner && i < n_cand && t * KEYS + j < share;
    key[j] = v ? order_key(i < n_csa ? f4[j & 3] : extra[i - n_csa]) : 0u;
    valid |= (uint32_t)v << j;
  }
  // Four radix passes of 8 bits: the digit of the k-th largest key, high digit first.  Buffers alternate between passes:
  // the pair a pass does not use is cleared at its start (its last readers and writers finished before the previous
  // pass's barrier; the peers add to it only after this pass's barrier).
  uint32_t mask = 0;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass, buf = pass & 1;
    const uint32_t prefix = sh_prefix;
    if (t >= 256) { hist[buf ^ 1][t - 256] = 0; tot[buf ^ 1][t - 256] = 0; }
#pragma unroll
    for (int j = 0; j < KEYS; ++j) {
      const bool in = ((valid >> j) & 1u) && (key[j] & mask) == prefix;
      const uint32_t bin = in ? (key[j] >> shift) & 255u : 256u;
      // the scores of one list share their high digits: when the whole warp hits one bin, one lane adds for all
      int uniform;
      __match_all_sync(0xffffffffu, bin, &uniform);
      if (uniform) { if (in && (t & 31) == 0) atomicAdd(&hist[buf][bin], 32); }
      else if (in) atomicAdd(&hist[buf][bin], 1);
    }
    __syncthreads();
    if (t < 256) {
      const int v = hist[buf][t];
      if (v) {
#pragma unroll
        for (uint32_t r = 0; r < CS; ++r) add_peer(&tot[buf][t], r, v);
      }
    }
    cluster_sync();                                               // every CTA's histogram has been added everywhere
    if (t < 32) {                                                 // warp 0 finds the bin holding the rem-th largest key: lane l owns bins 255-8l .. 248-8l
      const int lane = t, rem = sh_remaining;
      int h[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { h[j] = tot[buf][255 - (lane * 8 + j)]; sum += h[j]; }
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
      const int excl = incl - sum;
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
  const int r_take = sh_remaining;      // how many of the scores equal to it are taken (lowest indices)
  // ordered compaction: keys above and equal to the threshold before this thread, in the CTA (one block scan of both
  // counts packed in a word) and in the CTAs before it (every CTA adds its totals into the CTAs of higher rank)
  int mine = 0;
#pragma unroll
  for (int j = 0; j < KEYS; ++j) {
    const bool v = (valid >> j) & 1u;
    mine += (int)(v && key[j] > thr) + ((int)(v && key[j] == thr) << 16);
  }
  int before;                            // exclusive scan of `mine` over the CTA's threads
  {
    const int lane = t & 31, w = t >> 5;
    int x = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    if (lane == 31) wsum[w] = x;
    __syncthreads();
    if (t == 0) {
      int run = 0;
      for (int i = 0; i < THREADS / 32; ++i) { const int v = wsum[i]; wsum[i] = run; run += v; }
      wsum[THREADS / 32] = run;
    }
    __syncthreads();
    before = wsum[w] + x - mine;
    if (t < (int)CS && t > (int)rank) { add_peer(&before_sm[0], (uint32_t)t, wsum[THREADS / 32] & 0xFFFF); add_peer(&before_sm[1], (uint32_t)t, wsum[THREADS / 32] >> 16); }
  }
  cluster_sync();                                                 // the counts of the CTAs before this one are there
  int eq_run = (before >> 16) + before_sm[1], pos = (before & 0xFFFF) + before_sm[0];
  pos += min(r_take, eq_run);             // of the equal keys before this thread, the first r_take are taken
  uint32_t mbytes[KEYS / 4] = {0u, 0u, 0u, 0u};             // the selection as a byte per candidate, for the tile plan
#pragma unroll
  for (int j = 0; j < KEYS; ++j) {
    const bool v = (valid >> j) & 1u, eq = v && key[j] == thr;
    if ((v && key[j] > thr) || (eq && eq_run < r_take)) {
      const int i = i0 + j, val = i < n_csa ? i : pe.newc_blk[i - n_csa];
      sel[pos] = val; if (usr) usr[pos] = val;
      ++pos;
      mbytes[j >> 2] |= 1u << (8 * (j & 3));
    }
    eq_run += eq;
  }
  if (owner && pl.tc)                                          // (i0 is a multiple of 16 and so is the row length)
    *reinterpret_cast<uint4*>(ws + pl.off_selmask + ((size_t)b * D + n) * pl.mask_ld + i0) = make_uint4(mbytes[0], mbytes[1], mbytes[2], mbytes[3]);
  if (gt == 0) *selcnt = k;
}

// Lists that topk_kernel would have to re-read from the score array pass after pass (more than its 9 x 256 register keys),
// up to the cluster's capacity.
bool topk_long_applies(const tsv_shape&, const TvaPlan& p) {
  return p.need_scores && !p.idx_fused && p.cand_cap > 9 * 256 && p.cand_cap <= lsel::MAXC;
}

int launch_topk_long(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                     int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(s.D * lsel::CS), (unsigned)s.B, 1);
  cfg.blockDim = dim3(lsel::THREADS, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = lsel::CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (s.dtype == TSV_BF16) { TSV_PREP(topk_long_kernel<bf16>); e = cudaLaunchKernelEx(&cfg, topk_long_kernel<bf16>, s, p, c, nd, sc, topk_idx, ws, status); }
  else { TSV_PREP(topk_long_kernel<float>); e = cudaLaunchKernelEx(&cfg, topk_long_kernel<float>, s, p, c, nd, sc, topk_idx, ws, status); }
  count_launch();
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
