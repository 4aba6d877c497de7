// branch_state_build: chain-private online compression along every root-to-node path.
//
// Grid (sequence, element slab).  The scalar part of every fold (max gate, sum of weights, the two
// blend coefficients, done flags) is a chain over at most 32 nodes: thread 0 of each CTA loads all
// gates and parents up front (independent loads, one memory latency) and walks the chain in
// registers.  Each thread then owns ONE vector element: it loads that element of every node's
// compression vector up front, folds along the tree with the inherited values kept in shared
// memory (indexed by parent), and stores states and closed entries.  No load depends on a store.
#include "kernels.h"

namespace tsv {

struct FoldCoef {
  float a, b, s;     // acc' = a * acc_parent + b * c ; s = sum of weights after the fold
  int32_t done;      // block closes at this node
  int32_t empty;     // the inherited block holds no token (inherited numbers are ignored)
};

__device__ __forceinline__ void scalar_fold(FoldCoef& fc, float& mx_out, float& s_out, int p, int blk, float mxp, float sp, float g) {
  const bool empty = (p % blk) == 0;
  float mx2, a, b, s2;
  if (empty) { mx2 = g; a = 0.f; b = 1.f; s2 = 1.f; }
  else {
    mx2 = fmaxf(mxp, g);
    a = expf(mxp - mx2);
    b = expf(g - mx2);
    s2 = fmaf(sp, a, b);
  }
  fc.a = a; fc.b = b; fc.s = s2; fc.empty = empty;
  fc.done = ((p + 1) % blk) == 0;
  mx_out = fc.done ? 0.f : mx2;
  s_out = fc.done ? 0.f : s2;
}

constexpr int kBsbThreads = 128;

// DEFER: the C128-deferred schedule is on (a separate instantiation, so that the timely schedule's code is untouched by it)
template <typename T, int DMAX, bool DEFER>
__global__ void __launch_bounds__(kBsbThreads) bsb_kernel(const tsv_shape s, const tsv_cache c, const tsv_nodes nd,
                                                          const tsv_scratch sc, int32_t* __restrict__ status) {
  extern __shared__ float hist[];                      // [D][kBsbThreads] post-fold value of this thread's element per node
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ FoldCoef fcs[TSV_MAX_D], fhs[TSV_MAX_D];
  __shared__ float cmx[TSV_MAX_D], cs[TSV_MAX_D], hmx[TSV_MAX_D], hs[TSV_MAX_D];   // thread 0's chain state per node
  const int b = blockIdx.x, D = s.D;
  const int d = s.d, di = s.di;
  const int e = blockIdx.y * kBsbThreads + threadIdx.x;   // element index: [0,d) CSA kv | [d,d+di) CSA indexer key | [d+di,2d+di) HCA kv
  const bool live = e < 2 * d + di;
  const int which = e < d ? 0 : (e < d + di ? 1 : 2);
  const int el = which == 0 ? e : (which == 1 ? e - d : e - d - di);
  const int dim = which == 1 ? di : d;
  const T* cin = reinterpret_cast<const T*>(which == 0 ? nd.c_csa : (which == 1 ? nd.ikc : nd.c_hca));
  const float* pers = which == 0 ? c.csa_acc_kv : (which == 1 ? c.csa_acc_ik : c.hca_acc_kv);
  // C128-deferred schedule: the HCA slabs of a sequence in which no HCA block can close inside the tree have nothing to do
  // (they learn the length first, one load, and leave before fetching any vector)
  if (DEFER && which == 2 && blockIdx.y * kBsbThreads >= (unsigned)(d + di) && hca_deferred(s, c.L[b])) return;
  // issue this thread's loads before the scalar chain is known (padding slots load too: the memory is there)
  float cv[DMAX];
#pragma unroll
  for (int n = 0; n < DMAX; ++n) cv[n] = (live && n < D) ? to_f(cin[((size_t)b * D + n) * dim + el]) : 0.f;
  const float pv = live ? pers[(size_t)b * dim + el] : 0.f;
  float gcl = 0.f, ghl = 0.f;                        // lane n of warp 0 fetches node n's gates; thread 0 collects them by shuffle
  if (threadIdx.x < D) { gcl = nd.g_csa[(size_t)b * D + threadIdx.x]; ghl = nd.g_hca[(size_t)b * D + threadIdx.x]; }
  float pcm = 0.f, pcs = 0.f, phm = 0.f, phs = 0.f;
  if (threadIdx.x == 0) { pcm = c.csa_mx[b]; pcs = c.csa_s[b]; phm = c.hca_mx[b]; phs = c.hca_s[b]; }
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
  float gc[DMAX], gh[DMAX];
  if (threadIdx.x < 32) {
#pragma unroll
    for (int n = 0; n < DMAX; ++n) { gc[n] = __shfl_sync(0xffffffffu, gcl, n); gh[n] = __shfl_sync(0xffffffffu, ghl, n); }
  }

  const bool hdef = DEFER && hca_deferred(s, tm.L) && !tm.status;     // (tm.L is 0 for a flagged length: such a sequence commits nothing)
  if (threadIdx.x == 0) {
    const bool writer = blockIdx.y == 0;
    if (tm.status && writer) atomicOr(status + b, tm.status);
    const int nn = tm.status ? 0 : tm.nn;
#pragma unroll
    for (int n = 0; n < DMAX; ++n) {
      if (n < D) {
        float m1 = 0.f, s1 = 0.f, m2 = 0.f, s2 = 0.f;
        if (n < nn) {
          const int p = tm.L + tm.depth[n], par = tm.parent[n];
          float mp = pcm, sp = pcs, mq = phm, sq = phs;
          if (n) { mp = cmx[par]; sp = cs[par]; mq = hmx[par]; sq = hs[par]; }
          scalar_fold(fcs[n], m1, s1, p, s.m_csa, mp, sp, gc[n]);
          if (hdef) fhs[n].done = 0; else scalar_fold(fhs[n], m2, s2, p, s.m_hca, mq, sq, gh[n]);
        } else {
          fcs[n].done = fhs[n].done = 0;
        }
        cmx[n] = m1; cs[n] = s1; hmx[n] = m2; hs[n] = s2;
        if (writer) {
          sc.csa_mx[(size_t)b * D + n] = m1; sc.csa_s[(size_t)b * D + n] = s1;
          if (!hdef) { sc.hca_mx[(size_t)b * D + n] = m2; sc.hca_s[(size_t)b * D + n] = s2; }
          sc.csa_done[(size_t)b * D + n] = (uint8_t)fcs[n].done;
          sc.hca_done[(size_t)b * D + n] = (uint8_t)fhs[n].done;
        }
      }
    }
  }
  __syncthreads();
  if (!live || (which == 2 && hdef)) return;
  const int nn = tm.status ? 0 : tm.nn;
  float* sacc = which == 0 ? sc.csa_acc_kv : (which == 1 ? sc.csa_acc_ik : sc.hca_acc_kv);
  T* newe = reinterpret_cast<T*>(which == 0 ? sc.new_csa_kv : (which == 1 ? sc.new_csa_ik : sc.new_hca_kv));
  const FoldCoef* fc = which == 2 ? fhs : fcs;
#pragma unroll
  for (int n = 0; n < DMAX; ++n) {
    if (n < D) {
      const size_t o = ((size_t)b * D + n) * dim + el;
      float acc = 0.f, ent = 0.f;
      if (n < nn) {
        const FoldCoef f = fc[n];
        if (f.empty) acc = cv[n];
        else {
          const float ap = n ? hist[tm.parent[n] * kBsbThreads + threadIdx.x] : pv;
          acc = fmaf(f.a, ap, f.b * cv[n]);
        }
        if (f.done) { ent = acc / f.s; acc = 0.f; }
      }
      hist[n * kBsbThreads + threadIdx.x] = acc;
      sacc[o] = acc;
      newe[o] = from_f<T>(ent);
    }
  }
}

int launch_bsb(const tsv_shape& s, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, int32_t* status, cudaStream_t st) {
  const int elems = 2 * s.d + s.di;
  const dim3 grid(s.B, (elems + kBsbThreads - 1) / kBsbThreads);
  const size_t sm = (size_t)s.D * kBsbThreads * sizeof(float);
  const bool defer = (s.flags & TSV_FLAG_HCA_DEFERRED) != 0, bf = s.dtype == TSV_BF16, small = s.D <= 8;
#define TSV_BSB_LAUNCH(T_, DM_, DF_)                                              \
  do {                                                                            \
    TSV_PREP((bsb_kernel<T_, DM_, DF_>));                                         \
    bsb_kernel<T_, DM_, DF_><<<grid, kBsbThreads, sm, st>>>(s, c, nd, sc, status); \
  } while (0)
  if (small) {
    if (bf) { if (defer) TSV_BSB_LAUNCH(bf16, 8, true); else TSV_BSB_LAUNCH(bf16, 8, false); }
    else { if (defer) TSV_BSB_LAUNCH(float, 8, true); else TSV_BSB_LAUNCH(float, 8, false); }
  } else {
    if (bf) { if (defer) TSV_BSB_LAUNCH(bf16, TSV_MAX_D, true); else TSV_BSB_LAUNCH(bf16, TSV_MAX_D, false); }
    else { if (defer) TSV_BSB_LAUNCH(float, TSV_MAX_D, true); else TSV_BSB_LAUNCH(float, TSV_MAX_D, false); }
  }
#undef TSV_BSB_LAUNCH
  count_launch();
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
