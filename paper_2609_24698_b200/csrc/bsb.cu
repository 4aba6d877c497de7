// branch_state_build: chain-private online compression along every root-to-node path.
//
// Grid (sequence, element slab).  The scalar part of every fold (max gate, sum of weights, the two
// blend coefficients, done flags) follows the tree: in every CTA one warp per compressed layer (CSA,
// HCA) holds a node per lane, loads gates and parents up front (independent loads, one memory
// latency) and folds level by level, the parent's result arriving by shuffle.  Each thread then owns
// ONE vector element: it loads that element of every node's compression vector up front, folds along
// the tree with the inherited values kept in shared memory (indexed by parent), and stores states and
// closed entries.  No load depends on a store.
#include "kernels.h"

namespace tsv {

struct FoldCoef {
  float a, b, s;     // acc' = a * acc_parent + b * c ; s = sum of weights after the fold
  int32_t done;      // block closes at this node
  int32_t empty;     // the inherited block holds no token (inherited numbers are ignored)
};

// empty / done: position p opens / closes a block of blk tokens (they depend on the position alone: a caller that folds
// along a chain works them out ahead of it)
__device__ __forceinline__ void scalar_fold(FoldCoef& fc, float& mx_out, float& s_out, bool empty, bool done, float mxp, float sp, float g) {
  float mx2, a, b, s2;
  if (empty) { mx2 = g; a = 0.f; b = 1.f; s2 = 1.f; }
  else {
    mx2 = fmaxf(mxp, g);
    a = expf(mxp - mx2);
    b = expf(g - mx2);
    s2 = fmaf(sp, a, b);
  }
  fc.a = a; fc.b = b; fc.s = s2; fc.empty = empty;
  fc.done = done;
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
  const int b = blockIdx.x, D = s.D;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the selection may start the part of it that does not read this kernel's results
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
  T cvr[DMAX];                                         // kept as loaded: a conversion here would wait for the data before the tree's loads leave
#pragma unroll
  for (int n = 0; n < DMAX; ++n) cvr[n] = (live && n < D) ? cin[((size_t)b * D + n) * dim + el] : T(0.f);
  const float pv = live ? pers[(size_t)b * dim + el] : 0.f;
  // The scalar chains: warp 0 folds the CSA block states, warp 1 the HCA ones, lane n owning node n.  A node's fold needs
  // its parent's result, so the warp walks the tree level by level (nodes of one depth fold together, the parent's
  // running max and sum arrive by shuffle): as many steps as the tree is deep, not as it has nodes.
  const int lane = threadIdx.x & 31, chain = threadIdx.x >> 5;      // chain 0: CSA, 1: HCA (warps 2, 3 take no part)
  float gate = 0.f, pmx = 0.f, psum = 0.f;
  if (chain < 2 && lane < D) gate = (chain == 0 ? nd.g_csa : nd.g_hca)[(size_t)b * D + lane];
  if (chain < 2 && lane == 0) { pmx = (chain == 0 ? c.csa_mx : c.hca_mx)[b]; psum = (chain == 0 ? c.csa_s : c.hca_s)[b]; }
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);

  const bool hdef = DEFER && hca_deferred(s, tm.L) && !tm.status;     // (tm.L is 0 for a flagged length: such a sequence commits nothing)
  if (chain < 2) {
    const bool writer = blockIdx.y == 0;
    if (tm.status && writer && threadIdx.x == 0) atomicOr(status + b, tm.status);
    const int nn = tm.status ? 0 : tm.nn, n = lane;
    const bool valid = n < nn;
    const int depth = valid ? tm.depth[n] : -1, par = valid && n ? tm.parent[n] : 0;
    int maxd = depth;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) maxd = max(maxd, __shfl_xor_sync(0xffffffffu, maxd, o));
    FoldCoef fc;
    fc.a = fc.b = fc.s = 0.f; fc.done = 0; fc.empty = 0;
    float mx = 0.f, sm = 0.f;                          // this node's running max and sum after its fold
    const bool skip = chain == 1 && hdef;              // deferred schedule: no HCA branch states
    const int blk = chain == 0 ? s.m_csa : s.m_hca, p = tm.L + max(depth, 0);
    const bool opens = (p % blk) == 0, closes = ((p + 1) % blk) == 0;
    if (!skip) {
      for (int level = 0; level <= maxd; ++level) {    // uniform trip count
        const float mp = __shfl_sync(0xffffffffu, mx, par), sp = __shfl_sync(0xffffffffu, sm, par);
        if (depth == level)
          scalar_fold(fc, mx, sm, opens, closes, n ? mp : pmx, n ? sp : psum, gate);
      }
    }
    if (n < D) {
      (chain == 0 ? fcs : fhs)[n] = fc;
      if (writer) {
        if (chain == 0) { sc.csa_mx[(size_t)b * D + n] = mx; sc.csa_s[(size_t)b * D + n] = sm; sc.csa_done[(size_t)b * D + n] = (uint8_t)fc.done; }
        else {
          if (!hdef) { sc.hca_mx[(size_t)b * D + n] = mx; sc.hca_s[(size_t)b * D + n] = sm; }
          sc.hca_done[(size_t)b * D + n] = (uint8_t)fc.done;
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
        const float cvn = to_f(cvr[n]);
        if (f.empty) acc = cvn;
        else {
          const float ap = n ? hist[tm.parent[n] * kBsbThreads + threadIdx.x] : pv;
          acc = fmaf(f.a, ap, f.b * cvn);
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
