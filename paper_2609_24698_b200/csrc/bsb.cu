// branch_state_build: chain-private online compression along every root-to-node path.
// One CTA per sequence.  Thread 0 derives the tree facts and the scalar part of every fold
// (max gate, sum of weights, the two blend coefficients); then each thread owns a fixed set
// of vector elements and walks the nodes in index order (parents first), so the parent's
// post-fold value of an element is always one this same thread wrote earlier.
#include "kernels.h"

namespace tsv {

struct FoldCoef {
  float a, b, s;     // acc' = a * acc_parent + b * c ; s = sum of weights after the fold
  int32_t done;      // block closes at this node
  int32_t empty;     // the inherited block holds no token (inherited numbers are ignored)
};

__device__ inline void scalar_fold(FoldCoef& fc, float& mx_out, float& s_out, int p, int blk, float mxp, float sp, float g) {
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

template <typename T>
__global__ void __launch_bounds__(128) bsb_kernel(const tsv_shape s, const tsv_cache c, const tsv_nodes nd,
                                                  const tsv_scratch sc, int32_t* __restrict__ status) {
  __shared__ TreeMeta tm;
  __shared__ FoldCoef fcs[TSV_MAX_D], fhs[TSV_MAX_D];
  const int b = blockIdx.x, D = s.D;
  if (threadIdx.x == 0) {
    build_tree_meta(tm, s, c.L[b], nd.parent + (size_t)b * D, nd.n_nodes[b], c.csa_cap + b, c.hca_cap + b);
    if (tm.status) atomicOr(status + b, tm.status);
    const int nn = tm.status ? 0 : tm.nn;
    float cmx[TSV_MAX_D], cs[TSV_MAX_D], hmx[TSV_MAX_D], hs[TSV_MAX_D];
    for (int n = 0; n < D; ++n) {
      float m1 = 0.f, s1 = 0.f, m2 = 0.f, s2 = 0.f;
      if (n < nn) {
        const int p = tm.L + tm.depth[n], par = tm.parent[n];
        scalar_fold(fcs[n], m1, s1, p, s.m_csa, n ? cmx[par] : c.csa_mx[b], n ? cs[par] : c.csa_s[b], nd.g_csa[(size_t)b * D + n]);
        scalar_fold(fhs[n], m2, s2, p, s.m_hca, n ? hmx[par] : c.hca_mx[b], n ? hs[par] : c.hca_s[b], nd.g_hca[(size_t)b * D + n]);
      } else {
        fcs[n].done = fhs[n].done = 0;
      }
      cmx[n] = m1; cs[n] = s1; hmx[n] = m2; hs[n] = s2;
      sc.csa_mx[(size_t)b * D + n] = m1; sc.csa_s[(size_t)b * D + n] = s1;
      sc.hca_mx[(size_t)b * D + n] = m2; sc.hca_s[(size_t)b * D + n] = s2;
      sc.csa_done[(size_t)b * D + n] = (uint8_t)fcs[n].done;
      sc.hca_done[(size_t)b * D + n] = (uint8_t)fhs[n].done;
    }
  }
  __syncthreads();
  const int nn = tm.status ? 0 : tm.nn;
  const int d = s.d, di = s.di;
  // element index space: [0, d) CSA kv | [d, d+di) CSA indexer key | [d+di, 2d+di) HCA kv
  for (int e = threadIdx.x; e < 2 * d + di; e += blockDim.x) {
    const int which = e < d ? 0 : (e < d + di ? 1 : 2);
    const int el = which == 0 ? e : (which == 1 ? e - d : e - d - di);
    const int dim = which == 1 ? di : d;
    const float* pers = which == 0 ? c.csa_acc_kv : (which == 1 ? c.csa_acc_ik : c.hca_acc_kv);
    float* sacc = which == 0 ? sc.csa_acc_kv : (which == 1 ? sc.csa_acc_ik : sc.hca_acc_kv);
    const T* cin = reinterpret_cast<const T*>(which == 0 ? nd.c_csa : (which == 1 ? nd.ikc : nd.c_hca));
    T* newe = reinterpret_cast<T*>(which == 0 ? sc.new_csa_kv : (which == 1 ? sc.new_csa_ik : sc.new_hca_kv));
    const FoldCoef* fc = which == 2 ? fhs : fcs;
    for (int n = 0; n < D; ++n) {
      const size_t o = ((size_t)b * D + n) * dim + el;
      if (n >= nn) { sacc[o] = 0.f; newe[o] = from_f<T>(0.f); continue; }
      const FoldCoef f = fc[n];
      const float cv = to_f(cin[o]);
      float acc;
      if (f.empty) acc = cv;
      else {
        const float ap = n ? sacc[((size_t)b * D + tm.parent[n]) * dim + el] : pers[(size_t)b * dim + el];
        acc = fmaf(f.a, ap, f.b * cv);
      }
      if (f.done) { newe[o] = from_f<T>(acc / f.s); acc = 0.f; }
      else newe[o] = from_f<T>(0.f);
      sacc[o] = acc;
    }
  }
}

int launch_bsb(const tsv_shape& s, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, int32_t* status, cudaStream_t st) {
  if (s.dtype == TSV_BF16) bsb_kernel<bf16><<<s.B, 128, 0, st>>>(s, c, nd, sc, status);
  else bsb_kernel<float><<<s.B, 128, 0, st>>>(s, c, nd, sc, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
