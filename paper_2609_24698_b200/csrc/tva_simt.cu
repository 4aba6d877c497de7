// tree_verify_attn on CUDA cores (fp32 FMA): the path for fp32 storage and for every shape the
// tensor-core kernels do not cover; also the on-device cross-check of those kernels.
//
// One CTA = (sequence, node, group of 16 heads, split of the node's key list).  The key list
// of a node is the concatenation of five segments, resolved to row pointers on the fly:
//   selected CSA entries | committed HCA entries | in-tree HCA entries of the path |
//   committed window positions | ancestors-or-self.
// Keys are staged 32 at a time in shared memory in the storage dtype; S = QK^T and O += PK
// run as register-tiled fp32 loops with an online softmax per head.  A node whose list fits
// one split writes its output directly; otherwise partial (max, sum, O) go to the workspace
// and attn_combine_kernel merges them in split order (deterministic).
#include "kernels.h"

namespace tsv {

constexpr int kHeadsPerCta = 16;
constexpr int kKeyTile = 32;

struct NodeKeys {
  int32_t n_sel, n_hca, n_newh, win_lo, n_win, n_tree, total;
  int32_t n_newc;
  int32_t newc[TSV_MAX_D], newc_blk[TSV_MAX_D], newh[TSV_MAX_D], tree[TSV_MAX_D];
};

__device__ inline void node_keys(NodeKeys& nk, const TreeMeta& tm, const tsv_shape& s, int n, int n_sel,
                                 const uint8_t* csa_done_b, const uint8_t* hca_done_b) {
  nk.n_newc = nk.n_newh = nk.n_tree = 0;
  for (int j = 0; j <= n; ++j) {
    if (!((tm.anc[n] >> j) & 1u)) continue;
    nk.tree[nk.n_tree++] = j;
    if (j == n) break;
    if (csa_done_b[j]) { nk.newc[nk.n_newc] = j; nk.newc_blk[nk.n_newc++] = (tm.L + tm.depth[j]) / s.m_csa; }
    if (hca_done_b[j]) nk.newh[nk.n_newh++] = j;
  }
  const int p = tm.L + tm.depth[n];
  nk.win_lo = max(0, p - s.window + 1);
  nk.n_win = max(0, tm.L - nk.win_lo);
  nk.n_sel = n_sel;
  nk.n_hca = tm.n_hca;
  nk.total = nk.n_sel + nk.n_hca + nk.n_newh + nk.n_win + nk.n_tree;
}

template <typename T>
__device__ __forceinline__ const T* key_row(int j, const NodeKeys& nk, const TreeMeta& tm, const tsv_shape& s, int b,
                                            const int32_t* sel, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc) {
  const size_t d = s.d;
  if (j < nk.n_sel) {
    const int idx = sel[j];
    if (idx < tm.n_csa) return reinterpret_cast<const T*>(c.csa_kv) + (size_t)csa_rows_of(c, s, b)(idx) * d;
    int a = nk.newc[0];
    for (int i = 0; i < nk.n_newc; ++i) if (nk.newc_blk[i] == idx) a = nk.newc[i];
    return reinterpret_cast<const T*>(sc.new_csa_kv) + ((size_t)b * s.D + a) * d;
  }
  j -= nk.n_sel;
  if (j < nk.n_hca) return reinterpret_cast<const T*>(c.hca_kv) + (size_t)hca_rows_of(c, s, b)(j) * d;
  j -= nk.n_hca;
  if (j < nk.n_newh) return reinterpret_cast<const T*>(sc.new_hca_kv) + ((size_t)b * s.D + nk.newh[j]) * d;
  j -= nk.n_newh;
  if (j < nk.n_win) return reinterpret_cast<const T*>(c.win_kv) + (size_t)tok_row_of(c, s, b, nk.win_lo + j) * d;
  j -= nk.n_win;
  return reinterpret_cast<const T*>(nd.kv) + ((size_t)b * s.D + nk.tree[j]) * d;
}

// NCH = 16-byte chunks of a row each thread of a 16-thread head group owns in the PV phase.
template <typename T, int NCH>
__global__ void __launch_bounds__(256) attn_simt_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                        const tsv_scratch sc, void* __restrict__ out_, char* __restrict__ ws) {
  constexpr int V = Vec<T>::N;
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ TreeMeta tm;
  __shared__ NodeKeys nk;
  const int d = s.d, H = s.H, D = s.D;
  const int hgroups = (H + kHeadsPerCta - 1) / kHeadsPerCta;
  const int split = blockIdx.x, n = blockIdx.y / hgroups, hg = blockIdx.y % hgroups, b = blockIdx.z;
  const int tid = threadIdx.x;
  const int rowstride = d + V;                               // padded row, in elements (16 bytes of pad)
  T* Qs = reinterpret_cast<T*>(smem);                        // [16][d]
  T* Ks = Qs + (size_t)kHeadsPerCta * d;                     // [32][rowstride]
  float* Ps = reinterpret_cast<float*>(Ks + (size_t)kKeyTile * rowstride);   // [16][32]
  T* out = reinterpret_cast<T*>(out_);

  const int32_t* sel = reinterpret_cast<const int32_t*>(ws + pl.off_sel) + ((size_t)b * D + n) * s.topk;
  if (tid == 0) {
    build_tree_meta(tm, s, c.L[b], nd.parent + (size_t)b * D, nd.n_nodes[b], c.csa_cap + b, c.hca_cap + b);
    if (!tm.status && n < tm.nn)
      node_keys(nk, tm, s, n, reinterpret_cast<const int32_t*>(ws + pl.off_selcnt)[(size_t)b * D + n],
                sc.csa_done + (size_t)b * D, sc.hca_done + (size_t)b * D);
  }
  __syncthreads();
  const int h0 = hg * kHeadsPerCta;
  const int nh = min(kHeadsPerCta, H - h0);
  if (tm.status || n >= tm.nn) {                             // flagged sequence / padding node: zeros
    if (split == 0) {
      float z[V];
#pragma unroll
      for (int t = 0; t < V; ++t) z[t] = 0.f;
      for (int i = tid; i < nh * d / V; i += blockDim.x) st16(out + (((size_t)b * D + n) * H + h0) * d + (size_t)i * V, z);
    }
    return;
  }
  const int N = nk.total;
  const int nsplit = (N + pl.ks - 1) / pl.ks;
  if (split >= nsplit) return;
  const int k_begin = split * pl.ks, k_end = min(N, k_begin + pl.ks);

  // stage Q of this head group
  for (int i = tid; i < nh * d / V; i += blockDim.x) {
    const uint4 v = *reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(nd.q) + (((size_t)b * D + n) * H + h0) * d + (size_t)i * V);
    *reinterpret_cast<uint4*>(Qs + (size_t)i * V) = v;
  }
  const int h = tid >> 4, sub = tid & 15;                    // head within the group, lane within the head's 16 threads
  const bool hv = h < nh;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int t = 0; t < V; ++t) acc[i][t] = 0.f;
  const int chunks = d / V;
  const float scale = s.sm_scale;

  for (int k0 = k_begin; k0 < k_end; k0 += kKeyTile) {
    __syncthreads();                                         // previous tile fully consumed
    {   // stage 32 key rows: 8 threads per row
      const int r = tid >> 3, c8 = tid & 7;
      const int j = k0 + r;
      if (j < k_end) {
        const T* src = key_row<T>(j, nk, tm, s, b, sel, c, nd, sc);
        for (int ch = c8; ch < chunks; ch += 8)
          *reinterpret_cast<uint4*>(Ks + (size_t)r * rowstride + ch * V) = *reinterpret_cast<const uint4*>(src + ch * V);
      } else {
        for (int ch = c8; ch < chunks; ch += 8) *reinterpret_cast<uint4*>(Ks + (size_t)r * rowstride + ch * V) = make_uint4(0, 0, 0, 0);
      }
    }
    __syncthreads();
    // S = scale * q . k for keys sub and sub + 16
    float s0 = 0.f, s1 = 0.f;
    if (hv) {
      const T* qrow = Qs + (size_t)h * d;
      const T* ka = Ks + (size_t)sub * rowstride;
      const T* kb = Ks + (size_t)(sub + 16) * rowstride;
      for (int ch = 0; ch < chunks; ++ch) {
        float qv[V], av[V], bv[V];
        ld16(qrow + ch * V, qv); ld16(ka + ch * V, av); ld16(kb + ch * V, bv);
#pragma unroll
        for (int t = 0; t < V; ++t) { s0 = fmaf(qv[t], av[t], s0); s1 = fmaf(qv[t], bv[t], s1); }
      }
    }
    s0 = (k0 + sub < k_end) ? s0 * scale : -INFINITY;
    s1 = (k0 + sub + 16 < k_end) ? s1 * scale : -INFINITY;
    float tmax = fmaxf(s0, s1);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    const float m_new = fmaxf(m_run, tmax);                  // finite: every tile holds >= 1 valid key
    const float p0 = expf(s0 - m_new), p1 = expf(s1 - m_new);
    float tsum = p0 + p1;
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, o);
    const float alpha = expf(m_run - m_new);                 // 0 on the first tile (m_run = -inf)
    l_run = fmaf(l_run, alpha, tsum);
    m_run = m_new;
    Ps[h * kKeyTile + sub] = p0;
    Ps[h * kKeyTile + sub + 16] = p1;
    __syncthreads();
    // O = alpha * O + P K ; thread owns chunks sub, sub + 16, ...
    if (hv) {
#pragma unroll
      for (int i = 0; i < NCH; ++i)
#pragma unroll
        for (int t = 0; t < V; ++t) acc[i][t] *= alpha;
      const int jmax = min(kKeyTile, k_end - k0);
      for (int j = 0; j < jmax; ++j) {
        const float p = Ps[h * kKeyTile + j];
        const T* krow = Ks + (size_t)j * rowstride;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          const int ch = sub + 16 * i;
          if (ch < chunks) {
            float kv[V];
            ld16(krow + ch * V, kv);
#pragma unroll
            for (int t = 0; t < V; ++t) acc[i][t] = fmaf(p, kv[t], acc[i][t]);
          }
        }
      }
    }
  }
  if (!hv) return;
  const size_t rowi = ((size_t)b * D + n) * H + h0 + h;
  if (nsplit == 1) {
    const float inv = 1.f / l_run;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int ch = sub + 16 * i;
      if (ch < chunks) {
        float o[V];
#pragma unroll
        for (int t = 0; t < V; ++t) o[t] = acc[i][t] * inv;
        st16(out + rowi * d + (size_t)ch * V, o);
      }
    }
  } else {
    float* po = reinterpret_cast<float*>(ws + pl.off_po) + (rowi * pl.nsplit + split) * d;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int ch = sub + 16 * i;
      if (ch < chunks)
#pragma unroll
        for (int t = 0; t < V; ++t) po[ch * V + t] = acc[i][t];
    }
    if (sub == 0) {
      float* pml = reinterpret_cast<float*>(ws + pl.off_pml) + (rowi * pl.nsplit + split) * 2;
      pml[0] = m_run; pml[1] = l_run;
    }
  }
}

// Merge of the split partials of one (sequence, node): one CTA, thread-per-element loops.
template <typename T>
__global__ void __launch_bounds__(256) attn_combine_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                           const tsv_scratch sc, void* __restrict__ out_, const char* __restrict__ ws) {
  __shared__ TreeMeta tm;
  __shared__ NodeKeys nk;
  const int n = blockIdx.x, b = blockIdx.y, D = s.D, H = s.H, d = s.d;
  if (threadIdx.x == 0) {
    build_tree_meta(tm, s, c.L[b], nd.parent + (size_t)b * D, nd.n_nodes[b], c.csa_cap + b, c.hca_cap + b);
    if (!tm.status && n < tm.nn)
      node_keys(nk, tm, s, n, reinterpret_cast<const int32_t*>(ws + pl.off_selcnt)[(size_t)b * D + n],
                sc.csa_done + (size_t)b * D, sc.hca_done + (size_t)b * D);
  }
  __syncthreads();
  if (tm.status || n >= tm.nn) return;
  const int nsplit = (nk.total + pl.ks - 1) / pl.ks;
  if (nsplit <= 1) return;
  T* out = reinterpret_cast<T*>(out_);
  const float* po = reinterpret_cast<const float*>(ws + pl.off_po);
  const float* pml = reinterpret_cast<const float*>(ws + pl.off_pml);
  for (int i = threadIdx.x; i < H * d; i += blockDim.x) {
    const size_t rowi = ((size_t)b * D + n) * H + i / d;
    const int e = i % d;
    float m = -INFINITY;
    for (int sp = 0; sp < nsplit; ++sp) m = fmaxf(m, pml[(rowi * pl.nsplit + sp) * 2]);
    float l = 0.f, o = 0.f;
    for (int sp = 0; sp < nsplit; ++sp) {
      const float w = expf(pml[(rowi * pl.nsplit + sp) * 2] - m);
      l = fmaf(pml[(rowi * pl.nsplit + sp) * 2 + 1], w, l);
      o = fmaf(po[(rowi * pl.nsplit + sp) * d + e], w, o);
    }
    out[rowi * d + e] = from_f<T>(o / l);
  }
}

template <typename T, int NCH>
static int launch_one(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                      void* out, char* ws, cudaStream_t st) {
  constexpr int V = Vec<T>::N;
  const int hgroups = (s.H + kHeadsPerCta - 1) / kHeadsPerCta;
  const size_t sm = ((size_t)kHeadsPerCta * s.d + (size_t)kKeyTile * (s.d + V)) * sizeof(T) + kHeadsPerCta * kKeyTile * sizeof(float);
  if (cudaFuncSetAttribute(attn_simt_kernel<T, NCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess) return TSV_ERR_CUDA;
  dim3 grid(p.nsplit, s.D * hgroups, s.B);
  TSV_PREP((attn_simt_kernel<T, NCH>));
  TSV_PREP(attn_combine_kernel<T>);
  attn_simt_kernel<T, NCH><<<grid, 256, sm, st>>>(s, p, c, nd, sc, out, ws);
  count_launch();
  if (p.nsplit > 1) { attn_combine_kernel<T><<<dim3(s.D, s.B), 256, 0, st>>>(s, p, c, nd, sc, out, ws); count_launch(); }
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

template <typename T>
static int launch_t(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                    void* out, char* ws, cudaStream_t st) {
  const int need = (s.d / Vec<T>::N + 15) / 16;
  if (need <= 1) return launch_one<T, 1>(s, p, c, nd, sc, out, ws, st);
  if (need <= 2) return launch_one<T, 2>(s, p, c, nd, sc, out, ws, st);
  if (need <= 4) return launch_one<T, 4>(s, p, c, nd, sc, out, ws, st);
  if (need <= 8) return launch_one<T, 8>(s, p, c, nd, sc, out, ws, st);
  return launch_one<T, 16>(s, p, c, nd, sc, out, ws, st);
}

int launch_tva_simt(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                    void* out, char* ws, int32_t* status, cudaStream_t st) {
  (void)status;
  return s.dtype == TSV_BF16 ? launch_t<bf16>(s, p, c, nd, sc, out, ws, st) : launch_t<float>(s, p, c, nd, sc, out, ws, st);
}

}  // namespace tsv
