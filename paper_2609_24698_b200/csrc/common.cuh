// Shared device helpers of the tree-verify kernels: storage-dtype access, tree metadata
// derived on the device from the raw parent array (depth, ancestor masks, validity).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tsv.h"

namespace tsv {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- storage dtype access
template <typename T> struct Vec;   // 16-byte vector of storage elements
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<bf16> { static constexpr int N = 8; };

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// 16-byte load of Vec<T>::N storage elements, widened to fp32.
__device__ __forceinline__ void ld16(const float* p, float* o) {
  float4 v = *reinterpret_cast<const float4*>(p);
  o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
__device__ __forceinline__ void ld16(const bf16* p, float* o) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void st16(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void st16(bf16* p, const float* v) {
  uint4 o;
  uint32_t* w = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = o;
}

// ---------------------------------------------------------------- cache rows
// Row of entry e of one sequence in one physical layer of the cache: a slab starting at row0 (flat caches), or through
// the sequence's page-table row with `per_page` entries of this layer per page (paged pool).
struct RowAddr {
  const int32_t* pt;
  int32_t per_page;
  int64_t row0;
  __device__ __forceinline__ int64_t operator()(int e) const {
    return pt ? (int64_t)__ldg(pt + e / per_page) * per_page + e % per_page : row0 + e;
  }
  // the same row relative to row0 (row0 is 0 in a paged pool): for code that keeps a base pointer of the slab
  __device__ __forceinline__ int64_t rel(int e) const {
    return pt ? (int64_t)__ldg(pt + e / per_page) * per_page + e % per_page : (int64_t)e;
  }
};
__device__ __forceinline__ RowAddr csa_rows_of(const tsv_cache& c, const tsv_shape& s, int b) {
  RowAddr r;
  r.pt = c.page_table ? c.page_table + (size_t)b * c.max_pages : nullptr;
  r.per_page = c.page_table ? c.page_tokens / s.m_csa : 1;
  r.row0 = c.page_table ? 0 : c.csa_row0[b];
  return r;
}
__device__ __forceinline__ RowAddr hca_rows_of(const tsv_cache& c, const tsv_shape& s, int b) {
  RowAddr r;
  r.pt = c.page_table ? c.page_table + (size_t)b * c.max_pages : nullptr;
  r.per_page = c.page_table ? c.page_tokens / s.m_hca : 1;
  r.row0 = c.page_table ? 0 : c.hca_row0[b];
  return r;
}

// Row of the token-level KV of position pos: slot pos % window of the sequence's ring, or through the page table.
__device__ __forceinline__ int64_t tok_row_of(const tsv_cache& c, const tsv_shape& s, int b, int pos) {
  if (c.page_table) return (int64_t)__ldg(c.page_table + (size_t)b * c.max_pages + pos / c.page_tokens) * c.page_tokens + pos % c.page_tokens;
  return (int64_t)b * s.window + pos % s.window;
}

// ---------------------------------------------------------------- tree metadata
// Built by ONE thread of a CTA into shared memory, then read by all after a barrier.
struct TreeMeta {
  int32_t L;            // committed length of this sequence in this layer
  int32_t nn;           // valid nodes
  int32_t status;       // TSV_ST_* found here (0 = usable)
  int32_t n_csa, n_hca; // committed entries
  int32_t depth[TSV_MAX_D];
  int32_t parent[TSV_MAX_D];
  uint32_t anc[TSV_MAX_D];   // bit j set iff j == n or j is an ancestor of n
};

// Validates and derives the per-sequence tree facts.  `caps` may be null (capacity unchecked).
__device__ inline void build_tree_meta(TreeMeta& tm, const tsv_shape& s, int32_t L, const int32_t* parent_b,
                                       int32_t nn, const int32_t* csa_cap_b, const int32_t* hca_cap_b) {
  int st = 0;
  if (nn < 1 || nn > s.D) { st |= TSV_ST_NODES; nn = 0; }
  if (L < 0 || (int64_t)L + s.D > s.max_L) { st |= TSV_ST_LENGTH; L = 0; }
  for (int n = 0; n < TSV_MAX_D; ++n) { tm.depth[n] = 0; tm.parent[n] = -1; tm.anc[n] = 0; }
  for (int n = 0; n < nn; ++n) {
    int p = parent_b[n];
    if (n == 0) {
      if (p != -1) st |= TSV_ST_PARENT;
      tm.anc[0] = 1u;
    } else if (p < 0 || p >= n) {
      st |= TSV_ST_PARENT;
    } else {
      tm.parent[n] = p;
      tm.depth[n] = tm.depth[p] + 1;
      tm.anc[n] = tm.anc[p] | (1u << n);
    }
  }
  if (csa_cap_b && (L + s.D) / s.m_csa > *csa_cap_b) st |= TSV_ST_CSA_CAP;
  if (hca_cap_b && (L + s.D) / s.m_hca > *hca_cap_b) st |= TSV_ST_HCA_CAP;
  tm.L = L; tm.nn = nn; tm.status = st;
  tm.n_csa = L / s.m_csa; tm.n_hca = L / s.m_hca;
}

// Cooperative front end of build_tree_meta: the first threads of the CTA fetch the parent array and the per-sequence
// scalars in parallel (one memory latency instead of a chain of dependent loads), then warp 0 derives the tree facts.
// Must be called by all threads of the CTA (contains two barriers); needs blockDim.x >= 64.
struct TreeStage { int32_t parent[TSV_MAX_D]; int32_t scal[4]; };
__device__ __forceinline__ void coop_tree_meta(TreeMeta& tm, TreeStage& st, const tsv_shape& s, const int32_t* L_b, const int32_t* parent_b,
                                               const int32_t* nn_b, const int32_t* csa_cap_b, const int32_t* hca_cap_b) {
  const int t = threadIdx.x;
  if (t < s.D) st.parent[t] = parent_b[t];
  if (t == 32) st.scal[0] = *L_b;
  if (t == 33) st.scal[1] = *nn_b;
  if (t == 34 && csa_cap_b) st.scal[2] = *csa_cap_b;
  if (t == 35 && hca_cap_b) st.scal[3] = *hca_cap_b;
  __syncthreads();
  if (t < 32) {
    // Same facts as build_tree_meta, lane n deriving node n: ancestors by walking up the staged parent array (a valid
    // array has parent < node, so the walk ends within D steps).  With any invalid entry the sequence is flagged and
    // every kernel skips it, so the facts of the other nodes need not match the serial routine then.
    int L = st.scal[0], nn = st.scal[1], stt = 0;
    if (nn < 1 || nn > s.D) { stt |= TSV_ST_NODES; nn = 0; }
    if (L < 0 || (int64_t)L + s.D > s.max_L) { stt |= TSV_ST_LENGTH; L = 0; }
    const int n = t;
    const int p = (n < nn) ? st.parent[n] : -1;
    const bool bad = (n < nn) && (n == 0 ? p != -1 : (p < 0 || p >= n));
    if (__any_sync(0xffffffffu, bad)) stt |= TSV_ST_PARENT;
    uint32_t anc = 0;
    int depth = 0;
    if (n < nn && !bad) {
      anc = 1u << n;
      int cur = p;
#pragma unroll 1
      for (int it = 0; it < TSV_MAX_D && cur >= 0 && cur < n; ++it) { anc |= 1u << cur; ++depth; cur = st.parent[cur]; }
    }
    tm.depth[n] = depth; tm.parent[n] = (n < nn && !bad && n > 0) ? p : -1; tm.anc[n] = anc;
    if (t == 0) {
      if (csa_cap_b && (L + s.D) / s.m_csa > st.scal[2]) stt |= TSV_ST_CSA_CAP;
      if (hca_cap_b && (L + s.D) / s.m_hca > st.scal[3]) stt |= TSV_ST_HCA_CAP;
      tm.L = L; tm.nn = nn; tm.status = stt;
      tm.n_csa = L / s.m_csa; tm.n_hca = L / s.m_hca;
    }
  }
  __syncthreads();
}

// Does the node at depth `depth` of a sequence of committed length L close a block of m tokens?  (What the state build
// writes into its done flags for a valid node: a function of the position alone, so kernels that run under the state
// build's tail work it out instead of reading the flag.)
__device__ __forceinline__ bool node_closes(int L, int depth, int m) { return ((L + depth + 1) % m) == 0; }

// C128-deferred schedule: no node of this sequence can close an HCA block (a node at depth delta closes one iff
// (L + delta + 1) % m_hca == 0, and delta <= D - 1), so its HCA branch states are not built and the accepted path is
// folded into the persistent state at commit time.
__device__ __forceinline__ bool hca_deferred(const tsv_shape& s, int L) {
  return (s.flags & TSV_FLAG_HCA_DEFERRED) && L >= 0 && (L % s.m_hca) + s.D < s.m_hca;
}

__device__ __forceinline__ float softmax_scale(const tsv_shape& s) {
  return s.sm_scale > 0.f ? s.sm_scale : rsqrtf((float)s.d);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exclusive block scan of one int per thread (256 threads); returns the thread's offset and the total.
__device__ __forceinline__ int block_excl_scan_256(int v, int* wsum /* shared[9] */, int& total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) wsum[w] = x;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int i = 0; i < 8; ++i) { const int t = wsum[i]; wsum[i] = run; run += t; }
    wsum[8] = run;
  }
  __syncthreads();
  total = wsum[8];
  return wsum[w] + x - v;
}

// The same for CTAs of up to 1024 threads (a multiple of 32): wsum is shared[33].
__device__ __forceinline__ int block_excl_scan(int v, int* wsum, int& total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) wsum[w] = x;
  __syncthreads();
  if (w == 0) {                                        // the warps' totals: an exclusive scan by warp 0
    const int tw = lane < nw ? wsum[lane] : 0;
    int y = tw;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int z = __shfl_up_sync(0xffffffffu, y, o);
      if (lane >= o) y += z;
    }
    wsum[lane] = y - tw;
    if (lane == 31) wsum[32] = y;
  }
  __syncthreads();
  total = wsum[32];
  return wsum[w] + x - v;
}

}  // namespace tsv
