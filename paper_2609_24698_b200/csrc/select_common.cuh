// Pieces shared by the selection kernels: the in-tree entries on a node's path, the order-preserving integer image of
// a score, and the ranking of the attention tiles.
#pragma once
#include "kernels.h"

namespace tsv {

// Strict ancestors of n that closed a CSA / HCA block, root first (ascending block index).
struct PathEntries {
  int32_t n_newc, n_newh;
  int32_t newc[TSV_MAX_D], newc_blk[TSV_MAX_D];
  int32_t newh[TSV_MAX_D];
};

__device__ inline void path_entries(PathEntries& pe, const TreeMeta& tm, const tsv_shape& s, int n,
                                    const uint8_t* csa_done_b, const uint8_t* hca_done_b) {
  pe.n_newc = pe.n_newh = 0;
  const uint32_t a = tm.anc[n] & ~(1u << n);
#pragma unroll 1                                        // (compact code: the kernels run with cold instruction caches)
  for (int j = 0; j < n; ++j) {
    if (!((a >> j) & 1u)) continue;
    if (csa_done_b[j]) { pe.newc[pe.n_newc] = j; pe.newc_blk[pe.n_newc++] = (tm.L + tm.depth[j]) / s.m_csa; }
    if (hca_done_b[j]) pe.newh[pe.n_newh++] = j;
  }
}

__device__ __forceinline__ uint32_t order_key(float f) {       // larger float -> larger key
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}


}  // namespace tsv
