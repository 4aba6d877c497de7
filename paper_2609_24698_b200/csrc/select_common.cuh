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


// Ranks the 256-row attention tiles of all sequences by the number of keys they will stage, most first, so that the
// paired attention kernel starts the long tiles first and the short ones fill the tail (run by ONE CTA of the selection
// launch).  The counts follow from lengths, node counts and done flags alone (for tiles on the contiguous-run path they
// are exact; for gathered tiles an estimate: only the order depends on them), so the ranking is ready before the
// plan kernel runs and each plan CTA can leave its record at its final position.
// nk_est: shared memory for 2048 ints.
__device__ __forceinline__ void rank_tiles_in(int32_t* nk_est, const tsv_shape& s, const TvaPlan& pl, const tsv_cache& c, const tsv_nodes& nd,
                                              const tsv_scratch& sc, char* __restrict__ ws) {
  const int D = s.D, nt = pl.tc_nt, ntile = s.B * nt, npt = 256 / s.H;
  int32_t* pos = reinterpret_cast<int32_t*>(ws + pl.off_pos);
  if (ntile > 2048) { for (int i = threadIdx.x; i < ntile; i += blockDim.x) pos[i] = i; return; }
  auto r32 = [](int x) { return (x + kBoxRows - 1) / kBoxRows * kBoxRows; };
  for (int i = threadIdx.x; i < ntile; i += blockDim.x) {
    const int b = i / nt, tile = i - b * nt;
    const int L = c.L[b], nn = nd.n_nodes[b];
    int est = 0;
    if (L >= 0 && (int64_t)L + D <= s.max_L && nn >= 1 && nn <= D && tile * npt < nn) {
      int ncd = 0, nhd = 0;
      for (int j = 0; j < nn; ++j) { ncd += sc.csa_done[(size_t)b * D + j] != 0; nhd += sc.hca_done[(size_t)b * D + j] != 0; }
      const int n_csa = L / s.m_csa, n_hca = L / s.m_hca, nh_in = n_hca <= kHcaMiscMax ? n_hca : 0, win = min(L, s.window);
      if (n_csa <= 2 * s.topk) est = r32(n_csa) + (n_hca > kHcaMiscMax ? r32(n_hca) : 0) + r32(win) + r32(nh_in + nn + ncd + nhd);
      else est = min(n_csa, npt * s.topk) + n_hca + win + 3 * nn;
    }
    nk_est[i] = est;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < ntile; i += blockDim.x) {
    const int ki = nk_est[i];
    int rank = 0;
    for (int j = 0; j < ntile; ++j) { const int kj = nk_est[j]; rank += (kj > ki) || (kj == ki && j < i); }
    pos[i] = rank;
  }
}
__device__ __forceinline__ void rank_tiles(const tsv_shape& s, const TvaPlan& pl, const tsv_cache& c, const tsv_nodes& nd,
                                           const tsv_scratch& sc, char* __restrict__ ws) {
  __shared__ int32_t nk_est[2048];
  rank_tiles_in(nk_est, s, pl, c, nd, sc, ws);
}

}  // namespace tsv
