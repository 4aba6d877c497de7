// accept_and_refresh: greedy acceptance walk, then commit of the accepted path into the
// persistent per-sequence state of every layer.  Two kernels in stream order:
//   aar_walk   (one CTA per sequence)        validates every layer, walks the tree, writes
//                                            accept_len / accept_path / bonus_tok
//   aar_commit (one CTA per sequence, layer) copies window rows, closed entries, open-block
//                                            state; bumps L.  Reads the verdict of aar_walk,
//                                            so all layers of a sequence commit or none does.
#include "kernels.h"

namespace tsv {

__global__ void __launch_bounds__(32) aar_walk_kernel(const tsv_shape s, const AarLayers ls, const int32_t* __restrict__ parent,
                                                      const int32_t* __restrict__ n_nodes, const int32_t* __restrict__ draft,
                                                      const int32_t* __restrict__ target, int32_t* __restrict__ accept_len,
                                                      int32_t* __restrict__ accept_path, int32_t* __restrict__ bonus,
                                                      int32_t* __restrict__ status, const int do_walk) {
  // One warp per sequence.  Lane l checks layer l's length and capacities (the same checks as build_tree_meta), lane n
  // checks node n's parent; the greedy walk runs on ballots: lane c holds node c's parent and draft token.
  const int b = blockIdx.x, D = s.D, lane = threadIdx.x;
  int st = 0;
  int nn = n_nodes[b];
  if (nn < 1 || nn > D) { st |= TSV_ST_NODES; nn = 0; }
  for (int l = lane; l < ls.n; l += 32) {
    int L = ls.l[l].c.L[b];
    if (L < 0 || (int64_t)L + D > s.max_L) { st |= TSV_ST_LENGTH; L = 0; }
    if ((L + D) / s.m_csa > ls.l[l].c.csa_cap[b]) st |= TSV_ST_CSA_CAP;
    if ((L + D) / s.m_hca > ls.l[l].c.hca_cap[b]) st |= TSV_ST_HCA_CAP;
  }
  const int par = lane < nn ? parent[(size_t)b * D + lane] : -1;
  if (lane < nn && (lane == 0 ? par != -1 : (par < 0 || par >= lane))) st |= TSV_ST_PARENT;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) st |= __shfl_xor_sync(0xffffffffu, st, o);
  if (lane == 0 && st) atomicOr(status + b, st);
  if (!do_walk) return;
  st |= status[b];                                     // flags raised earlier in the cycle (every lane reads the same word)
  st = __shfl_sync(0xffffffffu, st, 0);
  int len = 0, bt = -1;
  if (!st) {
    const int dr = lane < nn ? draft[(size_t)b * D + lane] : 0;
    const int tg = lane < nn ? target[(size_t)b * D + lane] : 0;
    int cur = 0;
    if (lane == 0) accept_path[(size_t)b * D] = 0;
    len = 1;
    for (;;) {
      const int want = __shfl_sync(0xffffffffu, tg, cur);
      const uint32_t match = __ballot_sync(0xffffffffu, lane > cur && lane < nn && par == cur && dr == want);
      if (!match) break;
      const int nxt = __ffs(match) - 1;                // the first matching child in node order
      if (lane == 0) accept_path[(size_t)b * D + len] = nxt;
      ++len;
      cur = nxt;
    }
    bt = __shfl_sync(0xffffffffu, tg, cur);
  }
  if (lane == 0) {
    for (int i = len; i < D; ++i) accept_path[(size_t)b * D + i] = -1;
    accept_len[b] = len;
    bonus[b] = bt;
  }
}

__device__ __forceinline__ void copy_row16(void* dst, const void* src, int bytes, int tid, int nthr) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  for (int i = tid; i < bytes / 16; i += nthr) d4[i] = s4[i];
}

__global__ void __launch_bounds__(128) aar_commit_kernel(const tsv_shape s, const AarLayers ls, const int32_t* __restrict__ accept_len,
                                                         const int32_t* __restrict__ accept_path, const int32_t* __restrict__ status) {
  const int b = blockIdx.x, D = s.D;
  const AarLayer& ly = ls.l[blockIdx.y];
  const int al = accept_len[b];
  if (status[b] != 0 || al <= 0) return;
  const int L = ly.c.L[b];
  __syncthreads();                      // every thread holds L before anyone moves it
  const int es = s.dtype == TSV_BF16 ? 2 : 4;
  const size_t rowb = (size_t)s.d * es, ikb = (size_t)s.di * es;
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int i = 0; i < al; ++i) {
    const int n = accept_path[(size_t)b * D + i];
    const int pos = L + i;
    const size_t nidx = (size_t)b * D + n;
    copy_row16((char*)ly.c.win_kv + (size_t)tok_row_of(ly.c, s, b, pos) * rowb, (const char*)ly.node_kv + nidx * rowb, (int)rowb, tid, nt);
    if (ly.sc.csa_done[nidx]) {
      const size_t row = (size_t)csa_rows_of(ly.c, s, b)(pos / s.m_csa);
      copy_row16((char*)ly.c.csa_kv + row * rowb, (const char*)ly.sc.new_csa_kv + nidx * rowb, (int)rowb, tid, nt);
      copy_row16((char*)ly.c.csa_ik + row * ikb, (const char*)ly.sc.new_csa_ik + nidx * ikb, (int)ikb, tid, nt);
    }
    if (ly.sc.hca_done[nidx]) {
      const size_t row = (size_t)hca_rows_of(ly.c, s, b)(pos / s.m_hca);
      copy_row16((char*)ly.c.hca_kv + row * rowb, (const char*)ly.sc.new_hca_kv + nidx * rowb, (int)rowb, tid, nt);
    }
  }
  const size_t last = (size_t)b * D + accept_path[(size_t)b * D + al - 1];
  // Open-block states of the last accepted node.  A block that this node closed leaves an empty state, whose stored numbers
  // nobody reads (emptiness is known from the position count): that copy is skipped.
  const bool csa_open = (L + al) % s.m_csa != 0, hca_open = (L + al) % s.m_hca != 0;
  if (csa_open) {
    copy_row16(ly.c.csa_acc_kv + (size_t)b * s.d, ly.sc.csa_acc_kv + last * s.d, s.d * 4, tid, nt);
    copy_row16(ly.c.csa_acc_ik + (size_t)b * s.di, ly.sc.csa_acc_ik + last * s.di, s.di * 4, tid, nt);
  }
  const bool hdef = hca_deferred(s, L);
  if (hdef) {
    // C128-deferred schedule: branch_state_build built no HCA states for this sequence (no block closes inside its tree);
    // the accepted tokens are folded into the persistent open block here, in path order, with the arithmetic of the state
    // build (scalar part by every thread alike, each thread its own vector elements), so the result has the same bits.
    float mx = ly.c.hca_mx[b], sw = ly.c.hca_s[b];
    float coef_a[TSV_MAX_D], coef_b[TSV_MAX_D];
    for (int i = 0; i < al; ++i) {
      const int n = accept_path[(size_t)b * D + i];
      const float g = ly.node_g_hca[(size_t)b * D + n];
      if ((L + i) % s.m_hca == 0) { mx = g; sw = 1.f; coef_a[i] = 0.f; coef_b[i] = 1.f; }
      else {
        const float mx2 = fmaxf(mx, g);
        coef_a[i] = expf(mx - mx2); coef_b[i] = expf(g - mx2);
        sw = fmaf(sw, coef_a[i], coef_b[i]);
        mx = mx2;
      }
    }
    for (int e = tid; e < s.d; e += nt) {
      float acc = ly.c.hca_acc_kv[(size_t)b * s.d + e];
      for (int i = 0; i < al; ++i) {
        const size_t nidx = (size_t)b * D + accept_path[(size_t)b * D + i];
        const float cv = s.dtype == TSV_BF16 ? to_f(reinterpret_cast<const bf16*>(ly.node_c_hca)[nidx * s.d + e])
                                             : reinterpret_cast<const float*>(ly.node_c_hca)[nidx * s.d + e];
        acc = (L + i) % s.m_hca == 0 ? cv : fmaf(coef_a[i], acc, coef_b[i] * cv);
      }
      ly.c.hca_acc_kv[(size_t)b * s.d + e] = acc;
    }
    __syncthreads();                    // every thread has read the old scalars before thread 0 replaces them
    if (tid == 0) { ly.c.hca_mx[b] = mx; ly.c.hca_s[b] = sw; }
  } else if (hca_open) {
    copy_row16(ly.c.hca_acc_kv + (size_t)b * s.d, ly.sc.hca_acc_kv + last * s.d, s.d * 4, tid, nt);
  }
  if (tid == 0) {
    ly.c.csa_mx[b] = ly.sc.csa_mx[last]; ly.c.csa_s[b] = ly.sc.csa_s[last];
    if (!hdef) { ly.c.hca_mx[b] = ly.sc.hca_mx[last]; ly.c.hca_s[b] = ly.sc.hca_s[last]; }
    ly.c.L[b] = L + al;
  }
}

int launch_aar(const tsv_shape& s, int n_layers, const tsv_cache* const* caches, const tsv_nodes* const* nodes,
               const tsv_scratch* const* scratch, const int32_t* parent, const int32_t* n_nodes,
               const int32_t* draft, const int32_t* target, int32_t* accept_len, int32_t* accept_path,
               int32_t* bonus, int32_t* status, cudaStream_t st) {
  AarLayers ls;
  for (int l0 = 0; l0 < n_layers; l0 += kAarLayersPerLaunch) {
    ls.n = n_layers - l0 < kAarLayersPerLaunch ? n_layers - l0 : kAarLayersPerLaunch;
    for (int i = 0; i < ls.n; ++i) { ls.l[i].c = *caches[l0 + i]; ls.l[i].node_kv = nodes[l0 + i]->kv; ls.l[i].node_c_hca = nodes[l0 + i]->c_hca; ls.l[i].node_g_hca = nodes[l0 + i]->g_hca; ls.l[i].sc = *scratch[l0 + i]; }
    const int last = l0 + ls.n >= n_layers;
    TSV_PREP(aar_walk_kernel);
    aar_walk_kernel<<<s.B, 32, 0, st>>>(s, ls, parent, n_nodes, draft, target, accept_len, accept_path, bonus, status, last);
    count_launch();
  }
  for (int l0 = 0; l0 < n_layers; l0 += kAarLayersPerLaunch) {
    ls.n = n_layers - l0 < kAarLayersPerLaunch ? n_layers - l0 : kAarLayersPerLaunch;
    for (int i = 0; i < ls.n; ++i) { ls.l[i].c = *caches[l0 + i]; ls.l[i].node_kv = nodes[l0 + i]->kv; ls.l[i].node_c_hca = nodes[l0 + i]->c_hca; ls.l[i].node_g_hca = nodes[l0 + i]->g_hca; ls.l[i].sc = *scratch[l0 + i]; }
    TSV_PREP(aar_commit_kernel);
    aar_commit_kernel<<<dim3(s.B, ls.n), 128, 0, st>>>(s, ls, accept_len, accept_path, status);
    count_launch();
  }
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
