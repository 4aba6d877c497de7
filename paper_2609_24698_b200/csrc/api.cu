// C-ABI front end: argument validation on the host, workspace carve-up, kernel dispatch.
// No allocation (host or device), no synchronisation.
#include <math.h>

#include <atomic>

#include "kernels.h"

namespace tsv {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static bool shape_ok(const tsv_shape* s) {
  if (!s) return false;
  if (s->dtype != TSV_FP32 && s->dtype != TSV_BF16) return false;
  if (s->B < 1 || s->D < 1 || s->D > TSV_MAX_D || s->H < 1 || s->H > 256) return false;
  if (s->d < 8 || s->d > 1024 || s->d % 8) return false;
  if (s->di < 8 || s->di > 512 || s->di % 8) return false;
  if (s->HI < 1 || s->HI > 16) return false;
  if (s->m_csa < 1 || s->m_hca < 1 || s->topk < 1) return false;
  if (s->window < s->D) return false;
  if (s->max_L < s->D || s->max_L > (int64_t)1 << 30) return false;
  return true;
}

static tsv_shape resolved(const tsv_shape* s) {
  tsv_shape r = *s;
  if (!(r.sm_scale > 0.f)) r.sm_scale = (float)(1.0 / sqrt((double)r.d));
  return r;
}

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

bool make_tva_plan(const tsv_shape& s, TvaPlan& p) {
  const int64_t pref = s.max_L / s.m_csa;
  p.cand_cap = (int32_t)(pref + s.D);
  p.score_ld = (p.cand_cap + 3) & ~3;
  p.need_scores = p.cand_cap > s.topk;
  p.idx_fused = p.need_scores && p.cand_cap <= kIdxFusedMax && s.HI <= 8 && (size_t)s.HI * s.di * sizeof(float) <= 32768;
  const int64_t ksel = p.cand_cap < s.topk ? p.cand_cap : s.topk;
  p.keys_max = (int32_t)(ksel + s.max_L / s.m_hca + s.D + s.window + s.D);
  const int hgroups = (s.H + 15) / 16;
  const int64_t base = (int64_t)s.B * s.D * hgroups;
  int64_t want = (2 * 148 + base - 1) / base;
  if (want < 1) want = 1;
  int64_t ks = (p.keys_max + want - 1) / want;
  ks = (ks + 31) / 32 * 32;
  if (ks < 64) ks = 64;
  p.ks = (int32_t)ks;
  p.nsplit = (int32_t)((p.keys_max + ks - 1) / ks);
  size_t off = 0;
  p.off_selcnt = off; off = up256(off + (size_t)s.B * s.D * sizeof(int32_t));
  p.off_sel = off;    off = up256(off + (size_t)s.B * s.D * s.topk * sizeof(int32_t));
  p.off_scores = off; if (p.need_scores) off = up256(off + (size_t)s.B * s.D * p.score_ld * sizeof(float));
  p.off_po = off;     if (p.nsplit > 1) off = up256(off + (size_t)s.B * s.D * s.H * p.nsplit * s.d * sizeof(float));
  p.off_pml = off;    if (p.nsplit > 1) off = up256(off + (size_t)s.B * s.D * s.H * p.nsplit * 2 * sizeof(float));
  p.tc = tva_tc_eligible(s);
  p.tc_nt = p.tc_maxk = p.tc_chmax = p.tc_misc_rows = 0;
  p.off_krow = p.off_kmask = p.off_nkeys = p.off_tpo = p.off_tpml = p.off_box = p.off_mode = p.off_misc = p.off_order = p.off_tcnt = off;
  p.off_selmask = off;
  p.mask_ld = (p.cand_cap + 15) & ~15;
  if (p.tc) {
    tva_tc_plan_sizes(s, p);
    const size_t tiles = (size_t)s.B * p.tc_nt;
    p.off_krow = off;  off = up256(off + tiles * p.tc_maxk * sizeof(uint32_t));   // row codes of gathered tiles
    p.off_kmask = off; off = up256(off + tiles * p.tc_maxk);
    p.off_nkeys = off; off = up256(off + tiles * sizeof(int32_t));
    p.off_tpo = off;   if (p.tc_chmax > 1) off = up256(off + 2 * tiles * p.tc_chmax * 128 * s.d * sizeof(float));
    p.off_tpml = off;  if (p.tc_chmax > 1) off = up256(off + 2 * tiles * p.tc_chmax * 128 * 2 * sizeof(float));
    p.off_box = off;   off = up256(off + tiles * (p.tc_maxk / 32) * 2 * sizeof(int32_t));
    p.off_mode = off;  off = up256(off + tiles * sizeof(int32_t));
    p.off_misc = off;  off = up256(off + (size_t)s.B * p.tc_misc_rows * s.d * 2);
    p.off_order = off; off = up256(off + tiles * 4 * sizeof(int32_t));
    p.off_tcnt = off;  off = up256(off + 2 * tiles * sizeof(int32_t));     // finished chunks per 128-row tile (paired kernel)
    p.off_selmask = off; if (p.need_scores) off = up256(off + (size_t)s.B * s.D * p.mask_ld);
  }
  p.total = off;
  return true;
}

static inline bool al16(const void* p) { return ((uintptr_t)p & 15) == 0; }

static int check_cache(const tsv_cache* c, const tsv_shape* s) {
  if (!c) return TSV_ERR_NULL;
  const void* all[] = {c->L, c->csa_kv, c->csa_ik, c->csa_cap, c->hca_kv, c->hca_cap, c->win_kv,
                       c->csa_mx, c->csa_s, c->csa_acc_kv, c->csa_acc_ik, c->hca_mx, c->hca_s, c->hca_acc_kv};
  for (const void* p : all) if (!p) return TSV_ERR_NULL;
  if (c->page_table) {      // paged pool: one table for all physical layers; the page size divides into whole blocks
    if (c->page_tokens < 1 || c->max_pages < 1 || c->page_tokens % s->m_csa || c->page_tokens % s->m_hca || c->tok_rows < 1) return TSV_ERR_SHAPE;
  } else if (!c->csa_row0 || !c->hca_row0) return TSV_ERR_NULL;
  const void* vec[] = {c->csa_kv, c->csa_ik, c->hca_kv, c->win_kv, c->csa_acc_kv, c->csa_acc_ik, c->hca_acc_kv};
  for (const void* p : vec) if (!al16(p)) return TSV_ERR_ALIGN;
  return TSV_OK;
}

static int check_nodes(const tsv_nodes* n, bool attn) {
  if (!n) return TSV_ERR_NULL;
  const void* base[] = {n->kv, n->c_csa, n->ikc, n->g_csa, n->c_hca, n->g_hca, n->parent, n->n_nodes};
  for (const void* p : base) if (!p) return TSV_ERR_NULL;
  if (attn && (!n->q || !n->iq || !n->iw)) return TSV_ERR_NULL;
  const void* vec[] = {n->kv, n->c_csa, n->ikc, n->c_hca, n->q, n->iq};
  for (const void* p : vec) if (p && !al16(p)) return TSV_ERR_ALIGN;
  return TSV_OK;
}

static int check_scratch(const tsv_scratch* s) {
  if (!s) return TSV_ERR_NULL;
  const void* all[] = {s->csa_mx, s->csa_s, s->csa_acc_kv, s->csa_acc_ik, s->hca_mx, s->hca_s, s->hca_acc_kv,
                       s->new_csa_kv, s->new_csa_ik, s->new_hca_kv, s->csa_done, s->hca_done};
  for (const void* p : all) if (!p) return TSV_ERR_NULL;
  const void* vec[] = {s->csa_acc_kv, s->csa_acc_ik, s->hca_acc_kv, s->new_csa_kv, s->new_csa_ik, s->new_hca_kv};
  for (const void* p : vec) if (!al16(p)) return TSV_ERR_ALIGN;
  return TSV_OK;
}

// tree_verify_attn after validation.  All host work that can fail (tensor maps, kernel attributes) comes before the
// first launch, so a negative return means that nothing was enqueued by this call, unless a launch itself fails.
static int tva_stages(const tsv_shape& s, const TvaPlan& p_in, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, void* out,
                      int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st, int stages) {
  int r;
  TvaTcPrep prep;
  TvaPlan p = p_in;
  if (p.tc && !tva_tc_pair_usable(c)) p.tc = 0;       // no row counts for the tensor maps: the CUDA-core path (same workspace)
  if (p.tc && (stages & 6) && (r = prepare_tva_tc(s, p, c, nd, out, ws, prep))) return r;
  if ((stages & 1) && (r = launch_tva_select(s, p, c, nd, sc, topk_idx, ws, status, st))) return r;
  if (!(stages & 6)) return TSV_OK;
  if (p.tc) return launch_tva_tc(s, p, prep, c, nd, sc, out, ws, status, st, (stages & 2) != 0);
  return launch_tva_simt(s, p, c, nd, sc, out, ws, status, st);
}

}  // namespace tsv

using namespace tsv;

extern "C" {

int tsv_version(void) { return 1000; }

uint64_t tsv_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

const char* tsv_error_string(int code) {
  switch (code) {
    case TSV_OK: return "ok";
    case TSV_ERR_NULL: return "a required pointer is NULL";
    case TSV_ERR_ALIGN: return "a vector pointer is not 16-byte aligned";
    case TSV_ERR_SHAPE: return "unsupported shape";
    case TSV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TSV_ERR_CUDA: return "a CUDA runtime call failed";
    case TSV_ERR_LIMIT: return "size beyond a built-in maximum of this entry point";
    default: return "unknown error code";
  }
}

size_t tsv_workspace_bytes(const tsv_shape* shape) {
  if (!shape_ok(shape)) return 0;
  TvaPlan p;
  make_tva_plan(resolved(shape), p);
  return p.total;
}

int branch_state_build(const tsv_shape* shape, const tsv_cache* cache, const tsv_nodes* nodes, const tsv_scratch* scratch,
                       int32_t* status, void* stream) {
  if (!shape || !status) return TSV_ERR_NULL;
  if (!shape_ok(shape)) return TSV_ERR_SHAPE;
  int r;
  if ((r = check_cache(cache, shape)) || (r = check_nodes(nodes, false)) || (r = check_scratch(scratch))) return r;
  return launch_bsb(resolved(shape), *cache, *nodes, *scratch, status, (cudaStream_t)stream);
}

int tree_verify_attn(const tsv_shape* shape, const tsv_cache* cache, const tsv_nodes* nodes, const tsv_scratch* scratch,
                     void* out, int32_t* topk_idx, void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  if (!shape || !status || !out) return TSV_ERR_NULL;
  if (!shape_ok(shape)) return TSV_ERR_SHAPE;
  int r;
  if ((r = check_cache(cache, shape)) || (r = check_nodes(nodes, true)) || (r = check_scratch(scratch))) return r;
  if (!al16(out)) return TSV_ERR_ALIGN;
  const tsv_shape s = resolved(shape);
  TvaPlan p;
  make_tva_plan(s, p);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < p.total) return TSV_ERR_WORKSPACE;
  return tva_stages(s, p, *cache, *nodes, *scratch, out, topk_idx, (char*)workspace, status, (cudaStream_t)stream, 3);
}

// Not part of the public interface (not declared in tsv.h): tree_verify_attn restricted to some of its stages, for
// per-stage timing by the benchmark.  stages: bit 0 = CSA selection, bit 1 = attention (tile plan + attention kernels),
// bit 2 = the attention kernels WITHOUT the tile plan (tensor-core path: the plan a previous call left is used again; the
// finished-chunk counters of two-chunk tiles are not reset, so only timings of such a call mean anything).
// The attention stage alone reuses the selection a previous full call on the same inputs left in `workspace`.
int tsv_bench_tree_verify_attn_stages(const tsv_shape* shape, const tsv_cache* cache, const tsv_nodes* nodes, const tsv_scratch* scratch,
                                      void* out, int32_t* topk_idx, void* workspace, size_t workspace_bytes, int32_t* status, void* stream,
                                      int stages) {
  if (!shape || !status || !out) return TSV_ERR_NULL;
  if (!shape_ok(shape)) return TSV_ERR_SHAPE;
  int r;
  if ((r = check_cache(cache, shape)) || (r = check_nodes(nodes, true)) || (r = check_scratch(scratch))) return r;
  if (!al16(out)) return TSV_ERR_ALIGN;
  const tsv_shape s = resolved(shape);
  TvaPlan p;
  make_tva_plan(s, p);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < p.total) return TSV_ERR_WORKSPACE;
  return tva_stages(s, p, *cache, *nodes, *scratch, out, topk_idx, (char*)workspace, status, (cudaStream_t)stream, stages & 7);
}

int accept_and_refresh(const tsv_shape* shape, int32_t n_layers, const tsv_cache* const* caches, const tsv_nodes* const* nodes,
                       const tsv_scratch* const* scratch, const int32_t* draft_tok, const int32_t* target_tok,
                       int32_t* accept_len, int32_t* accept_path, int32_t* bonus_tok, int32_t* status, void* stream) {
  if (!shape || !caches || !nodes || !scratch || !draft_tok || !target_tok || !accept_len || !accept_path || !bonus_tok || !status)
    return TSV_ERR_NULL;
  if (!shape_ok(shape)) return TSV_ERR_SHAPE;
  if (n_layers < 1 || n_layers > 4096) return TSV_ERR_SHAPE;
  int r;
  for (int l = 0; l < n_layers; ++l)
    if ((r = check_cache(caches[l], shape)) || (r = check_nodes(nodes[l], false)) || (r = check_scratch(scratch[l]))) return r;
  return launch_aar(resolved(shape), n_layers, caches, nodes, scratch, nodes[0]->parent, nodes[0]->n_nodes, draft_tok, target_tok, accept_len,
                    accept_path, bonus_tok, status, (cudaStream_t)stream);
}

}  // extern "C"
