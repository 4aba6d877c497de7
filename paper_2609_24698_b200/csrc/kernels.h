// Internal interface between the C-ABI front end (api.cu) and the kernel files.
#pragma once
#include "common.cuh"

namespace tsv {

void count_launch(int n = 1);

// Every kernel of the library asks for the same (maximal) shared-memory carve-out: consecutive kernels with different
// carve-outs make the SMs drain and reconfigure between launches, which costs far more than these kernels run.
#define TSV_PREP(kernel)                                                                                          \
  do {                                                                                                            \
    static bool done_ = false;                                                                                    \
    if (!done_) {                                                                                                 \
      cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared); \
      done_ = true;                                                                                               \
    }                                                                                                             \
  } while (0)   // bumps the reporting counter behind tsv_kernel_launches()

// Per-layer pointers accept_and_refresh needs, packed so that a group of layers fits in
// kernel-parameter space.
struct AarLayer {
  tsv_cache c;
  const void* node_kv;
  const void* node_c_hca;      // HCA compression vectors and gate logits of the nodes (C128-deferred schedule)
  const float* node_g_hca;
  tsv_scratch sc;
};
constexpr int kAarLayersPerLaunch = 12;
struct AarLayers {
  AarLayer l[kAarLayersPerLaunch];
  int32_t n;
};

// Workspace carve-up of tree_verify_attn (byte offsets from a 256-byte aligned base).
struct TvaPlan {
  int32_t cand_cap;      // max CSA candidates per node (committed + in-tree)
  int32_t score_ld;      // floats per node row of the score array: cand_cap rounded up to 4 (16-byte rows)
  int32_t need_scores;   // cand_cap > topk: some node may have to rank its candidates
  int32_t idx_fused;     // ranked nodes score their committed entries inside topk_kernel (short candidate lists: the
                         // separate scoring kernel, which exits at once for every sequence that needs no ranking, is not launched)
  int32_t keys_max;      // max keys one node can attend to
  int32_t ks;            // keys per split (CUDA-core path)
  int32_t nsplit;        // max splits per node
  size_t off_selcnt, off_sel, off_scores, off_po, off_pml, total;
  // tensor-core path (bf16, d = 512): row tiles per sequence, key-list capacity per tile, max chunks per tile
  int32_t tc, tc_nt, tc_maxk, tc_chmax;
  int32_t tc_misc_rows;              // rows of the per-sequence packed buffer
  size_t off_krow, off_kmask, off_nkeys, off_tpo, off_tpml, off_box, off_mode, off_misc, off_order, off_tcnt;
  // selection as a byte per candidate (1 = selected), one row of mask_ld bytes per node, written for the nodes that rank:
  // the tile plan combines the rows of a tile's nodes into its per-key node masks
  size_t off_selmask;
  int32_t mask_ld;
};
bool make_tva_plan(const tsv_shape& s, TvaPlan& p);

int launch_bsb(const tsv_shape& s, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, int32_t* status, cudaStream_t st);
int launch_aar(const tsv_shape& s, int n_layers, const tsv_cache* const* caches, const tsv_nodes* const* nodes,
               const tsv_scratch* const* scratch, const int32_t* parent, const int32_t* n_nodes,
               const int32_t* draft, const int32_t* target, int32_t* accept_len, int32_t* accept_path,
               int32_t* bonus, int32_t* status, cudaStream_t st);
// indexer scores of all nodes of a sequence as one small GEMM per tile of entries (bf16, 128-wide indexer rows, D * HI <= 32)
bool idx_score_tc_applies(const tsv_shape& s);
void launch_idx_score_tc(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc, char* ws,
                         int32_t* status, cudaStream_t st);
int launch_tva_select(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                      int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st);
// per-node top-k of short candidate lists with the benchmark's indexer shape (scores, ranks and selects in one CTA)
bool topk_fused_applies(const tsv_shape& s, const TvaPlan& p);
int launch_topk_fused(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                      int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st);
// per-node top-k of long candidate lists by a thread-block cluster per node
bool topk_long_applies(const tsv_shape& s, const TvaPlan& p);
int launch_topk_long(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                     int32_t* topk_idx, char* ws, int32_t* status, cudaStream_t st);
int launch_tva_simt(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                    void* out, char* ws, int32_t* status, cudaStream_t st);

constexpr int kIdxFusedMax = 2272;   // candidate capacity up to which topk_kernel computes the indexer scores itself
constexpr int kBoxRows = 32;       // rows of one TMA box; contiguous key runs are padded to a multiple of it
constexpr int kHcaMiscMax = 32;    // up to this many HCA entries travel in the packed per-sequence buffer
bool tva_tc_eligible(const tsv_shape& s);
// the tensor-core path needs the caller's row count of the CSA arrays (tensor maps) and the driver's map encoder; without
// them a shape it would take runs on the CUDA-core path
bool tva_tc_pair_usable(const tsv_cache& c);
// Host-side preparation of the tensor-core attention path: everything that can fail on the host (tensor maps, kernel
// attributes) is done here, before any kernel of the call is enqueued.
struct TvaTcPrep {
  alignas(64) unsigned char maps[19 * 128];   // the paired kernel's tensor maps (a CUtensorMap is 128 bytes)
};
int prepare_tva_tc_pair(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, void* out, char* ws, TvaTcPrep& prep);
// general: gathered tiles or tiles of more than two chunks may occur (else the instantiation without that code runs)
int launch_tva_tc_pair(const tsv_shape& s, const TvaPlan& p, const TvaTcPrep& prep, bool general, void* out, char* ws, int32_t* status, cudaStream_t st);
void tva_tc_plan_sizes(const tsv_shape& s, TvaPlan& p);
int prepare_tva_tc(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, void* out, char* ws, TvaTcPrep& prep);
// with_plan = false: the tile plan a previous call left in the workspace is used again (timing aid of the benchmark)
int launch_tva_tc(const tsv_shape& s, const TvaPlan& p, const TvaTcPrep& prep, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                  void* out, char* ws, int32_t* status, cudaStream_t st, bool with_plan = true);

}  // namespace tsv
