/*
 * tsv.h -- C ABI of the tree-speculation verify path over online-compressed attention
 *          (CSA "C4" sparse cache + HCA "C128" dense cache + sliding window), B200 / sm_100a.
 *
 * Three calls make one verify cycle of one attention layer stack:
 *
 *     for every layer:  branch_state_build(...)  ->  tree_verify_attn(...)
 *     then once:        accept_and_refresh(all layers)
 *
 * Conventions
 *   - Every `void*` / typed pointer inside the structs is a DEVICE pointer unless the
 *     comment says HOST.  The structs themselves and `tsv_shape` live in HOST memory and
 *     are read during the call only.
 *   - The caller owns every buffer.  The library allocates nothing and never synchronises: all
 *     work is enqueued on `stream` and the call returns.  Between calls it keeps nothing of the
 *     caller's data; what it does keep per process is set-up it does once (kernel attributes,
 *     the number of CTA pairs a device holds, the driver entry point for tensor maps), the
 *     launch counter behind tsv_kernel_launches(), and for tree_verify_attn_static the
 *     address of its built-in array.
 *   - Stream order: the calls of a layer run in the order given above on one stream.  Some kernels of
 *     tree_verify_attn are launched as PROGRAMMATIC DEPENDENTS of the kernel before them on the stream: the part
 *     of them that reads only the call's inputs (tsv_nodes, the committed tsv_cache) may run before that kernel
 *     has finished, and that part already writes the call's workspace, topk_idx and status; they wait for
 *     it before they read anything the library's own kernels write.  For the caller this matters in one
 *     case only: a kernel of the caller's that is enqueued directly before tree_verify_attn and itself
 *     signals its dependents early (griddepcontrol.launch_dependents /
 *     cudaTriggerProgrammaticLaunchCompletion) must, before it signals, have written whatever it writes
 *     of that call's inputs and have read whatever it reads of that call's workspace, topk_idx and
 *     status.  Kernels that do not use that feature are complete before any of the library's kernels
 *     starts, as always.
 *   - "storage dtype" = tsv_shape.dtype (fp32 or bf16): all vectors and cache rows.  All
 *     partial-block accumulators, gates and weights are fp32.
 *   - Row-major, innermost dimension contiguous, no padding.  Vector pointers must be
 *     16-byte aligned and d, di multiples of 8.
 *   - Cache buffers (csa_kv, csa_ik, hca_kv, win_kv) must hold finite numbers in EVERY allocated
 *     row, also in rows not committed yet (allocate them zero-filled): the tensor-core kernels
 *     fetch whole 32-row boxes and multiply the unused rows by an exact zero weight.
 *   - Node n of sequence b sits at depth delta_n (root = node 0 = depth 0) and at position
 *     p_n = L[b] + delta_n.  n_csa = L / m_csa and n_hca = L / m_hca committed entries.
 *   - Return value: 0 or a negative TSV_ERR_* for problems the host can see BEFORE any
 *     launch (nothing is enqueued then: argument checks, tensor-map encoding and kernel
 *     attributes all precede the first launch).  Only a failing kernel launch itself
 *     (TSV_ERR_CUDA out of cudaLaunchKernel) can leave earlier kernels of the same call
 *     enqueued; skip accept_and_refresh for that cycle then.  Problems only the device can see (bad parent
 *     array, node count, capacity, length) are reported per sequence in `status[b]`
 *     (bit-or of TSV_ST_*): that sequence's outputs are zero-filled and
 *     accept_and_refresh commits nothing for it (L unchanged).  `status` is or-ed into, never
 *     cleared: zero it at the start of a cycle.  No kernel traps or waits without a bound.
 */
#ifndef TSV_H_
#define TSV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TSV_MAX_D 32          /* tree nodes per sequence the ABI can express (32-bit ancestor masks) */

enum { TSV_FP32 = 0, TSV_BF16 = 1 };

enum {
  TSV_OK = 0,
  TSV_ERR_NULL = -1,          /* a required pointer is NULL                                */
  TSV_ERR_ALIGN = -2,         /* a vector pointer is not 16-byte aligned                   */
  TSV_ERR_SHAPE = -3,         /* unsupported shape (see tsv_shape)                         */
  TSV_ERR_WORKSPACE = -4,     /* workspace NULL/too small/misaligned                       */
  TSV_ERR_CUDA = -5,          /* a CUDA runtime call failed (launch configuration etc.)    */
  TSV_ERR_LIMIT = -6          /* size beyond a built-in maximum of this entry point        */
};

enum {                         /* per-sequence status bits, device-written */
  TSV_ST_NODES = 1,           /* n_nodes[b] outside 1..D                                   */
  TSV_ST_PARENT = 2,          /* parent[0] != -1 or parent[n] outside [0, n)               */
  TSV_ST_LENGTH = 4,          /* L[b] < 0 or L[b] + D > max_L                              */
  TSV_ST_CSA_CAP = 8,         /* csa_cap[b] < (L + D) / m_csa                              */
  TSV_ST_HCA_CAP = 16,        /* hca_cap[b] < (L + D) / m_hca                              */
  TSV_ST_INTERNAL = 32        /* a bounded wait inside a kernel gave up                    */
};

enum {                         /* tsv_shape.flags */
  TSV_FLAG_FORCE_SIMT = 1,    /* tree_verify_attn: use the CUDA-core kernels even where the
                                  tensor-core kernels apply                                 */
  TSV_FLAG_HCA_DEFERRED = 2   /* C128-deferred refresh schedule (Section "Performance Optimization": C4 is refreshed
                                  timely, C128 writes are delayed and combined once the accepted path is known).
                                  For a sequence in which no HCA block can close inside the tree
                                  ((L % m_hca) + D < m_hca), branch_state_build builds no HCA branch states: the
                                  scratch fields hca_mx, hca_s, hca_acc_kv and new_hca_kv of that sequence are left
                                  untouched (hca_done is written, all 0), and accept_and_refresh folds the accepted
                                  path's (g_hca, c_hca) into the persistent open HCA block itself, in path order, with
                                  the arithmetic of branch_state_build -- the committed state is bit-identical to the
                                  timely schedule's.  Sequences in which a block may close inside the tree take the
                                  timely path.  Give the same flag to all three calls of a cycle.               */
};

/* Problem shape; HOST memory.
 * Supported: 1 <= D <= 32, window >= D, d and di multiples of 8 (d <= 1024, di <= 512),
 * H <= 256, HI <= 16, m_csa >= 1, m_hca >= 1, topk >= 1.  */
typedef struct tsv_shape {
  int32_t dtype;              /* TSV_FP32 | TSV_BF16                                        */
  int32_t B;                  /* sequences                                                  */
  int32_t D;                  /* node slots per sequence (verification budget, root incl.)  */
  int32_t H;                  /* query heads; one shared KV head (key == value)             */
  int32_t d;                  /* KV dim                                                     */
  int32_t m_csa, topk;        /* CSA block length; entries selected per node                */
  int32_t HI, di;             /* indexer heads x dim                                        */
  int32_t m_hca;              /* HCA block length                                           */
  int32_t window;             /* uncompressed window: query at p sees positions p-w+1 .. p  */
  float sm_scale;             /* softmax scale; <= 0 means 1/sqrt(d)                        */
  int64_t max_L;              /* bound on L[b] + D for every sequence; sizes grids/workspace */
  int32_t flags;              /* TSV_FLAG_*                                                 */
  int32_t reserved;
} tsv_shape;

/* Persistent state of ONE layer for all B sequences -- the committed prefix.
 * Read-only for branch_state_build / tree_verify_attn; written by accept_and_refresh only. */
typedef struct tsv_cache {
  int32_t *L;                 /* [B] committed tokens                                       */
  void *csa_kv;               /* CSA entries, rows of d;  sequence b owns rows               */
  void *csa_ik;               /*   csa_row0[b] .. csa_row0[b] + csa_cap[b]; same rows of di */
  const int64_t *csa_row0;    /* [B]                                                        */
  const int32_t *csa_cap;     /* [B] rows reserved                                          */
  void *hca_kv;               /* HCA entries, rows of d                                     */
  const int64_t *hca_row0;    /* [B]                                                        */
  const int32_t *hca_cap;     /* [B]                                                        */
  void *win_kv;               /* [B][window][d] ring of uncompressed KV, slot = pos % window */
  float *csa_mx, *csa_s;      /* [B] open CSA block: running max gate, sum of weights       */
  float *csa_acc_kv;          /* [B][d]  weighted sum of compression vectors                */
  float *csa_acc_ik;          /* [B][di] weighted sum of indexer-key vectors                */
  float *hca_mx, *hca_s;      /* [B] open HCA block                                         */
  float *hca_acc_kv;          /* [B][d]                                                     */
  int64_t csa_rows;           /* HOST value: rows allocated in csa_kv / csa_ik (all slabs); the tensor-core attention
                               * path builds its tensor maps from it: with 0 ("unknown") every shape runs on the
                               * CUDA-core path                                               */
  int64_t hca_rows;           /* HOST value: rows allocated in hca_kv (0: a layer without HCA entries) */
  /* Paged pool (Section "Temporary Branch States and Compressed-State Handling": a page-based pool seen as one logical
   * layer and several physical layers that share page-level pointers).  With page_table non-NULL the CSA and HCA entries
   * of a sequence do not sit in one slab each: logical page lp holds the entries of tokens [lp, lp + 1) * page_tokens, and
   * ONE table gives its physical page for every physical layer: entry e of the CSA cache (kv and indexer key) is row
   *     page_table[b][e / epp] * epp + e % epp,   epp = page_tokens / m_csa,
   * entry h of the HCA cache is row  page_table[b][h / hpp] * hpp + h % hpp,  hpp = page_tokens / m_hca.
   * The third physical layer is the token-level KV: win_kv is then not a ring but a pool of tok_rows rows, the KV of the
   * token at position p in row  page_table[b][p / page_tokens] * page_tokens + p % page_tokens  (only the last `window`
   * positions of a sequence are ever read; the refresh writes position L + i of every accepted node).
   * csa_row0 / hca_row0 are ignored then (may be NULL); csa_cap / hca_cap still give the entries the sequence's assigned
   * pages can hold, and the pages must cover positions up to L + D - 1.  page_tokens must be a multiple of m_csa and of
   * m_hca.  The tensor-core path fetches rows by 32-row TMA boxes where a page holds whole boxes of the layer (CSA: epp a
   * multiple of 32, e.g. 128-token pages with m_csa = 4: one box per page; window: page_tokens a multiple of 32); otherwise,
   * and for HCA rows beyond the first 32 entries unless hpp is a multiple of 32, it gathers the rows four at a time by
   * index. */
  const int32_t *page_table;  /* [B][max_pages] device, or NULL: flat slabs and window ring   */
  int32_t page_tokens;        /* HOST value                                                 */
  int32_t max_pages;          /* HOST value: columns of page_table                          */
  int64_t tok_rows;           /* HOST value: rows allocated in win_kv when it is a token pool */
} tsv_cache;

/* Per-cycle inputs of ONE layer for all tree nodes; read-only. */
typedef struct tsv_nodes {
  const void *q;              /* [B][D][H][d]   queries                                     */
  const void *kv;             /* [B][D][d]      the node's own uncompressed KV              */
  const void *c_csa;          /* [B][D][d]      CSA compression vector                      */
  const void *ikc;            /* [B][D][di]     CSA indexer-key compression vector          */
  const float *g_csa;         /* [B][D]         CSA gate logit                              */
  const void *c_hca;          /* [B][D][d]      HCA compression vector                      */
  const float *g_hca;         /* [B][D]         HCA gate logit                              */
  const void *iq;             /* [B][D][HI][di] indexer queries                             */
  const float *iw;            /* [B][D][HI]     indexer head weights                        */
  const int32_t *parent;      /* [B][D] parent[0] = -1, 0 <= parent[n] < n                  */
  const int32_t *n_nodes;     /* [B] 1..D; slots >= n_nodes[b] are padding                  */
} tsv_nodes;

/* Scratch pad of ONE layer: branch-private temporary state, written by branch_state_build,
 * read by tree_verify_attn and accept_and_refresh, dead afterwards. */
typedef struct tsv_scratch {
  float *csa_mx, *csa_s;      /* [B][D]  state of the open CSA block after node n           */
  float *csa_acc_kv;          /* [B][D][d]                                                  */
  float *csa_acc_ik;          /* [B][D][di]                                                 */
  float *hca_mx, *hca_s;      /* [B][D]                                                     */
  float *hca_acc_kv;          /* [B][D][d]                                                  */
  void *new_csa_kv;           /* [B][D][d]  entry closed at node n (valid where csa_done)   */
  void *new_csa_ik;           /* [B][D][di]                                                 */
  void *new_hca_kv;           /* [B][D][d]  (valid where hca_done)                          */
  uint8_t *csa_done;          /* [B][D] 1 iff (p_n + 1) % m_csa == 0                         */
  uint8_t *hca_done;          /* [B][D]                                                     */
} tsv_scratch;

/* Library version (major * 1000 + minor). */
int tsv_version(void);

/* Kernels this library has launched in this process so far (monotonic counter; reporting only). */
uint64_t tsv_kernel_launches(void);

/* Text for a TSV_ERR_* code; static storage. */
const char *tsv_error_string(int code);

/* Bytes of `workspace` tree_verify_attn needs for this shape (uses max_L).  0 on bad shape. */
size_t tsv_workspace_bytes(const tsv_shape *shape);

/*
 * branch_state_build -- temporary state isolation (Sections "Three-Stage Speculative Forward":
 * chains sharing a prefix reuse its state but compress independently after branching;
 * "Temporary Branch States and Compressed-State Handling": chain-private compressed tokens and
 * compression-intermediate buffers live in a scratch pad).
 *
 * For every node, in parent-before-child order: take the open-block state of the parent (the
 * root takes the persistent one), fold the node's (gate, compression vectors) into it by the
 * online softmax-pooling update  mx' = max(mx, g); s' = s e^{mx-mx'} + e^{g-mx'};
 * acc' = acc e^{mx-mx'} + e^{g-mx'} c  (an open block with p_n % m == 0 tokens is empty and its
 * stored numbers are ignored).  A node with (p_n + 1) % m == 0 closes the block: the entry
 * acc'/s' is rounded to the storage dtype into new_*[b][n], done[b][n] = 1 and the node's
 * state becomes empty (zeros).  Done for the CSA cache (kv entry + indexer key, same weights)
 * and the HCA cache.  Padding nodes get zero state and done = 0.  `cache` is not written.
 */
int branch_state_build(const tsv_shape *shape, const tsv_cache *cache, const tsv_nodes *nodes,
                       const tsv_scratch *scratch, int32_t *status /* [B] device */, void *stream);

/*
 * tree_verify_attn -- branch-aware causal verification (Section "Branch-Aware Causal Verification
 * and Isolation": a candidate attends to the accepted context and to the ancestors on its own
 * branch, never to other branches, whatever the physical order of the nodes).
 *
 * For node n and head h:  out = sum_j softmax_j(sm_scale q.K_j) K_j  with ONE softmax over
 *   (a) the top-k CSA entries by indexer score  sum_hi iw relu(iq . ik_e)  among the n_csa
 *       committed entries plus the entries closed inside the tree at strict ancestors of n
 *       (k_eff = min(topk, #candidates); ties to the lower block index),
 *   (b) all n_hca committed HCA entries plus those closed at strict ancestors,
 *   (c) the committed window positions max(0, p_n - w + 1) .. L-1,
 *   (d) the KV of n itself and of its ancestors.
 * out       [B][D][H][d] storage dtype; zero for padding nodes and flagged sequences.
 * topk_idx  [B][D][topk] int32 or NULL: ascending logical block indices of (a), -1 padded;
 *           index >= n_csa names the entry closed at the ancestor whose position lies in it.
 * workspace device, 256-byte aligned, >= tsv_workspace_bytes(shape); contents are scratch.
 * Needs `scratch` as written by branch_state_build of the same layer and cycle.
 */
int tree_verify_attn(const tsv_shape *shape, const tsv_cache *cache, const tsv_nodes *nodes,
                     const tsv_scratch *scratch, void *out, int32_t *topk_idx,
                     void *workspace, size_t workspace_bytes, int32_t *status, void *stream);

/*
 * accept_and_refresh -- accepted-path state refresh (Sections "Compressed-State Consistency and
 * Accepted-Path Refresh" and "Temporary Branch States and Compressed-State Handling": select a
 * specific path, keep its token-level KV, its completed CSA/HCA entries and its
 * compression-intermediate buffers, drop every rejected branch).
 *
 * Walk: cur = 0, path = [0]; repeat: c = lowest-index child of cur with
 * draft_tok[c] == target_tok[cur]; stop if none; append c.  Then, for every layer and
 * i < accept_len with n = path[i]: win_kv[(L+i) % window] = kv[n]; entries closed at n are
 * appended at rows (L+i)/m_csa and (L+i)/m_hca; the persistent open-block states become the
 * scratch states of the last accepted node; L += accept_len.
 * caches / nodes / scratch: HOST arrays of n_layers HOST pointers to the per-layer structs
 * (parent and n_nodes are read from nodes[0]).  Tokens are [B][D] int32.
 * accept_len [B], accept_path [B][D] (-1 padded), bonus_tok [B] (= target at the last accepted
 * node): device outputs.  A sequence with status[b] != 0 (on entry or found here, over ALL
 * layers) commits nothing in any layer and reports accept_len 0.
 */
int accept_and_refresh(const tsv_shape *shape, int32_t n_layers, const tsv_cache *const *caches,
                       const tsv_nodes *const *nodes, const tsv_scratch *const *scratch,
                       const int32_t *draft_tok, const int32_t *target_tok, int32_t *accept_len,
                       int32_t *accept_path, int32_t *bonus_tok, int32_t *status, void *stream);

/*
 * tree_verify_attn_static -- tree_verify_attn without a caller-provided workspace.
 * (No counterpart in the paper: this is a convenience of this library.)
 *
 * For callers that cannot allocate device memory at the point of the call -- an engine that
 * gives out all device memory from its own pool at start-up, a plug-in that must leave its
 * host's allocator alone, a request loop where an allocation would stall the device.  The
 * workspace lives in a device array of TSV_STATIC_WORKSPACE_BYTES built into the library
 * (each GPU that loads the library holds that much until the process exits).  The call runs
 * no cudaMalloc / cudaFree and no allocating library routine; inputs and outputs are still the
 * caller's.  Arguments, results and status handling are those of tree_verify_attn.
 *   - Shapes whose tsv_workspace_bytes() exceeds TSV_STATIC_WORKSPACE_BYTES are refused with
 *     TSV_ERR_LIMIT and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); that look-up makes the runtime load the library's device code on the device,
 *     which is when the array's bytes are reserved there.  Make that first call at start-up:
 *     before the rest of the device memory is handed out, and before starting any stream capture.
 *     If it fails (TSV_ERR_CUDA), nothing was enqueued and no error is left pending.
 *   - All calls on a device share the one array, which keeps whatever the last call left in
 *     it.  Nothing in it has to start at zero -- every region is written before it is read
 *     within a call -- but two calls that overlap on the GPU (different streams, no
 *     dependency between them) race on it: order them.
 */
#define TSV_STATIC_WORKSPACE_BYTES (16u << 20)
int tree_verify_attn_static(const tsv_shape *shape, const tsv_cache *cache, const tsv_nodes *nodes,
                            const tsv_scratch *scratch, void *out, int32_t *topk_idx,
                            int32_t *status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TSV_H_ */
