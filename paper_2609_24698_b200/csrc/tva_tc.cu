// tree_verify_attn on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 storage, d = 512: the tile plan and the
// merge of multi-chunk tiles.  (The attention kernel itself is in tva_tc_pair.cu.)
//
// Rows are grouped in plan tiles of 256 query rows = 256/H consecutive tree nodes x H heads; all of them attend over the
// SAME staged key rows (key == value, MQA), so S = Q K^T and O = P K are dense contractions.  Which node sees which key is
// a per-key bitmask applied to the S fragment after it is read back from tensor memory.
//
//   tc_plan_kernel   per (sequence, plan tile): the keys visible to at least one node of the tile, as four runs {CSA
//                    entries, HCA entries, window ring, packed misc rows} padded to 32 rows, with a node mask per key.
//                    Contiguous-run tiles (every node selects all CSA candidates, or the CSA slab is at most 2 x topk
//                    rows): the runs as 32-row TMA boxes.  Gathered tiles (selection far from dense, or a paged pool
//                    whose pages do not hold whole boxes): the first run holds only the entries some node of the tile
//                    selected, and every key is named by array << 30 | row for four-row TMA gathers.
//                    Each tile CTA leaves its record {tile, mode, keys} at the tile's scheduling position (its rank by
//                    estimated key count, most first); an extra CTA per sequence packs the small scattered rows.
//   tc_combine_pair_kernel  merges the chunks of the paired kernel's multi-chunk tiles (fixed order).
#include "tc_common.cuh"

namespace tsv {


// ------------------------------------------------------------------------------------------------ plan
constexpr int kRankTilesMax = 2048;                    // beyond that many tiles they keep their natural order
// Estimated number of keys a tile of a sequence stages, from its committed length and node count alone (for tiles on the
// contiguous-run path it is exact up to the entries closed inside the tree; only the order of the tiles depends on it).
__device__ __forceinline__ int tile_keys_estimate(const tsv_shape& s, int L, int nn, int tile, int npt) {
  if (L < 0 || (int64_t)L + s.D > s.max_L || nn < 1 || nn > s.D || tile * npt >= nn) return 0;
  auto r32 = [](int x) { return (x + kBoxRows - 1) / kBoxRows * kBoxRows; };
  const int n_csa = L / s.m_csa, n_hca = L / s.m_hca, nh_in = n_hca <= kHcaMiscMax ? n_hca : 0, win = min(L, s.window);
  if (n_csa <= 2 * s.topk) return r32(n_csa) + (n_hca > kHcaMiscMax ? r32(n_hca) : 0) + r32(win) + r32(nh_in + nn);
  return min(n_csa, npt * s.topk) + n_hca + win + 3 * nn;
}

// GENERAL: gathered tiles may occur (see gathered_tiles_possible); the instantiation without them keeps the short
// latency chain of the contiguous-run plan.
template <bool GENERAL>
__device__ __forceinline__ void tc_plan_tile(const tsv_shape& s, const TvaPlan& pl, const tsv_cache& c, const tsv_nodes& nd,
                                             const tsv_scratch& sc, char* __restrict__ ws, uint8_t* cmask, int* est, int* ahead_sm) {
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ int n_cand[8], win_lo[8];
  __shared__ int dense;
  const int tile = blockIdx.x, b = blockIdx.y, D = s.D, H = s.H;
  const int npt = tc::PR / H, n0 = tile * npt;
  const size_t tix = (size_t)b * pl.tc_nt + tile;
  uint32_t* krow = reinterpret_cast<uint32_t*>(ws + pl.off_krow) + tix * pl.tc_maxk;    // gathered tiles: array << 30 | row per key
  uint8_t* kmask = reinterpret_cast<uint8_t*>(ws + pl.off_kmask) + tix * pl.tc_maxk;
  int32_t* nkeys = reinterpret_cast<int32_t*>(ws + pl.off_nkeys) + tix;
  int32_t* mode = reinterpret_cast<int32_t*>(ws + pl.off_mode) + tix;
  // the cache row offsets are fetched together with the tree scalars (one memory latency for all)
  __shared__ uint8_t cdone[TSV_MAX_D], hdone[TSV_MAX_D];
  __shared__ int64_t row0_sm[2];
  // (the length and node count of "its" tile's sequence, for the ranking of the tiles: requested now, used after the tree's loads)
  const int ntile = s.B * pl.tc_nt;
  const bool ranked_order = ntile <= kRankTilesMax && blockIdx.x < (unsigned)pl.tc_nt;
  int eL = -1, enn = 0;
  if (ranked_order && (int)threadIdx.x < ntile) { eL = c.L[threadIdx.x / pl.tc_nt]; enn = nd.n_nodes[threadIdx.x / pl.tc_nt]; }
  if (threadIdx.x == 40) row0_sm[0] = c.page_table ? 0 : c.csa_row0[b];
  if (threadIdx.x == 41) row0_sm[1] = c.page_table ? 0 : c.hca_row0[b];
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
  if (ranked_order) {                                  // estimated key counts of all tiles
    if ((int)threadIdx.x < ntile) est[threadIdx.x] = tile_keys_estimate(s, eL, enn, threadIdx.x % pl.tc_nt, npt);
#pragma unroll 1
    for (int i = threadIdx.x + blockDim.x; i < ntile; i += blockDim.x)
      est[i] = tile_keys_estimate(s, c.L[i / pl.tc_nt], nd.n_nodes[i / pl.tc_nt], i % pl.tc_nt, npt);
  }
  // thread 0 leaves the tile's record {tile, mode, keys} at that position as soon as it knows the key count
  auto leave_record = [&](int nk, int md) {
    *nkeys = nk; *mode = md;
    reinterpret_cast<int4*>(ws + pl.off_order)[ntile <= kRankTilesMax ? *ahead_sm : (int)tix] = make_int4((int)tix, md, nk, 0);
  };
  // The kernel is launched as a programmatic dependent of the selection kernel (itself one of the state build) and runs
  // under those kernels' tails as far as it reads only the caller's inputs and the committed caches: the done flags are
  // worked out from the positions, and a tile no node of which ranks is planned completely.  It waits for the two kernels
  // (griddepcontrol.wait, below) before it reads what they write: the entries closed inside the tree (packing CTA), the
  // ranking nodes' mask rows.
  if (threadIdx.x < D) {
    const bool valid = !tm.status && (int)threadIdx.x < tm.nn;
    cdone[threadIdx.x] = valid && node_closes(tm.L, tm.depth[threadIdx.x], s.m_csa);
    hdone[threadIdx.x] = valid && node_closes(tm.L, tm.depth[threadIdx.x], s.m_hca);
  }
  __syncthreads();
  // The tile's scheduling position: how many tiles come before it by estimated key count (complete after the next barrier).
  if (ranked_order) {
    const int mine = est[tix];
    int ahead = 0;
#pragma unroll 1
    for (int j = threadIdx.x; j < ntile; j += blockDim.x) { const int e = est[j]; ahead += (e > mine) || (e == mine && j < (int)tix); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ahead += __shfl_xor_sync(0xffffffffu, ahead, o);
    if ((threadIdx.x & 31) == 0 && ahead) atomicAdd(ahead_sm, ahead);
  }
  // rows of the sequence's CSA and HCA entries: slabs, or through the page table of a paged pool
  RowAddr csa_row, hca_row;
  csa_row.pt = hca_row.pt = c.page_table ? c.page_table + (size_t)b * c.max_pages : nullptr;
  csa_row.per_page = c.page_table ? c.page_tokens / s.m_csa : 1; hca_row.per_page = c.page_table ? c.page_tokens / s.m_hca : 1;
  csa_row.row0 = row0_sm[0]; hca_row.row0 = row0_sm[1];
  // runs of consecutive rows exist in a paged pool only where a page holds whole 32-row boxes of the layer
  const bool csa_runs = !c.page_table || (csa_row.per_page % kBoxRows == 0 && c.page_tokens % kBoxRows == 0), hca_runs = !c.page_table || hca_row.per_page % kBoxRows == 0;
  if (blockIdx.x >= (unsigned)pl.tc_nt) {
    // The extra CTA of the sequence (grid x = tiles + 1): rows that are small and scattered (few HCA entries, tree nodes,
    // entries closed inside the tree) are packed into one contiguous per-sequence buffer so that TMA boxes can fetch
    // them.  Kept off the tile CTAs: the copy is a chain of its own (addresses, loads, stores).
    if (tm.status) return;
    const size_t rowb = (size_t)s.d * 2;
    const int nh_in = tm.n_hca <= kHcaMiscMax ? tm.n_hca : 0;
    int ncd = 0, nhd = 0;
#pragma unroll 1
    for (int j = 0; j < tm.nn; ++j) { ncd += cdone[j] != 0; nhd += hdone[j] != 0; }
    const int n_misc = nh_in + tm.nn + ncd + nhd;
    uint4* dst = reinterpret_cast<uint4*>(ws + pl.off_misc + (size_t)b * pl.tc_misc_rows * rowb);
    const int rows_out = (n_misc + kBoxRows - 1) / kBoxRows * kBoxRows;
    // The source of every packed row is worked out once (thread r: row r), then the copy runs flat over (row, 16-byte
    // piece) items, eight of a thread in flight.  Rows [0, first) and the zero padding behind n_misc are the caller's
    // data; the rows between are the state build's and copied after the wait.  (Compact code on purpose: the kernel runs
    // once per layer with cold instruction caches.)
    __shared__ const uint4* srcs[kHcaMiscMax + 3 * TSV_MAX_D];
    constexpr int CPR = tc::DH * 2 / 16;               // 16-byte pieces per row
#pragma unroll 1
    for (int r = threadIdx.x; r < rows_out; r += blockDim.x) {
      const char* src = nullptr;
      if (r < nh_in) src = (const char*)c.hca_kv + (size_t)hca_row(r) * rowb;
      else if (r < nh_in + tm.nn) src = (const char*)nd.kv + ((size_t)b * D + (r - nh_in)) * rowb;
      else if (r < n_misc) {
        int ord = r - nh_in - tm.nn;
        const bool isc = ord < ncd;
        if (!isc) ord -= ncd;
        const uint8_t* dn = isc ? cdone : hdone;
        int a = 0;
#pragma unroll 1
        for (int j = 0; j < tm.nn; ++j) if (dn[j]) { if (ord == 0) { a = j; break; } --ord; }
        src = (const char*)(isc ? sc.new_csa_kv : sc.new_hca_kv) + ((size_t)b * D + a) * rowb;
      }
      srcs[r] = reinterpret_cast<const uint4*>(src);
    }
    __syncthreads();
    const int first = nh_in + tm.nn;
#pragma unroll 1
    for (int phase = 0; phase < 2; ++phase) {
      if (phase) {
        if (n_misc == first) break;
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the entries closed inside the tree
      }
      const int lo = phase ? first * CPR : 0, hi = phase ? n_misc * CPR : rows_out * CPR;
#pragma unroll 1
      for (int i0 = lo + threadIdx.x; i0 < hi; i0 += 8 * blockDim.x) {
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int i = i0 + k * blockDim.x, r = i / CPR;
          const bool in = i < hi && (phase || r < first || r >= n_misc);
          const uint4* src = in ? srcs[r] : nullptr;
          v[k] = src ? __ldg(src + (i - r * CPR)) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int i = i0 + k * blockDim.x, r = i / CPR;
          if (i < hi && (phase || r < first || r >= n_misc)) dst[i] = v[k];
        }
      }
    }
    return;
  }
  if (threadIdx.x < 32) {                              // lane nl: candidates and window start of node n0 + nl
    const int lane = threadIdx.x, n = n0 + lane;
    const uint32_t cmaskbits = __ballot_sync(0xffffffffu, lane < D && cdone[lane]);   // nodes that close a CSA block
    const bool real = lane < npt && n < tm.nn;
    const int nc = tm.n_csa + (real ? __popc(tm.anc[n] & ((1u << n) - 1u) & cmaskbits) : 0);   // + blocks closed at strict ancestors
    if (lane < npt) {
      n_cand[lane] = nc;
      win_lo[lane] = max(0, tm.L + tm.depth[real ? n : 0] - s.window + 1);
    }
    const uint32_t over = __ballot_sync(0xffffffffu, real && nc > s.topk);
    if (lane == 0) dense = over == 0;
  }
  __syncthreads();
  if (tm.status || n0 >= tm.nn) { if (threadIdx.x == 0) leave_record(0, 1); return; }
  const int nvalid = min(npt, tm.nn - n0);
  const uint32_t validbits = (1u << nvalid) - 1u;
  const int n_csa = tm.n_csa;
  // Ranked nodes: node bits per committed CSA entry (cmask) and, per node, which blocks closed inside the tree are in
  // its selection (bit = block index - n_csa).  The selection kernel left, for every node that ranks, a byte per
  // candidate (1 = selected): the rows of the tile's nodes are combined sixteen entries at a time (coalesced 16-byte
  // loads; the tile CTA of a ranked sequence is on the critical path of the whole stage).
  //
  // Where gathered tiles may occur the array is padded by one word after every `per` entries (per: the power of two that
  // spreads the entries over the CTA's threads): the compaction below gives a thread `per` consecutive entries, and
  // without the padding the threads of a warp would all read the same bank.
  __shared__ uint32_t newc_bits[8];
  int psh = 3;                                         // log2(per)
  if (GENERAL) while (((int)blockDim.x << psh) < n_csa) ++psh;
  auto phys = [&](int i) { return GENERAL ? i + ((i >> psh) << 2) : i; };
  // Contiguous-run tiles with ranking nodes (`late`): everything that does not depend on the selection -- boxes, the masks of
  // the HCA, window and packed runs -- is written before the wait; after it only the masks of the committed CSA run (the
  // combined mask rows, stored straight into the key masks) and of the entries closed inside the tree.
  const bool runs_ok = !GENERAL || ((dense || n_csa <= 2 * s.topk) && csa_runs && (hca_runs || tm.n_hca <= kHcaMiscMax));
  const bool late = !dense && runs_ok;
  uint32_t allbits = 0, rankbits = 0;                  // nodes that take every committed entry / nodes that rank
#pragma unroll 1
  for (int nl = 0; nl < nvalid; ++nl) { if (n_cand[nl] <= s.topk) allbits |= 1u << nl; else rankbits |= 1u << nl; }
  const uint8_t* mrow = reinterpret_cast<const uint8_t*>(ws + pl.off_selmask) + ((size_t)b * D + n0) * pl.mask_ld;
  // In-tree entries: candidate n_csa + o of a node is the block closed at the o-th of its strict ancestors that closed one.
  // Warp nl looks at node n0 + nl, lane a at ancestor a: one load per lane, all in flight together (the caller synchronises).
  auto fetch_newc_bits = [&]() {
    const int nl = threadIdx.x >> 5, a = threadIdx.x & 31;
    if (nl < 8) {
      const uint32_t closed = __ballot_sync(0xffffffffu, a < D && cdone[a]);
      uint32_t v = 0;
      if (nl < nvalid && ((rankbits >> nl) & 1u)) {
        const uint32_t up = tm.anc[n0 + nl] & closed & ((1u << (n0 + nl)) - 1u);     // strict ancestors that closed a block
        if ((up >> a) & 1u) {
          const int o = __popc(up & ((1u << a) - 1u));
          const int dblk = (tm.L + tm.depth[a]) / s.m_csa - n_csa;
          if (mrow[(size_t)nl * pl.mask_ld + n_csa + o] && dblk >= 0 && dblk < 32) v = 1u << dblk;
        }
      }
      v = __reduce_or_sync(0xffffffffu, v);
      if (a == 0) newc_bits[nl] = v;
    }
  };
  // sixteen committed entries from entry i: the node bits of each as four words of four mask bytes
  auto combine16 = [&](int i, uint32_t acc[4]) {
    const uint32_t all4 = 0x01010101u * allbits;
    acc[0] = acc[1] = acc[2] = acc[3] = all4;
#pragma unroll
    for (int nl = 0; nl < 8; ++nl) {
      if ((rankbits >> nl) & 1u) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(mrow + (size_t)nl * pl.mask_ld + i));
        acc[0] |= (v.x & 0x01010101u) << nl; acc[1] |= (v.y & 0x01010101u) << nl;
        acc[2] |= (v.z & 0x01010101u) << nl; acc[3] |= (v.w & 0x01010101u) << nl;
      }
    }
  };
  if (!dense && !runs_ok) {
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the selection's mask rows
    fetch_newc_bits();
    uint32_t* cm32 = reinterpret_cast<uint32_t*>(cmask);
#pragma unroll 2
    for (int i = 16 * threadIdx.x; i < n_csa; i += 16 * blockDim.x) {
      uint32_t acc[4];
      combine16(i, acc);
#pragma unroll
      for (int q = 0; q < 4; ++q) cm32[phys(i + 4 * q) >> 2] = acc[q];      // (bytes past n_csa are never read)
    }
    __syncthreads();
  }
  // is the entry closed at node a (a strict ancestor of node n0 + nl) among that node's selected CSA entries?
  auto newc_selected = [&](int nl, int a) {
    if (n_cand[nl] <= s.topk) return true;
    const int dblk = (tm.L + tm.depth[a]) / s.m_csa - n_csa;
    return dblk >= 0 && dblk < 32 && ((newc_bits[nl] >> dblk) & 1u);
  };
  {
    // the packed per-sequence rows (written by the sequence's extra CTA): few HCA entries, tree nodes, entries closed in the tree
    const int nh_in = tm.n_hca <= kHcaMiscMax ? tm.n_hca : 0;
    int ncd = 0, nhd = 0;
#pragma unroll 1
    for (int j = 0; j < tm.nn; ++j) { ncd += cdone[j] != 0; nhd += hdone[j] != 0; }
    const int n_misc = nh_in + tm.nn + ncd + nhd;
    // Ranked nodes still take the contiguous-run path while the run is at most twice the selection size: all committed
    // entries are staged and the unselected ones are masked per node.  Beyond that (or where a paged pool's pages do not
    // hold whole boxes) the tile is GATHERED: the same four runs, but the first holds only the committed entries some node
    // of the tile selected, and every key is named by its row (array << 30 | row) for four-row TMA gathers.
    int n_uni = n_csa;                                 // keys of the first run
    __shared__ int uni_tot;
    if (!runs_ok) {
      // Ordered compaction of the selected entries: a thread owns `per` consecutive entries, counts its selected ones
      // (four mask bytes per word), one block scan, then writes its rows and masks at consecutive positions.
      __shared__ int wsum_c[33];
      const uint32_t* cm32 = reinterpret_cast<const uint32_t*>(cmask);
      const int per = 1 << psh, beg = min(n_csa, (int)threadIdx.x << psh), end = min(n_csa, beg + per);
      const uint32_t* mine = cm32 + (phys(beg) >> 2);  // this thread's words (its share starts on a word: per is a multiple of 8)
      const uint32_t dmask = dense ? validbits : 0u;   // (a dense tile comes here only from a paged pool with odd pages)
      int cnt = 0;
      for (int i = beg; i < end; i += 4) {
        uint32_t w = dense ? 0x01010101u * dmask : mine[(i - beg) >> 2];
        if (end - i < 4) w &= (1u << (8 * (end - i))) - 1u;
        cnt += (w & 0xFFu ? 1 : 0) + (w & 0xFF00u ? 1 : 0) + (w & 0xFF0000u ? 1 : 0) + (w & 0xFF000000u ? 1 : 0);
      }
      int total;
      int pos = block_excl_scan(cnt, wsum_c, total);
      if (threadIdx.x == 0) uni_tot = total;
      for (int i = beg; i < end; i += 4) {
        uint32_t w = dense ? 0x01010101u * dmask : mine[(i - beg) >> 2];
        if (end - i < 4) w &= (1u << (8 * (end - i))) - 1u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t m = (w >> (8 * j)) & 0xFFu;
          if (m) { krow[pos] = (uint32_t)csa_row(i + j); kmask[pos] = (uint8_t)m; ++pos; }
        }
      }
      __syncthreads();
      n_uni = uni_tot;
    }
    {
      int2* box = reinterpret_cast<int2*>(ws + pl.off_box) + tix * (size_t)(pl.tc_maxk / kBoxRows);
      // four runs, each padded to whole boxes: committed CSA entries, HCA entries (when too many for the packed rows),
      // the window ring, the packed rows.  One pass over all keys: a thread finds the run of its key by comparison, so
      // the runs' (short, latency-bound) mask computations overlap instead of following each other.
      // the window: the ring in slot order, or (paged pool) the positions from the 32-aligned start of the box that holds
      // the oldest window position up to L - 1 (the positions before the window are masked like every position a node
      // cannot see)
      const int win_a = c.page_table ? (max(0, tm.L - s.window) & ~(kBoxRows - 1)) : 0;
      const int cnt[4] = {n_uni, tm.n_hca > kHcaMiscMax ? tm.n_hca : 0, c.page_table ? tm.L - win_a : min(tm.L, s.window), n_misc};
      const int64_t start[4] = {0, 0, (int64_t)b * s.window, (int64_t)b * pl.tc_misc_rows};
      int k0[5];                                       // first key of each run
      k0[0] = 0;
#pragma unroll
      for (int g = 0; g < 4; ++g) k0[g + 1] = k0[g] + (cnt[g] + kBoxRows - 1) / kBoxRows * kBoxRows;
      const int kb = k0[4];
      // row of key i of run g (g >= 1, or the whole CSA slab as run 0 of a contiguous-run tile)
      auto run_row = [&](int g, int i) -> int64_t {
        return g == 0 ? csa_row(i) : g == 1 ? hca_row(i) : (g == 2 && c.page_table) ? tok_row_of(c, s, b, win_a + i) : start[g] + i;
      };
      if (runs_ok) {
        for (int bi = threadIdx.x; bi < kb / kBoxRows; bi += blockDim.x) {
          const int k = bi * kBoxRows;
          const int g = k >= k0[3] ? 3 : (k >= k0[2] ? 2 : (k >= k0[1] ? 1 : 0));
          // (a box of a cache run never crosses a page: it starts on a multiple of 32 entries and per_page is one too)
          box[bi] = make_int2(g, (int)run_row(g, k - k0[g]));
        }
      }
      // (gathered tiles: the compaction above has written the keys of the first run already)
#pragma unroll 1
      for (int k = (runs_ok ? 0 : n_uni) + threadIdx.x; k < kb; k += blockDim.x) {
        const int g = k >= k0[3] ? 3 : (k >= k0[2] ? 2 : (k >= k0[1] ? 1 : 0));
        const int i = k - k0[g];
        uint32_t m = 0;
        if (late && (g == 0 || (g == 3 && i >= nh_in + tm.nn && i < nh_in + tm.nn + ncd))) continue;   // after the wait, below
        if (i < cnt[g]) {
          if (g == 0) m = validbits;                                 // (dense contiguous-run tiles only: see the loop's start and the line above)
          else if (g == 1) m = validbits;
          else if (g == 2) {
            const int pos = c.page_table ? win_a + i : tm.L - 1 - ((tm.L - 1 - i) % s.window);
#pragma unroll 1
            for (int nl = 0; nl < nvalid; ++nl) if (pos >= win_lo[nl]) m |= 1u << nl;
          } else if (i < nh_in) m = validbits;
          else if (i < nh_in + tm.nn) {
            const int j = i - nh_in;
#pragma unroll 1
            for (int nl = 0; nl < nvalid; ++nl) if ((tm.anc[n0 + nl] >> j) & 1u) m |= 1u << nl;
          } else {
            int ord = i - nh_in - tm.nn;
            const bool isc = ord < ncd;
            if (!isc) ord -= ncd;
            const uint8_t* dn = isc ? cdone : hdone;
            int a = 0;
#pragma unroll 1
            for (int j = 0; j < tm.nn; ++j) if (dn[j]) { if (ord == 0) { a = j; break; } --ord; }
#pragma unroll 1
            for (int nl = 0; nl < nvalid; ++nl)
              if (a != n0 + nl && ((tm.anc[n0 + nl] >> a) & 1u) && (!isc || newc_selected(nl, a))) m |= 1u << nl;
          }
        }
        kmask[k] = (uint8_t)m;
        // gathered tiles: the key's row; the padding of a run repeats the run's first row (masked)
        if (!runs_ok) krow[k] = ((uint32_t)g << 30) | (uint32_t)(cnt[g] ? run_row(g, i < cnt[g] ? i : 0) : 0);
      }
      if (threadIdx.x == 0) leave_record(kb, runs_ok ? 1 : 2);
      if (late) {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the selection's mask rows
        fetch_newc_bits();
        // the committed CSA run (its first key is key 0 of the tile): sixteen key masks per store; the run's padding is zero
        uint4* km4 = reinterpret_cast<uint4*>(kmask);
        for (int i = 16 * threadIdx.x; i < k0[1]; i += 16 * blockDim.x) {
          uint32_t acc[4] = {0u, 0u, 0u, 0u};
          if (i < n_csa) combine16(i, acc);             // (a mask row holds a multiple of 16 bytes that covers n_csa)
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int left = n_csa - (i + 4 * q);
            if (left < 4) acc[q] = left <= 0 ? 0u : acc[q] & ((1u << (8 * left)) - 1u);
          }
          km4[i >> 4] = make_uint4(acc[0], acc[1], acc[2], acc[3]);
        }
        __syncthreads();
        // the CSA entries closed inside the tree (ncd keys of the packed run)
        if ((int)threadIdx.x < ncd) {
          int ord = threadIdx.x, a = 0;
#pragma unroll 1
          for (int j = 0; j < tm.nn; ++j) if (cdone[j]) { if (ord == 0) { a = j; break; } --ord; }
          uint32_t m = 0;
#pragma unroll 1
          for (int nl = 0; nl < nvalid; ++nl)
            if (a != n0 + nl && ((tm.anc[n0 + nl] >> a) & 1u) && newc_selected(nl, a)) m |= 1u << nl;
          kmask[k0[3] + nh_in + tm.nn + threadIdx.x] = (uint8_t)m;
        }
      }
      return;
    }
  }
}

// Plan of every (sequence, 256-row tile).  Each tile CTA leaves one 16-byte record {tile, mode, keys} at the tile's
// scheduling position: its rank among all tiles by estimated key count, most first, which every CTA works out for itself
// from the lengths and node counts of all sequences (the paired attention kernel takes the tiles in that order, long
// ones first and short ones in the tail, and learns all it needs about its tile from one load).  A tile no node of which
// ranks is planned from the caller's inputs alone: its CTA never waits for the kernels before this one.
// NT threads per CTA: 256, or 1024 for gathered tiles over long candidate lists (the union of a tile's selections over tens
// of thousands of entries is the work of ONE CTA, alone on its SM).
template <bool GENERAL, int NT>
__global__ void __launch_bounds__(NT) tc_plan_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                                         const tsv_scratch sc, char* __restrict__ ws) {
  extern __shared__ uint8_t cmask_sm[];                // [cand_cap] node bits per committed CSA entry (ranked case only)
  __shared__ int est_sm[kRankTilesMax];
  __shared__ int ahead_sm;
  const bool tile_cta = blockIdx.x < (unsigned)pl.tc_nt;
  const size_t tix = (size_t)blockIdx.y * pl.tc_nt + blockIdx.x;
  if (threadIdx.x == 0) ahead_sm = 0;
  if (threadIdx.x < 2 && tile_cta)                      // finished-chunk counters of the tile's two 128-row halves
    reinterpret_cast<int32_t*>(ws + pl.off_tcnt)[tix * 2 + threadIdx.x] = 0;
  tc_plan_tile<GENERAL>(s, pl, c, nd, sc, ws, cmask_sm, est_sm, &ahead_sm);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // (at the END of the CTA's work: the attention kernel's CTAs take their places as this kernel's leave)
  // one CTA waits for the selection in any case, so that the completion of this kernel implies that one's
  if (blockIdx.x == 0 && blockIdx.y == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------ merge
// Merge of the paired kernel's multi-chunk tiles (launched with its general instantiation): every chunk left its NORMALISED partial output (bf16) with
// the row's (reference max, sum); the row's output is the average of the partial outputs weighted by sum * 2^(max - row max).
// grid (128-row tiles, sequences, groups of 8 rows): a warp merges one row, a lane owns 16 consecutive columns; the chunks
// are accumulated in order, four chunks' loads in flight.
__global__ void __launch_bounds__(256) tc_combine_pair_kernel(const tsv_shape s, const TvaPlan pl, void* __restrict__ out_, const char* __restrict__ ws) {
  using namespace tc;
  const int rt = blockIdx.x, tile = rt >> 1, b = blockIdx.y;
  const size_t tix = (size_t)b * pl.tc_nt + tile, rix = (size_t)b * 2 * pl.tc_nt + rt;
  const int mode = reinterpret_cast<const int32_t*>(ws + pl.off_mode)[tix];
  const int nk = reinterpret_cast<const int32_t*>(ws + pl.off_nkeys)[tix];
  if ((mode != 1 && mode != 2) || nk <= 0) return;
  int nch, CL;
  chunking_x(nk, true, nch, CL);
  if (nch <= 1) return;                                          // the paired kernel wrote the output itself
  const int rows_seq = s.D * s.H, row0 = rt * BM;
  const int lane = threadIdx.x & 31, row = blockIdx.z * 8 + (threadIdx.x >> 5);
  if (row >= BM || row0 + row >= rows_seq) return;
  // (a chunk's bf16 tile lies at the start of the chunk's slot of BM x DH floats)
  const uint4* po = reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(ws + pl.off_tpo) + (rix * pl.tc_chmax * 2 * BM + row) * DH) + 2 * lane;
  const float2* pml = reinterpret_cast<const float2*>(ws + pl.off_tpml) + rix * pl.tc_chmax * BM + row;
  float m = -INFINITY;
  for (int ch = lane; ch < nch; ch += 32) { const float2 ml = pml[(size_t)ch * BM]; if (ml.y > 0.f) m = fmaxf(m, ml.x); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float l = 0.f, acc[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) acc[k] = 0.f;
  for (int c0 = 0; c0 < nch; c0 += 4) {
    float2 ml[4];
    uint4 v[4][2];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int ch = c0 + u < nch ? c0 + u : nch - 1;
      ml[u] = pml[(size_t)ch * BM];
      v[u][0] = po[(size_t)ch * 2 * BM * (DH / 8)]; v[u][1] = po[(size_t)ch * 2 * BM * (DH / 8) + 1];
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (c0 + u >= nch || !(ml[u].y > 0.f)) continue;
      const float w = ml[u].y * exp2f(ml[u].x - m);
      l += w;
      const uint32_t wd[8] = {v[u][0].x, v[u][0].y, v[u][0].z, v[u][0].w, v[u][1].x, v[u][1].y, v[u][1].z, v[u][1].w};
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        acc[2 * k] = fmaf(__uint_as_float(wd[k] << 16), w, acc[2 * k]);
        acc[2 * k + 1] = fmaf(__uint_as_float(wd[k] & 0xFFFF0000u), w, acc[2 * k + 1]);
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  uint32_t o[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[2 * k] * inv, acc[2 * k + 1] * inv);
    o[k] = *reinterpret_cast<const uint32_t*>(&h2);
  }
  uint4* orow = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0 + row) * DH) + 2 * lane;
  orow[0] = make_uint4(o[0], o[1], o[2], o[3]);
  orow[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

bool tva_tc_eligible(const tsv_shape& s) {
  return s.dtype == TSV_BF16 && s.d == tc::DH && s.H >= 32 && s.H <= 128 && (128 % s.H) == 0 && !(s.flags & TSV_FLAG_FORCE_SIMT);
}

void tva_tc_plan_sizes(const tsv_shape& s, TvaPlan& p) {
  const int npt = tc::PR / s.H;
  p.tc_nt = (s.D * s.H + tc::PR - 1) / tc::PR;
  const int64_t ksel = p.cand_cap < s.topk ? p.cand_cap : s.topk;
  int64_t uni = (int64_t)npt * ksel;
  if (uni > p.cand_cap) uni = p.cand_cap;
  int64_t mk = uni + s.max_L / s.m_hca + s.window + 3 * (int64_t)s.D + 8;
  const int64_t br = kBoxRows;
  p.tc_misc_rows = (int32_t)((kHcaMiscMax + 3 * s.D + br - 1) / br * br);
  // (+ one box: in a paged pool the window run starts on a 32-aligned position and may be a box longer than the window)
  // (a tile takes the whole committed CSA run only while that is at most twice the selection size)
  const int64_t run_csa = p.cand_cap < 2 * (int64_t)s.topk ? p.cand_cap : 2 * (int64_t)s.topk;
  const int64_t runs = (run_csa + br - 1) / br * br + (s.max_L / s.m_hca + br - 1) / br * br + (s.window + br - 1) / br * br + br + p.tc_misc_rows;
  if (runs > mk) mk = runs;
  // gathered tiles: the union of the nodes' selections, HCA entries, window and packed rows as four runs padded to boxes
  const int64_t gath = (uni + br - 1) / br * br + (s.max_L / s.m_hca + br - 1) / br * br + (s.window + br - 1) / br * br + br + p.tc_misc_rows;
  if (gath > mk) mk = gath;
  p.tc_maxk = (int32_t)((mk + 127) / 128 * 128);
  p.tc_chmax = (p.tc_maxk + tc::NC - 1) / tc::NC;
}

static size_t plan_smem_bytes(const TvaPlan& p) { return p.need_scores ? (((size_t)p.cand_cap + 3) & ~(size_t)3) + 4 * 1024 + 16 : 0; }   // node bits per entry, cleared by words (+ the padding words)
// Can the plan kernel produce a gathered tile for these capacities?  (A committed CSA run longer than twice the
// selection size, or a paged pool whose pages do not hold whole 32-row boxes of a layer.)
static bool gathered_tiles_possible(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c) {
  if (p.need_scores && p.cand_cap > 2 * (int64_t)s.topk) return true;
  if (c.page_table) {
    const int epp = c.page_tokens / s.m_csa, hpp = c.page_tokens / s.m_hca;
    if (epp % kBoxRows || c.page_tokens % kBoxRows) return true;
    if (hpp % kBoxRows && s.max_L / s.m_hca > kHcaMiscMax) return true;
  }
  return false;
}

// Host-side work of the tensor-core path that can fail, before anything of the call is enqueued.
int prepare_tva_tc(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, void* out, char* ws, TvaTcPrep& prep) {
  const size_t plan_sm = plan_smem_bytes(p);
  if (plan_sm > 32 * 1024 && (cudaFuncSetAttribute(tc_plan_kernel<true, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_sm) != cudaSuccess ||
                              cudaFuncSetAttribute(tc_plan_kernel<true, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_sm) != cudaSuccess ||
                              cudaFuncSetAttribute(tc_plan_kernel<false, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_sm) != cudaSuccess)) {
    cudaGetLastError();
    return TSV_ERR_CUDA;
  }
  TSV_PREP((tc_plan_kernel<true, 1024>));
  TSV_PREP((tc_plan_kernel<true, 256>));
  TSV_PREP((tc_plan_kernel<false, 256>));
  TSV_PREP(tc_combine_pair_kernel);
  return prepare_tva_tc_pair(s, p, c, nd, out, ws, prep);
}

int launch_tva_tc(const tsv_shape& s, const TvaPlan& p, const TvaTcPrep& prep, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                  void* out, char* ws, int32_t* status, cudaStream_t st, bool with_plan) {
  const bool gathered = gathered_tiles_possible(s, p, c);
  const dim3 pgrid(p.tc_nt + 1, s.B);                                                                              // x: tiles + the packing CTA
  if (with_plan) {
    cudaLaunchConfig_t cfg = {};
    const bool wide = gathered && p.cand_cap > 8192;    // long candidate lists: the CTA's passes over all entries want many threads
    cfg.gridDim = pgrid; cfg.blockDim = dim3(wide ? 1024 : 256, 1, 1); cfg.dynamicSmemBytes = plan_smem_bytes(p); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;        // may start under the selection kernel's tail (it waits inside)
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (wide) cudaLaunchKernelEx(&cfg, tc_plan_kernel<true, 1024>, s, p, c, nd, sc, ws);
    else if (gathered) cudaLaunchKernelEx(&cfg, tc_plan_kernel<true, 256>, s, p, c, nd, sc, ws);
    else cudaLaunchKernelEx(&cfg, tc_plan_kernel<false, 256>, s, p, c, nd, sc, ws);
  }
  count_launch();
  // general: some tile may have more than two chunks of the longest kind, or be gathered; then every multi-chunk tile
  // leaves bf16 partial outputs for the merge kernel
  const bool general = (p.tc_maxk + tc::NCX - 1) / tc::NCX > 2 || gathered;
  const int r = launch_tva_tc_pair(s, p, prep, general, out, ws, status, st);
  if (r != TSV_OK) return r;
  if (general && p.tc_chmax > 1) {
    tc_combine_pair_kernel<<<dim3(2 * p.tc_nt, s.B, tc::BM / 8), 256, 0, st>>>(s, p, out, ws);   // z: groups of 8 rows
    count_launch();
  }
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
