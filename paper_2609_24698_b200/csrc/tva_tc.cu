// tree_verify_attn on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 storage, d = 512: the tile plan, the
// pointer-gather attention kernel and the merge of multi-chunk tiles.  (The main attention kernel, for key lists made of
// contiguous runs, is in tva_tc_pair.cu.)
//
// Rows are grouped in plan tiles of 256 query rows = 256/H consecutive tree nodes x H heads; all of them attend over the
// SAME staged key rows (key == value, MQA), so S = Q K^T and O = P K are dense contractions.  Which node sees which key is
// a per-key bitmask applied to the S fragment after it is read back from tensor memory.
//
//   tc_plan_kernel   per (sequence, plan tile): the keys visible to at least one node of the tile.
//                    mode 1 (every node selects all CSA candidates, or the CSA slab is at most 2 x topk rows): contiguous
//                    runs {CSA slab, HCA slab, window ring, packed misc rows} as 32-row TMA boxes + node masks;
//                    mode 0 (selection far from dense): row pointers of the union of the nodes' selections + masks.
//                    Each tile CTA leaves its record {tile, mode, keys} at the scheduling position the selection kernel
//                    computed (most keys first); an extra CTA per sequence packs the small scattered rows.
//   tc_attn_kernel   mode-0 tiles, one CTA per 128 rows and chunk of <= 512 keys:
//       phase 1  S[128 x CL] = Q K^T      tcgen05.mma kind::f16, A = Q slice (smem, K-major), B = 256 key rows x 64 dims
//       phase 2  exact softmax of the chunk on the fp32 S read with tcgen05.ld; P (bf16) written back over S (tcgen05.st)
//       phase 3  O[128 x 256] = P K[:, half] twice; A = P from TMEM, B = 64 key rows x 256 dims (smem, MN-major)
//     Operand tiles stream through a ring of seven 32 KiB slots filled with 16-byte cp.async copies written in the
//     128-byte swizzle pattern (any row from any source array, zero fill for padding), four stages ahead of the MMA
//     issue; slots are released by tcgen05.commit on per-slot mbarriers.  Every wait is bounded.
//   tc_combine_kernel merges the chunks of mode-0 tiles that needed more than one (fixed order), per 128 rows.
#include "tc_common.cuh"

namespace tsv {


// ------------------------------------------------------------------------------------------------ plan
// GENERAL: gathered tiles may occur (see gathered_tiles_possible); the instantiation without them keeps the short
// latency chain of the contiguous-run plan.
template <bool GENERAL>
__device__ __forceinline__ void tc_plan_tile(const tsv_shape& s, const TvaPlan& pl, const tsv_cache& c, const tsv_nodes& nd,
                                             const tsv_scratch& sc, char* __restrict__ ws, uint8_t* cmask) {
  __shared__ TreeMeta tm;
  __shared__ TreeStage tstage;
  __shared__ int n_cand[8], win_lo[8];
  __shared__ int dense;
  const int tile = blockIdx.x, b = blockIdx.y, D = s.D, H = s.H;
  const int npt = tc::PR / H, n0 = tile * npt;
  const size_t tix = (size_t)b * pl.tc_nt + tile;
  uint64_t* kptr = reinterpret_cast<uint64_t*>(ws + pl.off_kptr) + tix * pl.tc_maxk;
  uint8_t* kmask = reinterpret_cast<uint8_t*>(ws + pl.off_kmask) + tix * pl.tc_maxk;
  int32_t* nkeys = reinterpret_cast<int32_t*>(ws + pl.off_nkeys) + tix;
  // the done flags and the cache row offsets are fetched together with the tree scalars (one memory latency for all)
  __shared__ uint8_t cdone[TSV_MAX_D], hdone[TSV_MAX_D];
  __shared__ int64_t row0_sm[2];
  if (threadIdx.x >= 64 && threadIdx.x < 64 + D) cdone[threadIdx.x - 64] = sc.csa_done[(size_t)b * D + threadIdx.x - 64];
  if (threadIdx.x >= 96 && threadIdx.x < 96 + D) hdone[threadIdx.x - 96] = sc.hca_done[(size_t)b * D + threadIdx.x - 96];
  if (threadIdx.x == 40) row0_sm[0] = c.page_table ? 0 : c.csa_row0[b];
  if (threadIdx.x == 41) row0_sm[1] = c.page_table ? 0 : c.hca_row0[b];
  coop_tree_meta(tm, tstage, s, c.L + b, nd.parent + (size_t)b * D, nd.n_nodes + b, c.csa_cap + b, c.hca_cap + b);
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
    if (tm.status || !pl.tc_tma) return;
    const size_t rowb = (size_t)s.d * 2;
    const int nh_in = tm.n_hca <= kHcaMiscMax ? tm.n_hca : 0;
    int ncd = 0, nhd = 0;
    for (int j = 0; j < tm.nn; ++j) { ncd += cdone[j] != 0; nhd += hdone[j] != 0; }
    const int n_misc = nh_in + tm.nn + ncd + nhd;
    uint4* dst = reinterpret_cast<uint4*>(ws + pl.off_misc + (size_t)b * pl.tc_misc_rows * rowb);
    const int rows_out = (n_misc + kBoxRows - 1) / kBoxRows * kBoxRows, cpr = (int)(rowb / 16);
    // warp per row, eight rows of a warp in flight: the source of a row is worked out once, all loads of the batch are
    // issued before the first store
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    auto row_src = [&](int r) -> const uint4* {
      const char* src = nullptr;
      if (r < nh_in) src = (const char*)c.hca_kv + (size_t)hca_row(r) * rowb;
      else if (r < nh_in + tm.nn) src = (const char*)nd.kv + ((size_t)b * D + (r - nh_in)) * rowb;
      else if (r < n_misc) {
        int ord = r - nh_in - tm.nn;
        const bool isc = ord < ncd;
        if (!isc) ord -= ncd;
        const uint8_t* dn = isc ? cdone : hdone;
        int a = 0;
        for (int j = 0; j < tm.nn; ++j) if (dn[j]) { if (ord == 0) { a = j; break; } --ord; }
        src = (const char*)(isc ? sc.new_csa_kv : sc.new_hca_kv) + ((size_t)b * D + a) * rowb;
      }
      return reinterpret_cast<const uint4*>(src);
    };
    if (cpr == 64) {                                   // d = 512 in bf16: two 16-byte pieces of a row per lane
      for (int r0 = w; r0 < rows_out; r0 += 8 * nw) {
        uint4 v[8][2];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int r = r0 + k * nw;
          const uint4* src = r < rows_out ? row_src(r) : nullptr;
          v[k][0] = src ? __ldg(src + lane) : make_uint4(0, 0, 0, 0);
          v[k][1] = src ? __ldg(src + 32 + lane) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int r = r0 + k * nw;
          if (r < rows_out) { dst[(size_t)r * 64 + lane] = v[k][0]; dst[(size_t)r * 64 + 32 + lane] = v[k][1]; }
        }
      }
    } else {
      for (int r = w; r < rows_out; r += nw) {
        const uint4* src = row_src(r);
        for (int cc = lane; cc < cpr; cc += 32) dst[(size_t)r * cpr + cc] = src ? src[cc] : make_uint4(0, 0, 0, 0);
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
  int32_t* mode = reinterpret_cast<int32_t*>(ws + pl.off_mode) + tix;
  if (tm.status || n0 >= tm.nn) { if (threadIdx.x == 0) { *nkeys = 0; *mode = pl.tc_tma ? 1 : 0; } return; }
  const int nvalid = min(npt, tm.nn - n0);
  const uint32_t validbits = (1u << nvalid) - 1u;
  const int n_csa = tm.n_csa;
  const size_t rowb = (size_t)s.d * 2;
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
  if (GENERAL) while ((256 << psh) < n_csa) ++psh;
  auto phys = [&](int i) { return GENERAL ? i + ((i >> psh) << 2) : i; };
  if (!dense) {
    uint32_t allbits = 0, rankbits = 0;                // nodes that take every committed entry / nodes that rank
    for (int nl = 0; nl < nvalid; ++nl) { if (n_cand[nl] <= s.topk) allbits |= 1u << nl; else rankbits |= 1u << nl; }
    const uint8_t* mrow = reinterpret_cast<const uint8_t*>(ws + pl.off_selmask) + ((size_t)b * D + n0) * pl.mask_ld;
    if (threadIdx.x < 8) {
      // in-tree entries: candidate n_csa + o of a node is the block closed at the o-th of its strict ancestors that closed one
      uint32_t bits = 0;
      const int nl = threadIdx.x;
      if (nl < nvalid && ((rankbits >> nl) & 1u)) {
        int o = 0;
        for (int a = 0; a < n0 + nl; ++a) {
          if (!((tm.anc[n0 + nl] >> a) & 1u) || !cdone[a]) continue;
          const int dblk = (tm.L + tm.depth[a]) / s.m_csa - n_csa;
          if (mrow[(size_t)nl * pl.mask_ld + n_csa + o] && dblk >= 0 && dblk < 32) bits |= 1u << dblk;
          ++o;
        }
      }
      newc_bits[nl] = bits;
    }
    uint32_t* cm32 = reinterpret_cast<uint32_t*>(cmask);
    const uint32_t all4 = 0x01010101u * allbits;
#pragma unroll 2
    for (int i = 16 * threadIdx.x; i < n_csa; i += 16 * blockDim.x) {
      uint32_t acc[4] = {all4, all4, all4, all4};
#pragma unroll
      for (int nl = 0; nl < 8; ++nl) {
        if ((rankbits >> nl) & 1u) {
          const uint4 v = __ldcg(reinterpret_cast<const uint4*>(mrow + (size_t)nl * pl.mask_ld + i));
          acc[0] |= (v.x & 0x01010101u) << nl; acc[1] |= (v.y & 0x01010101u) << nl;
          acc[2] |= (v.z & 0x01010101u) << nl; acc[3] |= (v.w & 0x01010101u) << nl;
        }
      }
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
  if (pl.tc_tma) {
    // the packed per-sequence rows (written by the sequence's extra CTA): few HCA entries, tree nodes, entries closed in the tree
    const int nh_in = tm.n_hca <= kHcaMiscMax ? tm.n_hca : 0;
    int ncd = 0, nhd = 0;
    for (int j = 0; j < tm.nn; ++j) { ncd += cdone[j] != 0; nhd += hdone[j] != 0; }
    const int n_misc = nh_in + tm.nn + ncd + nhd;
    // Ranked nodes still take the contiguous-run path while the run is at most twice the selection size: all committed
    // entries are staged and the unselected ones are masked per node.  Beyond that (or where a paged pool's pages do not
    // hold whole boxes) the tile is GATHERED: the same four runs, but the first holds only the committed entries some node
    // of the tile selected, and every key is named by its row (array << 30 | row) for four-row TMA gathers.
    const bool runs_ok = !GENERAL || ((dense || n_csa <= 2 * s.topk) && csa_runs && (hca_runs || tm.n_hca <= kHcaMiscMax));
    int n_uni = n_csa;                                 // keys of the first run
    __shared__ int uni_tot;
    uint32_t* krow = reinterpret_cast<uint32_t*>(kptr);
    if (!runs_ok) {
      // Ordered compaction of the selected entries: a thread owns `per` consecutive entries, counts its selected ones
      // (four mask bytes per word), one block scan, then writes its rows and masks at consecutive positions.
      __shared__ int wsum_c[9];
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
      int pos = block_excl_scan_256(cnt, wsum_c, total);
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
      for (int k = (runs_ok ? 0 : n_uni) + threadIdx.x; k < kb; k += blockDim.x) {
        const int g = k >= k0[3] ? 3 : (k >= k0[2] ? 2 : (k >= k0[1] ? 1 : 0));
        const int i = k - k0[g];
        uint32_t m = 0;
        if (i < cnt[g]) {
          if (g == 0) m = dense ? validbits : cmask[phys(i)];       // (contiguous-run tiles only: see the loop's start)
          else if (g == 1) m = validbits;
          else if (g == 2) {
            const int pos = c.page_table ? win_a + i : tm.L - 1 - ((tm.L - 1 - i) % s.window);
            for (int nl = 0; nl < nvalid; ++nl) if (pos >= win_lo[nl]) m |= 1u << nl;
          } else if (i < nh_in) m = validbits;
          else if (i < nh_in + tm.nn) {
            const int j = i - nh_in;
            for (int nl = 0; nl < nvalid; ++nl) if ((tm.anc[n0 + nl] >> j) & 1u) m |= 1u << nl;
          } else {
            int ord = i - nh_in - tm.nn;
            const bool isc = ord < ncd;
            if (!isc) ord -= ncd;
            const uint8_t* dn = isc ? cdone : hdone;
            int a = 0;
            for (int j = 0; j < tm.nn; ++j) if (dn[j]) { if (ord == 0) { a = j; break; } --ord; }
            for (int nl = 0; nl < nvalid; ++nl)
              if (a != n0 + nl && ((tm.anc[n0 + nl] >> a) & 1u) && (!isc || newc_selected(nl, a))) m |= 1u << nl;
          }
        }
        kmask[k] = (uint8_t)m;
        // gathered tiles: the key's row; the padding of a run repeats the run's first row (masked)
        if (!runs_ok) krow[k] = ((uint32_t)g << 30) | (uint32_t)(cnt[g] ? run_row(g, i < cnt[g] ? i : 0) : 0);
      }
      if (threadIdx.x == 0) { *nkeys = kb; *mode = runs_ok ? 1 : 2; }
      return;
    }
  }
  if (threadIdx.x == 0) *mode = 0;
  // committed CSA entries, in index order
  // warp w owns a contiguous share of the entries: count its selected ones, exchange the counts once, then write the
  // pointers in index order at positions found with ballots (no block-wide scan per 256 entries: runs are up to 32768 long)
  int base = 0;
  {
    __shared__ int wcnt[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int share = ((n_csa + 7) / 8 + 31) & ~31;
    const int beg = min(n_csa, w * share), end = min(n_csa, beg + share);
    auto mask_of = [&](int i) -> uint32_t { return i < end ? (dense ? validbits : (uint32_t)cmask[phys(i)]) : 0u; };
    int cnt = 0;
    for (int i0 = beg; i0 < end; i0 += 32) cnt += mask_of(i0 + lane) != 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) wcnt[w] = cnt;
    __syncthreads();
    int pos0 = 0, total = 0;
    for (int x = 0; x < 8; ++x) { if (x < w) pos0 += wcnt[x]; total += wcnt[x]; }
    const uint32_t lt = (1u << lane) - 1u;
    for (int i0 = beg; i0 < end; i0 += 32) {
      const int i = i0 + lane;
      const uint32_t m = mask_of(i);
      const uint32_t sel_m = __ballot_sync(0xffffffffu, m != 0);
      if (m) {
        const int pos = pos0 + __popc(sel_m & lt);
        kptr[pos] = (uint64_t)((const char*)c.csa_kv + (size_t)csa_row(i) * rowb); kmask[pos] = (uint8_t)m;
      }
      pos0 += __popc(sel_m);
    }
    base = total;
  }
  // committed HCA entries
  for (int i = threadIdx.x; i < tm.n_hca; i += blockDim.x) {
    kptr[base + i] = (uint64_t)((const char*)c.hca_kv + (size_t)hca_row(i) * rowb); kmask[base + i] = (uint8_t)validbits;
  }
  base += tm.n_hca;
  // committed window positions seen by at least one node of the tile
  int lo = tm.L;
  for (int nl = 0; nl < nvalid; ++nl) lo = min(lo, win_lo[nl]);
  for (int i = threadIdx.x; i < tm.L - lo; i += blockDim.x) {
    const int pos = lo + i;
    uint32_t m = 0;
    for (int nl = 0; nl < nvalid; ++nl) if (pos >= win_lo[nl]) m |= 1u << nl;
    kptr[base + i] = (uint64_t)((const char*)c.win_kv + (size_t)tok_row_of(c, s, b, pos) * rowb); kmask[base + i] = (uint8_t)m;
  }
  base += max(0, tm.L - lo);
  __syncthreads();
  if (threadIdx.x == 0) {
    // tree nodes (ancestors-or-self) and the entries closed inside the tree at strict ancestors
    for (int j = 0; j < tm.nn; ++j) {
      uint32_t mt = 0, mc = 0, mh = 0;
      for (int nl = 0; nl < nvalid; ++nl) {
        const int n = n0 + nl;
        if (!((tm.anc[n] >> j) & 1u)) continue;
        mt |= 1u << nl;
        if (j == n) continue;
        if (hdone[j]) mh |= 1u << nl;
        if (cdone[j]) {
          if (newc_selected(nl, j)) mc |= 1u << nl;        // ranked nodes: is the entry in the node's selection?
        }
      }
      const size_t nrow = (size_t)b * D + j;
      if (mt) { kptr[base] = (uint64_t)((const char*)nd.kv + nrow * rowb); kmask[base++] = (uint8_t)mt; }
      if (mc) { kptr[base] = (uint64_t)((const char*)sc.new_csa_kv + nrow * rowb); kmask[base++] = (uint8_t)mc; }
      if (mh) { kptr[base] = (uint64_t)((const char*)sc.new_hca_kv + nrow * rowb); kmask[base++] = (uint8_t)mh; }
    }
    *nkeys = base;
  }
}

// Plan of every (sequence, 256-row tile).  Each tile CTA leaves one 16-byte record {tile, mode, keys} at the scheduling
// position the selection kernel computed for it (most keys first): the paired attention kernel takes the tiles in that
// order and learns all it needs about its tile from one load.
template <bool GENERAL>
__global__ void __launch_bounds__(256) tc_plan_kernel(const tsv_shape s, const TvaPlan pl, const tsv_cache c, const tsv_nodes nd,
                                                      const tsv_scratch sc, char* __restrict__ ws) {
  extern __shared__ uint8_t cmask_sm[];                // [cand_cap] node bits per committed CSA entry (ranked case only)
  const bool tile_cta = blockIdx.x < (unsigned)pl.tc_nt;
  const size_t tix = (size_t)blockIdx.y * pl.tc_nt + blockIdx.x;
  int pos = (int)tix;                                 // fetched now, used at the end
  if (tile_cta && threadIdx.x == 0) pos = reinterpret_cast<const int32_t*>(ws + pl.off_pos)[tix];   // (when the attention stage runs alone: the previous call's)
  if (threadIdx.x < 2 && tile_cta)                      // finished-chunk counters of the tile's two 128-row halves
    reinterpret_cast<int32_t*>(ws + pl.off_tcnt)[tix * 2 + threadIdx.x] = 0;
  tc_plan_tile<GENERAL>(s, pl, c, nd, sc, ws, cmask_sm);
  if (tile_cta && threadIdx.x == 0) {                 // thread 0 wrote the tile's key count and mode itself
    if (pos < 0 || pos >= s.B * pl.tc_nt) pos = (int)tix;
    reinterpret_cast<int4*>(ws + pl.off_order)[pos] =
        make_int4((int)tix, reinterpret_cast<const int32_t*>(ws + pl.off_mode)[tix], reinterpret_cast<const int32_t*>(ws + pl.off_nkeys)[tix], 0);
  }
}

// ------------------------------------------------------------------------------------------------ attention
namespace tc {

// 16 key-row pointers per thread: keys (tid>>3) + 32 j of the chunk, j = 0..15.  They serve the
// K stages of phase 1 (key tile kt, rows 32 i: j = 8 kt + i) and the V stages of phase 3
// (64-key block kb, rows 32 i: j = 2 kb + i).
struct KeyPtrs { const char* p[16]; uint32_t valid; };

template <int KT>
__device__ __forceinline__ void load_k_stage(const KeyPtrs& kp, uint32_t slot, int dk, int ntk, int tid) {
  const int r0 = tid >> 3, c = tid & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (i * 32 < ntk) {
      const int r = r0 + 32 * i;
      cp16(slot + r * 128 + ((c ^ (r & 7)) << 4), kp.p[8 * KT + i] + dk * 128 + c * 16, (kp.valid >> (8 * KT + i)) & 1u);
    }
  }
}
template <int KB>
__device__ __forceinline__ void load_v_stage(const KeyPtrs& kp, uint32_t slot, int half, int tid) {
  const int r0 = tid >> 3, c = tid & 7;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int r = r0 + 32 * i;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      cp16(slot + j * 8192 + r * 128 + ((c ^ (r & 7)) << 4), kp.p[2 * KB + i] + (half * 4 + j) * 128 + c * 16, (kp.valid >> (2 * KB + i)) & 1u);
  }
}

}  // namespace tc

__global__ void __launch_bounds__(tc::THREADS, 1) tc_attn_kernel(const tsv_shape s, const TvaPlan pl, const tsv_nodes nd, void* __restrict__ out_,
                                                                 char* __restrict__ ws, int32_t* __restrict__ status) {
  using namespace tc;
  extern __shared__ unsigned char smem_raw[];
  const int chunk = blockIdx.x, rt = blockIdx.y, tile = rt >> 1, b = blockIdx.z;     // rt: 128-row tile; tile: its plan tile
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int D = s.D, H = s.H;
  const size_t tix = (size_t)b * pl.tc_nt + tile;
  const size_t rix = (size_t)b * 2 * pl.tc_nt + rt;
  if (reinterpret_cast<const int32_t*>(ws + pl.off_mode)[tix] != 0) return;      // a contiguous-run tile: the TMA kernel's
  const int nk = reinterpret_cast<const int32_t*>(ws + pl.off_nkeys)[tix];
  const int rows_seq = D * H;
  if (rt * BM >= rows_seq) return;                              // second half of a plan tile that ends before it
  const int row0 = rt * BM;                                     // first row of the CTA's tile within the sequence
  bf16* out = reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0) * DH;
  if (nk <= 0) {                                                // flagged sequence or padding-only tile: zeros
    if (chunk == 0)
      for (int i = tid; i < BM * DH / 8; i += THREADS)
        if (row0 + i / (DH / 8) < rows_seq) reinterpret_cast<uint4*>(out)[i] = make_uint4(0, 0, 0, 0);
    return;
  }
  int nch, CL;
  chunking(nk, nch, CL);
  if (chunk >= nch) return;
  const int cbeg = chunk * CL, cend = min(nk, cbeg + CL);

  // ---- shared memory carve-up (tiles need 1024-byte alignment for the 128-byte swizzle)
  unsigned char* base = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Small& sm = *reinterpret_cast<Small*>(base);
  const uint32_t ring = smem_u32(base + SMALL);
  int fail = 0;

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.slot_free[i])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sm.acc_bar)));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // key masks of the chunk and this thread's 16 key-row pointers
  const uint64_t* kptr_g = reinterpret_cast<const uint64_t*>(ws + pl.off_kptr) + tix * pl.tc_maxk;
  const uint8_t* kmask_g = reinterpret_cast<const uint8_t*>(ws + pl.off_kmask) + tix * pl.tc_maxk;
  for (int i = tid; i < NC; i += THREADS) sm.kmask[i] = (cbeg + i < cend) ? kmask_g[cbeg + i] : (uint8_t)0;
  KeyPtrs kp;
  kp.valid = 0;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int key = cbeg + (tid >> 3) + 32 * j;
    const bool v = key < cend;
    kp.p[j] = v ? reinterpret_cast<const char*>(kptr_g[key]) : reinterpret_cast<const char*>(nd.q);
    kp.valid |= (uint32_t)v << j;
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tm = sm.tmem_base;

  // ---- stage stream
  const int nkt = (CL + 255) / 256;                 // key tiles of <= 256 keys
  const int per_dk = 1 + nkt;                       // one Q stage + nkt K stages per 64-wide slice of d
  const int G1 = 8 * per_dk;                        // stages of phase 1
  const int nvs = CL / 64;                          // V stages per half of d
  const int GT = G1 + 2 * nvs;
  const char* qsrc = reinterpret_cast<const char*>(nd.q) + ((size_t)b * rows_seq + row0) * DH * 2;

  auto load_stage = [&](int g) {
    if (g < GT) {
      const uint32_t slot = ring + (uint32_t)(g % NS) * SLOT;
      if (g < G1) {
        const int dk = g / per_dk, r = g % per_dk;
        if (r == 0) {                               // Q slice: 128 rows x 64 dims
          const int r0 = tid >> 3, c = tid & 7;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int row = r0 + 32 * i;
            cp16(slot + row * 128 + ((c ^ (row & 7)) << 4), qsrc + (size_t)row * DH * 2 + dk * 128 + c * 16, row0 + row < rows_seq);
          }
        } else {
          const int kt = r - 1, ntk = min(256, CL - kt * 256);
          if (kt == 0) load_k_stage<0>(kp, slot, dk, ntk, tid); else load_k_stage<1>(kp, slot, dk, ntk, tid);
        }
      } else {
        const int gv = g - G1, half = gv / nvs, kb = gv % nvs;
        switch (kb) {
          case 0: load_v_stage<0>(kp, slot, half, tid); break;
          case 1: load_v_stage<1>(kp, slot, half, tid); break;
          case 2: load_v_stage<2>(kp, slot, half, tid); break;
          case 3: load_v_stage<3>(kp, slot, half, tid); break;
          case 4: load_v_stage<4>(kp, slot, half, tid); break;
          case 5: load_v_stage<5>(kp, slot, half, tid); break;
          case 6: load_v_stage<6>(kp, slot, half, tid); break;
          default: load_v_stage<7>(kp, slot, half, tid); break;
        }
      }
    }
    cp_commit();
  };

  const uint32_t idesc_k256 = make_idesc(256, 0), idesc_k128 = make_idesc(128, 0), idesc_v = make_idesc(256, 1);
  const int q4 = warp & 3, hh = warp >> 2;          // TMEM lane quarter of this warp; column half it works on
  const int row = q4 * 32 + lane;
  const uint32_t tlane = tm + ((uint32_t)(q4 * 32) << 16);
  const uint32_t mybit = 1u << ((rt & 1) * (BM / H) + row / H);
  const float scale2 = s.sm_scale * 1.4426950408889634f;
  float m_row = 0.f, l_row = 0.f;
  uint32_t acc_parity = 0;

  // epilogue of one half of d: O[128 x 256] in TMEM columns 256..511
  auto epilogue = [&](int half) {
    if (!fail && !mbar_wait(&sm.acc_bar, acc_parity)) fail = 1;
    acc_parity ^= 1u;
    fence_after();
    const bool rowok = row0 + row < rows_seq;
    if (nch == 1) {
      const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
      bf16* orow = out + (size_t)row * DH + half * 256 + hh * 128;
#pragma unroll
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tlane + 256 + hh * 128 + c0, r);
        if (rowok) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float f[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) f[t] = __uint_as_float(r[v * 8 + t]) * inv;
            st16(orow + c0 + v * 8, f);
          }
        }
      }
    } else {
      float* po = reinterpret_cast<float*>(ws + pl.off_tpo) + ((rix * pl.tc_chmax + chunk) * BM + row) * DH + half * 256 + hh * 128;
#pragma unroll
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tlane + 256 + hh * 128 + c0, r);
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<float4*>(po + c0 + v * 4) = make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                                                    __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
      }
      if (half == 0 && hh == 0)
        reinterpret_cast<float2*>(ws + pl.off_tpml)[(rix * pl.tc_chmax + chunk) * BM + row] = make_float2(m_row, l_row);
    }
    fence_before();
    __syncthreads();                                 // O columns may be overwritten by the next half
    fence_after();
  };

  // exact softmax of the chunk: S (fp32, columns 0..CL) -> P (bf16 pairs, columns 0..CL/2)
  auto softmax = [&]() {
    if (!fail && !mbar_wait(&sm.acc_bar, acc_parity)) fail = 1;
    acc_parity ^= 1u;
    fence_after();
    const int nblk = CL / 128;
    float mx = -INFINITY;
    for (int e = 0; e < 2; ++e) {
      const int jb = 2 * e + hh;
      if (jb < nblk) {
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tlane + jb * 128 + c0, r);
#pragma unroll
          for (int t = 0; t < 32; ++t)
            if (sm.kmask[jb * 128 + c0 + t] & mybit) mx = fmaxf(mx, __uint_as_float(r[t]));
        }
      }
    }
    sm.xch[hh][row] = mx;
    __syncthreads();
    mx = fmaxf(sm.xch[0][row], sm.xch[1][row]);
    m_row = mx * scale2;                              // scale2 > 0
    const float moff = (mx == -INFINITY) ? 0.f : m_row;
    float sum = 0.f;
    for (int e = 0; e < 2; ++e) {
      const int jb = 2 * e + hh;
      uint32_t pk[64];
      if (jb < nblk) {
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tlane + jb * 128 + c0, r);
#pragma unroll
          for (int t = 0; t < 32; t += 2) {
            const uint32_t mk0 = sm.kmask[jb * 128 + c0 + t] & mybit, mk1 = sm.kmask[jb * 128 + c0 + t + 1] & mybit;
            const float p0 = mk0 ? ex2(fmaf(__uint_as_float(r[t]), scale2, -moff)) : 0.f;
            const float p1 = mk1 ? ex2(fmaf(__uint_as_float(r[t + 1]), scale2, -moff)) : 0.f;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);       // low half = even key
            const float2 back = __bfloat1622float2(h2);
            sum += back.x + back.y;
            pk[(c0 + t) >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        }
      }
      fence_before();
      __syncthreads();                                // every warp has read S blocks 2e and 2e+1
      fence_after();
      if (jb < nblk) {
#pragma unroll
        for (int v = 0; v < 4; ++v) tmem_st16(tlane + jb * 64 + v * 16, pk + v * 16);
      }
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    sm.xch[hh][row] = sum;
    fence_before();
    __syncthreads();
    fence_after();
    l_row = sm.xch[0][row] + sm.xch[1][row];
  };

  // prologue: LOOK stages in flight
  for (int g = 0; g < LOOK; ++g) load_stage(g);

  for (int g = 0; g < GT; ++g) {
    cp_wait<LOOK - 1>();                              // stage g has landed (this thread's copies)
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (g == G1) softmax();                           // S complete -> P in TMEM (also syncs the CTA)
    else if (g == G1 + nvs) epilogue(0);
    fence_before();
    __syncthreads();
    if (tid == 0) {
      fence_after();
      const uint32_t slot = ring + (uint32_t)(g % NS) * SLOT;
      if (g < G1) {
        const int dk = g / per_dk, r = g % per_dk;
        if (r > 0) {
          const int kt = r - 1, ntk = min(256, CL - kt * 256);
          const uint32_t qslot = ring + (uint32_t)((dk * per_dk) % NS) * SLOT;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_ss(tm + kt * 256, make_desc(qslot + ks * 32, 16, 1024), make_desc(slot + ks * 32, 16, 1024),
                   ntk == 256 ? idesc_k256 : idesc_k128, (dk | ks) != 0);
          mma_commit(&sm.slot_free[g % NS]);
          if (r == per_dk - 1) mma_commit(&sm.slot_free[(dk * per_dk) % NS]);        // Q slice no longer needed
          if (g == G1 - 1) mma_commit(&sm.acc_bar);
        }
      } else {
        const int gv = g - G1, kb = gv % nvs;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_ts(tm + 256, tm + kb * 32 + ks * 8, make_desc(slot + ks * 2048, 8192, 1024), idesc_v, (kb | ks) != 0);
        mma_commit(&sm.slot_free[g % NS]);
        if (kb == nvs - 1) mma_commit(&sm.acc_bar);
      }
    }
    // refill the slot of stage g-3 (its release was committed at least two iterations ago) with stage g+LOOK
    const int rs = g - 3;
    if (rs >= 0 && rs + NS < GT) {
      if (!fail && !mbar_wait(&sm.slot_free[rs % NS], (uint32_t)(rs / NS) & 1u)) fail = 1;
    }
    load_stage(g + LOOK);
  }
  epilogue(1);
  cp_wait<0>();
  if (fail && lane == 0) atomicOr(status + b, TSV_ST_INTERNAL);
  fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tm) : "memory");
}

// ------------------------------------------------------------------------------------------------ combine
__global__ void __launch_bounds__(256) tc_combine_kernel(const tsv_shape s, const TvaPlan pl, void* __restrict__ out_, const char* __restrict__ ws) {
  using namespace tc;
  const int rt = blockIdx.x, tile = rt >> 1, b = blockIdx.y;
  const size_t tix = (size_t)b * pl.tc_nt + tile, rix = (size_t)b * 2 * pl.tc_nt + rt;
  const int nk = reinterpret_cast<const int32_t*>(ws + pl.off_nkeys)[tix];
  int nch, CL;
  if (reinterpret_cast<const int32_t*>(ws + pl.off_mode)[tix] != 0) return;     // a tile of the paired kernel
  chunking(nk, nch, CL);
  if (nk <= 0 || nch <= 1) return;
  const int rows_seq = s.D * s.H, row0 = rt * BM;
  bf16* out = reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0) * DH;
  const float* po = reinterpret_cast<const float*>(ws + pl.off_tpo) + rix * pl.tc_chmax * BM * DH;
  const float2* pml = reinterpret_cast<const float2*>(ws + pl.off_tpml) + rix * pl.tc_chmax * BM;
  // grid z splits the tile's 128 rows into groups of 8: a warp merges one row, a lane owns columns 4 (l + 32 k) .. + 3.
  // The chunks are accumulated in order (the result does not depend on the launch shape), four chunks' loads in flight.
  const int lane = threadIdx.x & 31, row = blockIdx.z * 8 + (threadIdx.x >> 5);
  if (row >= BM || row0 + row >= rows_seq) return;
  float m = -INFINITY;
  for (int ch = lane; ch < nch; ch += 32) { const float2 ml = pml[ch * BM + row]; if (ml.y > 0.f) m = fmaxf(m, ml.x); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float l = 0.f;
  float4 acc[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < nch; c0 += 4) {
    float2 ml[4];
    float4 v[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int ch = c0 + u < nch ? c0 + u : nch - 1;
      ml[u] = pml[ch * BM + row];
      const float4* p4 = reinterpret_cast<const float4*>(po + ((size_t)ch * BM + row) * DH);
#pragma unroll
      for (int k = 0; k < 4; ++k) v[u][k] = p4[lane + 32 * k];
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (c0 + u >= nch || !(ml[u].y > 0.f)) continue;
      const float w = exp2f(ml[u].x - m);
      l = fmaf(ml[u].y, w, l);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc[k].x = fmaf(v[u][k].x, w, acc[k].x); acc[k].y = fmaf(v[u][k].y, w, acc[k].y);
        acc[k].z = fmaf(v[u][k].z, w, acc[k].z); acc[k].w = fmaf(v[u][k].w, w, acc[k].w);
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[k].x * inv, acc[k].y * inv), hi = __floats2bfloat162_rn(acc[k].z * inv, acc[k].w * inv);
    uint2 o2;
    o2.x = *reinterpret_cast<const uint32_t*>(&lo); o2.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + (size_t)row * DH + 4 * (lane + 32 * k)) = o2;
  }
}

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

static size_t plan_smem_bytes(const TvaPlan& p) { return p.need_scores ? (((size_t)p.cand_cap + 3) & ~(size_t)3) + 4 * 256 + 16 : 0; }   // node bits per entry, cleared by words (+ the padding words)
// The pointer-gather kernel (and its merge kernel) serves every tile when the caches do not allow TMA (the caller gave no
// row counts of the cache arrays); otherwise all tiles go to the paired kernel.
static bool gather_kernel_needed(bool tma) { return !tma; }
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
  prep.tma = tva_tc_pair_usable(c) ? 1 : 0;
  const size_t plan_sm = plan_smem_bytes(p);
  if (plan_sm > 32 * 1024 && (cudaFuncSetAttribute(tc_plan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_sm) != cudaSuccess ||
                              cudaFuncSetAttribute(tc_plan_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_sm) != cudaSuccess)) {
    cudaGetLastError();
    return TSV_ERR_CUDA;
  }
  if (gather_kernel_needed(prep.tma) &&
      cudaFuncSetAttribute(tc_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES) != cudaSuccess) {
    cudaGetLastError();
    return TSV_ERR_CUDA;
  }
  TSV_PREP(tc_plan_kernel<true>);
  TSV_PREP(tc_plan_kernel<false>);
  TSV_PREP(tc_attn_kernel);
  TSV_PREP(tc_combine_kernel);
  TSV_PREP(tc_combine_pair_kernel);
  if (prep.tma) return prepare_tva_tc_pair(s, p, c, nd, out, ws, prep);
  return TSV_OK;
}

int launch_tva_tc(const tsv_shape& s, const TvaPlan& p_in, const TvaTcPrep& prep, const tsv_cache& c, const tsv_nodes& nd, const tsv_scratch& sc,
                  void* out, char* ws, int32_t* status, cudaStream_t st) {
  TvaPlan p = p_in;
  p.tc_tma = prep.tma;
  const bool gathered = !p.tc_tma || gathered_tiles_possible(s, p, c);
  const dim3 pgrid(p.tc_nt + (p.tc_tma ? 1 : 0), s.B);                                                            // x: tiles (+ the packing CTA)
  if (gathered) tc_plan_kernel<true><<<pgrid, 256, plan_smem_bytes(p), st>>>(s, p, c, nd, sc, ws);
  else tc_plan_kernel<false><<<pgrid, 256, plan_smem_bytes(p), st>>>(s, p, c, nd, sc, ws);
  count_launch();
  if (p.tc_tma) {
    // general: some tile may have more than two chunks of the longest kind, or be gathered; then every multi-chunk tile
    // leaves bf16 partial outputs for the merge kernel
    const bool general = (p.tc_maxk + tc::NCX - 1) / tc::NCX > 2 || gathered;
    const int r = launch_tva_tc_pair(s, p, prep, general, out, ws, status, st);
    if (r != TSV_OK) return r;
    if (general && p.tc_chmax > 1) {
      tc_combine_pair_kernel<<<dim3(2 * p.tc_nt, s.B, tc::BM / 8), 256, 0, st>>>(s, p, out, ws);
      count_launch();
    }
  }
  if (gather_kernel_needed(p.tc_tma)) {
    tc_attn_kernel<<<dim3(p.tc_chmax, 2 * p.tc_nt, s.B), tc::THREADS, tc::SMEM_BYTES, st>>>(s, p, nd, out, ws, status);
    count_launch();
    if (p.tc_chmax > 1) {
      tc_combine_kernel<<<dim3(2 * p.tc_nt, s.B, tc::BM / 8), 256, 0, st>>>(s, p, out, ws);   // z: groups of 8 rows
      count_launch();
    }
  }
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
