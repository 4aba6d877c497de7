// tree_verify_attn, tensor-core kernel for tiles whose key rows form contiguous runs
// (every node of the tile selects all of its CSA candidates: the common short-prefix case).
//
// Same math and the same stage stream as tc_attn_kernel (Q slice | K tiles per 64-wide slice of d,
// then 64-key V stages per half of d), but operands arrive by TMA (cp.async.bulk.tensor, 128-byte
// swizzle, boxes of 32 rows x 64 dims) and the CTA is warp-specialised:
//   warp 0     producer: waits for a free ring slot, arms its mbarrier with the byte count and
//              issues the box copies of the stage (one elected lane)
//   warp 1     MMA issuer: waits for the slot to fill, issues tcgen05.mma, releases the slot
//              with tcgen05.commit (one elected lane)
//   warps 2-9  softmax on S read from TMEM, P written back to TMEM, epilogue of O
// The key list of a tile is a list of boxes {tensor map, first row}; runs are padded to 32 rows
// and the padding rows carry a zero node mask.  No block-wide barrier inside the main loop.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "tc_common.cuh"

namespace tsv {

namespace tma {

using namespace tc;

constexpr int TTHREADS = 320;
constexpr int BOXB = kBoxRows * 128;       // bytes of one box: kBoxRows rows x 128 bytes
constexpr float RESCALE_GAP = 16.f;        // log2 units a later piece's row max may exceed the running reference

struct Ctl {                               // control block at the start of dynamic shared memory
  uint64_t full[NS];
  uint64_t empty[NS];
  uint64_t acc_ev[7];                      // MMA -> compute warps, one barrier per event, each used once:
                                           //   [pc] S of piece pc is complete   [3 + p] part p of O is complete
  uint64_t cmp_ev[6];                      // compute warps -> MMA, one barrier per event, each used once:
                                           //   [pc] P of piece pc is in TMEM   [3 + p] part p of O has been read out
  uint32_t tmem_base;
  int32_t pad;
  uint32_t box[NCX / kBoxRows];            // tensor map id << 30 | first row
  uint8_t kmask[NCX];
  float xch[2][BM];
};
constexpr int CTLB = 3072;                 // control block bytes; the ring follows (needs a 1024-byte aligned base)
constexpr int NSX = 6;                     // ring slots of this kernel; the seventh 32 KiB area stages the output tiles
constexpr int SMEM_X = CTLB + (NSX + 1) * SLOT;
static_assert(sizeof(Ctl) <= CTLB, "control block overflow");

__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

constexpr uint32_t OOB_BOX = 0x3FFFFF00u;   // map 0, a row beyond every tensor: the box is zero-filled

}  // namespace tma

// Stage stream of one chunk (CL keys, pieces of 256 keys, the last one may hold 128):
//   for piece: for dk in 0..7:  [Q slice dk: 128 rows x 64]  [K: piece keys x 64 dims of slice dk]     (S piece += Q K^T)
//   for quarter of d in 0..3: for kb in 0..CL/128-1:  [V: 128 keys x 128 dims]                         (O quarter += P V)
__global__ void __launch_bounds__(tma::TTHREADS, 1)
tc_attn_tma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_csa,
                   const __grid_constant__ CUtensorMap map_hca, const __grid_constant__ CUtensorMap map_win,
                   const __grid_constant__ CUtensorMap map_misc, const __grid_constant__ CUtensorMap map_out, const tsv_shape s, const TvaPlan pl, void* __restrict__ out_,
                   char* __restrict__ ws, int32_t* __restrict__ status) {
  using namespace tma;
  extern __shared__ unsigned char smem_raw[];
  const int chunk = blockIdx.x, tile = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t tix = (size_t)b * pl.tc_nt + tile;
  if (reinterpret_cast<const int32_t*>(ws + pl.off_mode)[tix] != 1) return;      // not a contiguous-run tile
  const int nk = reinterpret_cast<const int32_t*>(ws + pl.off_nkeys)[tix];
  const int rows_seq = s.D * s.H, row0 = tile * BM;
  if (nk <= 0) {                                               // flagged sequence or padding-only tile: zeros
    if (chunk == 0) {
      uint4* o4 = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0) * DH);
      for (int i = tid; i < BM * DH / 8; i += TTHREADS)
        if (row0 + i / (DH / 8) < rows_seq) o4[i] = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  int nch, CL;
  chunking_x(nk, nch, CL);
  if (chunk >= nch) return;
  const int cbeg = chunk * CL, cend = min(nk, cbeg + CL);

  if (smem_u32(smem_raw) & 1023u) {                            // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0) atomicOr(status + b, TSV_ST_INTERNAL);
    return;
  }
  Ctl& sm = *reinterpret_cast<Ctl*>(smem_raw);
  const uint32_t ring = smem_u32(smem_raw + CTLB);

  if (tid == 0) {
    for (int i = 0; i < NSX; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
    for (int i = 0; i < 7; ++i) mbar_init(&sm.acc_ev[i], 1);
    for (int i = 0; i < 6; ++i) mbar_init(&sm.cmp_ev[i], 8);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  {
    const int2* box_g = reinterpret_cast<const int2*>(ws + pl.off_box) + tix * (size_t)(pl.tc_maxk / kBoxRows);
    const uint8_t* kmask_g = reinterpret_cast<const uint8_t*>(ws + pl.off_kmask) + tix * pl.tc_maxk;
    if (tid < NCX / kBoxRows) {
      uint32_t v = OOB_BOX;
      if (cbeg + tid * kBoxRows < cend) { const int2 bx = box_g[cbeg / kBoxRows + tid]; v = ((uint32_t)bx.x << 30) | (uint32_t)bx.y; }
      sm.box[tid] = v;
    }
    for (int i = tid; i < NCX; i += TTHREADS) sm.kmask[i] = (cbeg + i < cend) ? kmask_g[cbeg + i] : (uint8_t)0;
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tm = sm.tmem_base;

  // TMEM columns.  S piece 0 -> [0,256), pieces 1 and 2 -> [256,512) (fp32); P piece pc (bf16 pairs) -> [128 pc, 128 pc + 128).
  // CL <= 512: two pieces at most, O is computed in two halves of 256 columns at [256,512) (N = 256);
  // CL <= 768: three pieces, O in four quarters of 128 columns at [384,512) (N = 128).
  const int npc = (CL + 255) / 256;                 // S pieces
  const int NQ = CL <= 512 ? 2 : 4;                 // parts of d the PV product is computed in
  const int OW = DH / NQ;                           // columns of one part
  const uint32_t OCOL = 512 - OW;
  const int vkeys = 16384 / OW;                     // keys per V stage (32 KiB slot): 64 or 128
  // S stages: pass A covers pieces 0 and 1 (their S columns coexist), pass B piece 2; per pass and 64-wide slice dk of d:
  // one Q stage followed by one K stage per piece of the pass
  const int npA = npc < 2 ? npc : 2, perA = 1 + npA;
  const int GA = 8 * perA;
  const int G1 = GA + (npc > 2 ? 16 : 0);
  const int nvb = CL / vkeys;                       // V stages per part
  const int GT = G1 + NQ * nvb;
  int fail = 0;
#ifdef TSV_TIMELINE
  long long* tl = reinterpret_cast<long long*>(ws);
  const bool tlon = (blockIdx.x == 0 && blockIdx.y == 1 && blockIdx.z == 0);
#define TL(i) do { if (tlon) tl[i] = clock64(); } while (0)
  if (tlon && tid == 0) { tl[0] = clock64(); tl[1] = CL; tl[2] = GT; }
#else
#define TL(i) do { } while (0)
#endif

  // S stage g -> slice dk of d, r (0 = Q stage, else K stage), piece pc of the K stage, index gq of the pass's Q stage for dk
  auto dec = [&](int g, int& dk, int& r, int& pc, int& gq, bool& lastk) {
    if (g < GA) { dk = g / perA; r = g % perA; pc = r - 1; gq = dk * perA; lastk = r == perA - 1; }
    else { const int h = g - GA; dk = h >> 1; r = h & 1; pc = 2; gq = GA + 2 * dk; lastk = r == 1; }
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (lane 0 arms the barrier, lanes 0..7 each copy one box)
    const CUtensorMap* maps[4] = {&map_csa, &map_hca, &map_win, &map_misc};
    for (int g = 0; g < GT; ++g) {
      const int sl = g % NSX, use = g / NSX;
      const uint32_t slot = ring + (uint32_t)sl * SLOT;
      uint64_t* fb = &sm.full[sl];
      int nbox;
      int dk = 0, r = 0, pc = 0, gq = 0; bool lastk = false;
      if (g < G1) { dec(g, dk, r, pc, gq, lastk); nbox = r ? min(256, CL - pc * 256) / kBoxRows : BM / kBoxRows; } else nbox = SLOT / BOXB;
      if (lane == 0) {
        if (use > 0 && !fail && !mbar_wait(&sm.empty[sl], (uint32_t)(use - 1) & 1u)) fail = 1;
        TL(100 + g);
        mbar_expect_tx(fb, nbox * BOXB);
      }
      __syncwarp();
      if (lane < nbox) {
        if (g < G1) {
          if (r == 0) tma_box(slot + lane * BOXB, &map_q, dk * 64, b * rows_seq + row0 + kBoxRows * lane, fb);
          else {
            const uint32_t bx = sm.box[pc * (256 / kBoxRows) + lane];
            tma_box(slot + lane * BOXB, maps[bx >> 30], dk * 64, (int)(bx & 0x3FFFFFFFu), fb);
          }
        } else {
          const int gv = g - G1, part = gv / nvb, kb = gv % nvb;
          if (NQ == 2) {          // 64 keys x 256 dims: boxes (i = key box, j = 64-wide slice 0..3)
            const int i = lane >> 2, j = lane & 3;
            const uint32_t bx = sm.box[kb * (64 / kBoxRows) + i];
            tma_box(slot + j * 8192 + i * BOXB, maps[bx >> 30], (part * 4 + j) * 64, (int)(bx & 0x3FFFFFFFu), fb);
          } else {                // 128 keys x 128 dims: boxes (i = key box, j = slice 0..1)
            const int i = lane >> 1, j = lane & 1;
            const uint32_t bx = sm.box[kb * (128 / kBoxRows) + i];
            tma_box(slot + j * 16384 + i * BOXB, maps[bx >> 30], (part * 2 + j) * 64, (int)(bx & 0x3FFFFFFFu), fb);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_k256 = make_idesc(256, 0), idesc_k128 = make_idesc(128, 0), idesc_v = make_idesc(OW, 1);
      auto need_ev = [&](int e) { if (!fail && !mbar_wait(&sm.cmp_ev[e], 0)) fail = 1; };
      for (int g = 0; g < GT; ++g) {
        const int sl = g % NSX;
        if (!fail && !mbar_wait(&sm.full[sl], (uint32_t)(g / NSX) & 1u)) fail = 1;
        TL(300 + g);
        const uint32_t slot = ring + (uint32_t)sl * SLOT;
        if (g < G1) {
          int dk, r, pc, gq; bool lastk;
          dec(g, dk, r, pc, gq, lastk);
          if (r) {
            const int ntk = min(256, CL - pc * 256);
            if (pc == 2 && dk == 0) need_ev(1);        // piece 2 reuses the S columns of piece 1
            fence_after();
            const int qsl = gq % NSX;
            const uint32_t qslot = ring + (uint32_t)qsl * SLOT;
            const uint32_t scol = tm + (pc == 0 ? 0 : 256);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_ss(scol, make_desc(qslot + ks * 32, 16, 1024), make_desc(slot + ks * 32, 16, 1024),
                     ntk == 256 ? idesc_k256 : idesc_k128, (dk | ks) != 0);
            mma_commit(&sm.empty[sl]);
            if (lastk) {
              mma_commit(&sm.empty[qsl]);                 // the Q slice of this pass and dk is no longer needed
              if (dk == 7) {                              // the S pieces of this pass are complete
                if (g < GA) { mma_commit(&sm.acc_ev[0]); if (npA == 2) mma_commit(&sm.acc_ev[1]); } else mma_commit(&sm.acc_ev[2]);
              }
            }
          }
        } else {
          const int gv = g - G1, part = gv / nvb, kb = gv % nvb;
          if (kb == 0) need_ev(part == 0 ? npc - 1 : 3 + part - 1);   // all of P is in TMEM / the previous part of O has been read out
          fence_after();
          if (NQ == 2) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_ts(tm + OCOL, tm + kb * 32 + ks * 8, make_desc(slot + ks * 2048, 8192, 1024), idesc_v, (kb | ks) != 0);
          } else {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              mma_ts(tm + OCOL, tm + kb * 64 + ks * 8, make_desc(slot + ks * 2048, 16384, 1024), idesc_v, (kb | ks) != 0);
          }
          mma_commit(&sm.empty[sl]);
          if (kb == nvb - 1) mma_commit(&sm.acc_ev[3 + part]);
        }
        TL(500 + g);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (8 warps)
    const int q4 = warp & 3, hh = (warp - 2) >> 2;
    const int row = q4 * 32 + lane;
    const uint32_t tlane = tm + ((uint32_t)(q4 * 32) << 16);
    const uint32_t mybit = 1u << (row / s.H);
    const float scale2 = s.sm_scale * 1.4426950408889634f;
    float m_run = -INFINITY, l_part = 0.f;           // reference max (log2 units); this thread's share of the row sum

    for (int pc = 0; pc < npc; ++pc) {
      if (!fail && !mbar_wait(&sm.acc_ev[pc], 0)) fail = 1;
      fence_after();
      if (warp == 2 && lane == 0) TL(700 + 2 * pc);
      const int pkeys = min(256, CL - pc * 256);
      const bool mine = hh * 128 < pkeys;            // this warp's 128-key block exists in the piece
      const uint32_t scol = tlane + (pc == 0 ? 0 : 256) + hh * 128;   // S block (fp32 columns)
      const int k0 = pc * 256 + hh * 128;                              // first key of the block within the chunk
      // visibility of the block's keys for this lane's row, 32 keys per word (bit t = key c0 + t)
      uint32_t vis[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint32_t mk = mine ? sm.kmask[k0 + c * 32 + lane] : 0u;
        // lanes of a warp may belong to different nodes when H < 32: one ballot per node bit present in the warp
        const uint32_t lo = __shfl_sync(0xffffffffu, mybit, 0), hi = __shfl_sync(0xffffffffu, mybit, 31);
        uint32_t v = __ballot_sync(0xffffffffu, mk & mybit);
        if (lo != hi) {
          v = 0;
          for (uint32_t bit = lo; bit <= hi; bit <<= 1) { const uint32_t w = __ballot_sync(0xffffffffu, mk & bit); if (bit == mybit) v = w; }
        }
        vis[c] = v;
      }
      float mx = -INFINITY;
      if (mine) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld32(scol + c * 32, r);
          if (vis[c] == 0xffffffffu) {
#pragma unroll
            for (int t = 0; t < 32; ++t) mx = fmaxf(mx, __uint_as_float(r[t]));
          } else {
#pragma unroll
            for (int t = 0; t < 32; ++t) if ((vis[c] >> t) & 1u) mx = fmaxf(mx, __uint_as_float(r[t]));
          }
        }
      }
      sm.xch[hh][row] = mx;
      compute_sync();
      const float m_piece = fmaxf(sm.xch[0][row], sm.xch[1][row]) * scale2;
      // Keep one reference max per row.  A later piece may exceed it by up to RESCALE_GAP (weights up to 2^16 are
      // harmless in bf16/fp32); beyond that the P written so far and the running sum are rescaled.
      float factor = 1.f;
      if (m_piece > m_run + RESCALE_GAP || m_run == -INFINITY) {
        if (m_run != -INFINITY) factor = ex2(m_run - m_piece);
        m_run = m_piece;
      }
      if (__any_sync(0xffffffffu, factor != 1.f)) {  // warp-uniform: tcgen05.ld/st are warp-collective
        for (int pj = 0; pj < pc; ++pj) {
          const uint32_t pcol = tlane + pj * 128 + hh * 64;
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t r[32];
            tmem_ld32(pcol + v * 32, r);
#pragma unroll
            for (int t = 0; t < 32; ++t) {
              float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r[t]));
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(f.x * factor, f.y * factor);
              r[t] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            tmem_st16(pcol + v * 32, r);
            tmem_st16(pcol + v * 32 + 16, r + 16);
          }
        }
        l_part *= factor;
      }
      const float moff = (m_run == -INFINITY) ? 0.f : m_run;
      uint32_t pk[64];
      if (mine) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld32(scol + c * 32, r);
          if (vis[c] == 0xffffffffu) {
#pragma unroll
            for (int t = 0; t < 32; t += 2) {
              const float p0 = ex2(fmaf(__uint_as_float(r[t]), scale2, -moff));
              const float p1 = ex2(fmaf(__uint_as_float(r[t + 1]), scale2, -moff));
              l_part += p0 + p1;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);     // low half = even key
              pk[(c * 32 + t) >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
            }
          } else {
#pragma unroll
            for (int t = 0; t < 32; t += 2) {
              const float p0 = ((vis[c] >> t) & 1u) ? ex2(fmaf(__uint_as_float(r[t]), scale2, -moff)) : 0.f;
              const float p1 = ((vis[c] >> (t + 1)) & 1u) ? ex2(fmaf(__uint_as_float(r[t + 1]), scale2, -moff)) : 0.f;
              l_part += p0 + p1;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
              pk[(c * 32 + t) >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
            }
          }
        }
      }
      fence_before();
      compute_sync();                                // both S blocks of the piece have been read by every warp
      fence_after();
      if (mine) {
#pragma unroll
        for (int v = 0; v < 4; ++v) tmem_st16(tlane + pc * 128 + hh * 64 + v * 16, pk + v * 16);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.cmp_ev[pc]);    // this piece's P is in TMEM; its S columns may be reused
      if (warp == 2 && lane == 0) TL(701 + 2 * pc);
    }
    sm.xch[hh][row] = l_part;
    compute_sync();
    const float l_row = sm.xch[0][row] + sm.xch[1][row];

    const bool rowok = row0 + row < rows_seq;
    const bool full_tile = row0 + BM <= rows_seq;     // whole tile inside the sequence: rows may be stored as 32-row boxes
    const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
    const int cw = OW / 2;                            // columns of the part this thread handles: 128 or 64
    const uint32_t stage = ring + (uint32_t)NSX * SLOT + (uint32_t)(warp - 2) * 4096;   // this warp's 32 rows x 64 columns (bf16)
    bool store_pending = false;
    for (int part = 0; part < NQ; ++part) {
      if (!fail && !mbar_wait(&sm.acc_ev[3 + part], 0)) fail = 1;
      fence_after();
      if (warp == 2 && lane == 0) TL(720 + 2 * part);
      for (int c0 = 0; c0 < cw; c0 += 64) {
        uint32_t r0[32], r1[32];
        tmem_ld32(tlane + OCOL + hh * cw + c0, r0);
        tmem_ld32(tlane + OCOL + hh * cw + c0 + 32, r1);
        if (c0 + 64 >= cw && part < NQ - 1) {         // last columns are in registers: the MMA may overwrite this part
          fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.cmp_ev[3 + part]);
        }
        const int col = part * OW + hh * cw + c0;
        if (nch == 1 && full_tile) {
          // stage the 32 x 64 bf16 tile in the 128-byte swizzle pattern and store it with one TMA request
          if (store_pending) {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
          }
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            const uint32_t* src = v < 4 ? r0 + v * 8 : r1 + (v - 4) * 8;
            uint32_t w[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(src[2 * t]) * inv, __uint_as_float(src[2 * t + 1]) * inv);
              w[t] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage + lane * 128 + ((v ^ (lane & 7)) << 4)), "r"(w[0]), "r"(w[1]),
                         "r"(w[2]), "r"(w[3]) : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(col), "r"(b * rows_seq + row0 + q4 * 32), "r"(stage) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          store_pending = true;
        } else if (nch == 1) {
          if (rowok) {
            bf16* orow = reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0 + row) * DH + col;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              float f[8];
#pragma unroll
              for (int t = 0; t < 8; ++t) f[t] = __uint_as_float(r0[v * 8 + t]) * inv;
              st16(orow + v * 8, f);
#pragma unroll
              for (int t = 0; t < 8; ++t) f[t] = __uint_as_float(r1[v * 8 + t]) * inv;
              st16(orow + 32 + v * 8, f);
            }
          }
        } else {
          float* po = reinterpret_cast<float*>(ws + pl.off_tpo) + ((tix * pl.tc_chmax + chunk) * BM + row) * DH + col;
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            *reinterpret_cast<float4*>(po + v * 4) = make_float4(__uint_as_float(r0[v * 4]), __uint_as_float(r0[v * 4 + 1]),
                                                                 __uint_as_float(r0[v * 4 + 2]), __uint_as_float(r0[v * 4 + 3]));
            *reinterpret_cast<float4*>(po + 32 + v * 4) = make_float4(__uint_as_float(r1[v * 4]), __uint_as_float(r1[v * 4 + 1]),
                                                                      __uint_as_float(r1[v * 4 + 2]), __uint_as_float(r1[v * 4 + 3]));
          }
        }
      }
      if (nch > 1 && part == 0 && hh == 0)
        reinterpret_cast<float2*>(ws + pl.off_tpml)[(tix * pl.tc_chmax + chunk) * BM + row] = make_float2(m_run, l_row);
    }
    if (store_pending && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
  if (warp == 2 && lane == 0) TL(740);
  if (fail) atomicOr(status + b, TSV_ST_INTERNAL);
  fence_before();
  __syncthreads();
  if (tid == 0) TL(741);
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tm) : "memory");
}

// ------------------------------------------------------------------------------------------------ host side
static PFN_cuTensorMapEncodeTiled encode_fn() {
  static PFN_cuTensorMapEncodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(p);
  }
  return fn;
}

// rows x 512 bf16, row-major; boxes of 32 rows x 64 columns written with the 128-byte swizzle
static bool make_map(CUtensorMap* m, const void* basep, int64_t rows, int box_rows = kBoxRows) {
  PFN_cuTensorMapEncodeTiled fn = encode_fn();
  if (!fn || rows <= 0 || ((uintptr_t)basep & 15)) return false;
  const cuuint64_t gdim[2] = {(cuuint64_t)tc::DH, (cuuint64_t)rows};
  const cuuint64_t gstr[1] = {(cuuint64_t)tc::DH * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(basep), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tva_tc_tma_usable(const tsv_cache& c) { return c.csa_rows > 0 && c.hca_rows > 0 && encode_fn() != nullptr; }

int launch_tva_tc_tma(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, void* out, char* ws,
                      int32_t* status, cudaStream_t st) {
  CUtensorMap mq, mc, mh, mw, mm, mo;
  if (!make_map(&mq, nd.q, (int64_t)s.B * s.D * s.H) || !make_map(&mc, c.csa_kv, c.csa_rows) || !make_map(&mh, c.hca_kv, c.hca_rows) ||
      !make_map(&mw, c.win_kv, (int64_t)s.B * s.window) || !make_map(&mm, ws + p.off_misc, (int64_t)s.B * p.tc_misc_rows) ||
      !make_map(&mo, out, (int64_t)s.B * s.D * s.H, 32))
    return TSV_ERR_CUDA;
  if (cudaFuncSetAttribute(tc_attn_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tma::SMEM_X) != cudaSuccess) return TSV_ERR_CUDA;
  TSV_PREP(tc_attn_tma_kernel);
  tc_attn_tma_kernel<<<dim3(p.tc_chmax, p.tc_nt, s.B), tma::TTHREADS, tma::SMEM_X, st>>>(mq, mc, mh, mw, mm, mo, s, p, out, ws, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
