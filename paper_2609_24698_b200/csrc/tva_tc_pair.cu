// tree_verify_attn, tensor-core kernel run by PAIRS of CTAs (thread-block cluster of 2, tcgen05 cta_group::2), for key
// lists made of contiguous runs (fetched as TMA boxes) and for key lists of scattered rows (fetched four rows at a
// time by TMA gather).
//
// A pair covers 256 query rows of one sequence (256/H consecutive tree nodes x H heads); each CTA owns
// 128 of them in its own tensor memory.  The two SMs execute every MMA together (M = 256): the B operand
// -- the staged key rows -- is split between the two shared memories, so each SM fetches only HALF of
// the K tile (S = Q K^T: half of the keys) and half of the V tile (O = P K: half of the columns of d).
// That halves the bytes each SM pulls from L2.
//   warps 0, 10  producers: TMA boxes (cp.async.bulk.tensor, 128-byte swizzle) into 16 KiB slots; the copies of BOTH
//                CTAs complete on the mbarriers of the leader (rank 0) CTA
//   warp 1       MMA issuer (leader CTA only): tcgen05.mma.cta_group::2, slot release and accumulator
//                events by tcgen05.commit multicast to both CTAs
//   warps 2-9    softmax on the CTA's own S rows (TMEM), P written back to TMEM, epilogue of O through
//                swizzled shared-memory tiles and TMA stores; events to the leader's MMA warp by remote arrive
// Stage stream, TMEM column plan, running-max rule and chunking are those described at the kernel.
#include <cuda.h>
#include <stdio.h>
#include <cudaTypedefs.h>

#include "tc_common.cuh"

namespace tsv {

namespace pair {

using namespace tc;

constexpr int NPROD = 2;                    // producer warps: warp 0 and warp 10
constexpr int TTHREADS = 32 * (10 + NPROD - 1);   // warp 1: MMA issuer; warps 2-9: softmax and epilogue
constexpr int BOXB = kBoxRows * 128;       // bytes of one box: kBoxRows rows x 128 bytes
constexpr float RESCALE_GAP = 16.f;        // log2 units a later piece's row max may exceed the running reference

constexpr int NSX = 12;                    // 16 KiB slots of the staging area; a 32 KiB area after it stages the output tiles
constexpr int NQS = 8;                     // S phase: slots [0, 8) hold the Q slices (all of d, resident for every piece),
constexpr int NKS = NSX - NQS + 2;         //          slots [8, 14) are the ring of the K stages: the last two are the
                                           //          output staging area, idle until the first part of O is read out;
                                           // V phase: slots [0, 12) form the ring of the V stages

struct Ctl {                               // control block at the start of dynamic shared memory
  uint64_t fullQ[NQS];                     // Q slice dk has arrived (used once)
  uint64_t fullK[NKS], emptyK[NKS];        // ring of the K stages
  uint64_t fullV[NSX], emptyV[NSX];        // ring of the V stages (starts when the S products are complete)
  uint64_t acc_ev[7];                      // MMA -> other warps, one barrier per event, each used once:
                                           //   [pc] S of piece pc is complete   [3 + p] part p of O is complete
  uint64_t cmp_ev[6];                      // compute warps -> MMA, one barrier per event, each used once:
                                           //   [pc] P of piece pc is in TMEM   [3 + p] part p of O has been read out
  uint32_t tmem_base;
  int32_t merge_here;                      // set for the CTA that finished a multi-chunk tile last
  uint32_t box[NCX / kBoxRows];            // tensor map id << 30 | first row
  uint8_t kmask[NCX];
  float xch[2][BM];
};
constexpr int CTLB = 3072;                 // control block bytes; the ring follows (needs a 1024-byte aligned base)
constexpr int SLOTP = 16384;               // ring slot: every stage of a CTA is at most 16 KiB
constexpr int SMEM_X = CTLB + NSX * SLOTP + 32768;
static_assert(sizeof(Ctl) <= CTLB, "control block overflow");

__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
// shared::cluster address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA box copy into this CTA's shared memory; completion is counted on an mbarrier given by its cluster address
__device__ __forceinline__ void tma_box2(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
// four rows of a 2D tensor, given by their row indices, as four consecutive 128-byte lines of this CTA's shared memory
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* map, int x, const uint4& code, uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"((int)(code.x & 0x3FFFFFFFu)), "r"((int)(code.y & 0x3FFFFFFFu)),
                 "r"((int)(code.z & 0x3FFFFFFFu)), "r"((int)(code.w & 0x3FFFFFFFu)), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
// arrives on the same barrier (same shared-memory offset) in both CTAs of the pair once all prior MMAs have completed
__device__ __forceinline__ void mma2_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ uint32_t make_idesc2(int N, int b_mn_major) {      // M = 256 over the pair
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the two halves of the pair-wide barrier, for work that does not depend on the peer in between
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Tensor maps of one call: every source array with boxes of 32, 64 and 128 rows (64 columns, 128-byte swizzle), so that
// a stage whose key rows are consecutive rows of one array is fetched by ONE large request.
struct alignas(64) MapSet {
  CUtensorMap q;          // 128-row boxes
  CUtensorMap out;        // 32-row boxes (stores)
  CUtensorMap src[4][3];  // [csa, hca, window, packed misc][32, 64, 128 rows]
  CUtensorMap row[4];     // the same arrays with one-row boxes: gathers of four rows by index
  CUtensorMap part;       // normalised partial outputs of tiles of more than two chunks (bf16, 32-row boxes, stores)
};
constexpr int NMAPS = 19;

constexpr uint32_t OOB_BOX = 0x3FFFFF00u;   // map 0, a row beyond every tensor: the box is zero-filled

}  // namespace pair

// Per CTA (rank r of the pair), for a chunk of CL keys (pieces of 256 keys, the last may hold 128):
//   Q slices:  per 64-wide slice dk of d  [this CTA's 128 rows x 64 dims], fetched once, resident for all pieces
//   K stages:  piece after piece, per slice dk  [this CTA's half of the piece's keys x 64 dims]
//   V stages (after the last S product): CL <= 512: per half of d, per 64 keys:  [64 keys x this CTA's 128 of the half's 256 dims]
//                                        else       per quarter of d, per 128 keys: [128 keys x this CTA's 64 of the quarter's 128 dims]
//
// GENERAL: gathered tiles and tiles of more than two chunks may occur.  Shapes whose capacities rule both out (the
// benchmark's) run the instantiation without that code: the kernel is one long dependency chain per tile and its
// timing follows the code layout.
template <bool GENERAL>
__global__ void __launch_bounds__(pair::TTHREADS, 1)
tc_attn_pair_kernel(const __grid_constant__ pair::MapSet maps, const tsv_shape s,
                    const TvaPlan pl, void* __restrict__ out_, char* __restrict__ ws, int32_t* __restrict__ status) {
  using namespace pair;
  extern __shared__ unsigned char smem_raw[];
  // the two CTAs of a pair are neighbours in x; pairs take the (sequence, tile) items in the order the plan kernel left
  // (most keys first)
  const int chunk = blockIdx.y;
  // launched as a programmatic dependent of the tile plan: the CTAs take their places while that kernel's last CTAs
  // finish, and read nothing before it has completed
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int4 rec = reinterpret_cast<const int4*>(ws + pl.off_order)[blockIdx.x >> 1];   // {tile index, mode, keys, -}: one load
  const int item = rec.x;
  const int b = item / pl.tc_nt, tile = item % pl.tc_nt;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const size_t tix = (size_t)b * pl.tc_nt + tile;
  if (tid < (GENERAL ? NMAPS : 14))   // the descriptors of the tensor maps in use are fetched while the plan is read
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps) + (uint64_t)tid * sizeof(CUtensorMap)) : "memory");
  const size_t rix = (size_t)b * 2 * pl.tc_nt + 2 * tile + rank;  // this CTA's 128-row tile (partials of multi-chunk tiles)
  // every exit below is taken by both CTAs of the pair alike (it depends on the pair's plan only)
  if (rec.y != 1 && !(GENERAL && rec.y == 2)) return;          // neither a contiguous-run tile nor a gathered one
  const bool gather = GENERAL && rec.y == 2;                              // the key list is a list of row codes (array << 30 | row), not of boxes
  const int nk = rec.z;
  const int rows_seq = s.D * s.H, row0 = tile * PR + (int)rank * BM;           // first of this CTA's rows within the sequence
  if (nk <= 0) {                                               // flagged sequence or padding-only tile: zeros
    if (chunk == 0) {
      uint4* o4 = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0) * DH);
      for (int i = tid; i < BM * DH / 8; i += TTHREADS)
        if (row0 + i / (DH / 8) < rows_seq) o4[i] = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  int nch, CL;
  chunking_x(nk, GENERAL, nch, CL);
  if (chunk >= nch) return;
  const int cbeg = chunk * CL, cend = min(nk, cbeg + CL);

  Ctl& sm = *reinterpret_cast<Ctl*>(smem_raw);
  const uint32_t ring = smem_u32(smem_raw + CTLB);
  int fail = (smem_u32(smem_raw) & 1023u) ? 1 : 0;             // the swizzled tiles need a 1024-byte aligned base

  if (tid == 0) {
    for (int i = 0; i < NQS; ++i) mbar_init(&sm.fullQ[i], 1);
    for (int i = 0; i < NKS; ++i) { mbar_init(&sm.fullK[i], 1); mbar_init(&sm.emptyK[i], 1); }
    for (int i = 0; i < NSX; ++i) { mbar_init(&sm.fullV[i], 1); mbar_init(&sm.emptyV[i], 1); }
    for (int i = 0; i < 7; ++i) mbar_init(&sm.acc_ev[i], 1);
    for (int i = 0; i < 6; ++i) mbar_init(&sm.cmp_ev[i], 16);   // 8 compute warps of each CTA
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  // Pair-wide barrier, first half: this CTA's barriers exist and its tensor memory is allocated (thread 0 and warp 0 arrive
  // after doing that).  The plan's boxes and key masks are read while the peer gets there; the wait follows below.
  __syncwarp();
  cluster_arrive();
  {
    const int2* box_g = reinterpret_cast<const int2*>(ws + pl.off_box) + tix * (size_t)(pl.tc_maxk / kBoxRows);
    const uint8_t* kmask_g = reinterpret_cast<const uint8_t*>(ws + pl.off_kmask) + tix * pl.tc_maxk;
    if (tid < NCX / kBoxRows && !gather) {
      uint32_t v = OOB_BOX;
      if (cbeg + tid * kBoxRows < cend) { const int2 bx = box_g[cbeg / kBoxRows + tid]; v = ((uint32_t)bx.x << 30) | (uint32_t)bx.y; }
      sm.box[tid] = v;
    }
    for (int i = tid; i < NCX; i += TTHREADS) sm.kmask[i] = (cbeg + i < cend) ? kmask_g[cbeg + i] : (uint8_t)0;
  }
  fence_before();
  __syncthreads();
  cluster_wait();                                                // barriers of both CTAs exist before anyone signals them
  fence_after();
  const uint32_t tm = sm.tmem_base;

  // TMEM columns (per CTA, its own 128 rows).  S piece 0 -> [0,256), pieces 1 and 2 -> [256,512) (fp32);
  // P piece pc (bf16 pairs) -> [128 pc, 128 pc + 128).  CL <= 512: O in two halves of 256 columns at [256,512);
  // CL <= 768: O in four quarters of 128 columns at [384,512).
  const int npc = (CL + 255) / 256;                 // S pieces
  const int NQ = CL <= 512 ? 2 : 4;                 // parts of d the PV product is computed in
  const int OW = DH / NQ;                           // columns of one part
  const uint32_t OCOL = 512 - OW;
  const int vkeys = 16384 / OW;                     // keys per V stage: 64 or 128
  const int nvb = CL / vkeys;                       // V stages per part
  const int NKST = 8 * npc;                         // K stages: piece after piece, per piece the eight 64-wide slices of d
  const int NVST = NQ * nvb;                        // V stages

  if (warp == 0 || warp >= 10) {
    // ------------------------------------------------------------------ producers (both CTAs): stage g is issued by producer g % NPROD
    const int pw = warp == 0 ? 0 : warp - 9;
    // consecutive: do the nb boxes starting at list index i0 name consecutive rows of one array?
    auto consecutive = [&](int i0, int nb) {
      const uint32_t b0 = sm.box[i0];
      if ((b0 & 0x3FFFFFFFu) >= (OOB_BOX & 0x3FFFFFFFu)) return false;
      for (int i = 1; i < nb; ++i) if (sm.box[i0 + i] != b0 + (uint32_t)(i * kBoxRows)) return false;
      return true;
    };
    // Q slices: producer 0.  K stage gk = 8 pc + dk: producer (gk + 1) & 1, so that the first K stage leaves at the same
    // time as the first Q slice.  V stage gv: producer gv & 1.  Both CTAs' copies complete on the leader's barriers.
    auto issue_q = [&](int dk) {
      if (lane == 0) {
        if (rank == 0) mbar_expect_tx(&sm.fullQ[dk], 2 * SLOTP);
        tma_box2(ring + (uint32_t)dk * SLOTP, &maps.q, dk * 64, b * rows_seq + row0, map_to_rank(smem_u32(&sm.fullQ[dk]), 0));
      }
      __syncwarp();
    };
    // Gathered tiles: the keys' row codes stay in global memory (the tile plan left them there, four-aligned groups
    // never mix arrays); lane l fetches the codes of rows 4 l .. 4 l + 3 of a stage itself.  Keys past the end of the list
    // read row 0 of the first array (they are masked).
    const uint4* code_g = reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(ws + pl.off_krow) + tix * (size_t)pl.tc_maxk + cbeg);
    auto codes_at = [&](int key) { return cbeg + key < cend ? __ldg(code_g + (key >> 2)) : make_uint4(0u, 0u, 0u, 0u); };
    uint4 kcode = make_uint4(0u, 0u, 0u, 0u);                                // this lane's codes of the current piece's K stages
    int kcode_pc = -1;
    auto issue_k = [&](int gk) {
      const int pc = gk >> 3, dk = gk & 7, sl = gk % NKS, use = gk / NKS;
      const uint32_t slot = ring + (uint32_t)(NQS + sl) * SLOTP;
      const uint32_t fb_leader = map_to_rank(smem_u32(&sm.fullK[sl]), 0);
      const int bytes = min(256, CL - pc * 256) * 64;                        // bytes THIS CTA copies in the stage
      if (gather && kcode_pc != pc) {                                        // this CTA's half of the piece's keys: bytes / 128 rows
        kcode_pc = pc;
        if (lane * 512 < bytes) kcode = codes_at(pc * 256 + (int)rank * (bytes >> 7) + 4 * lane);
      }
      if (lane == 0) {
        if (use > 0 && !fail && !mbar_wait(&sm.emptyK[sl], (uint32_t)(use - 1) & 1u)) fail = 1;
        if (rank == 0) mbar_expect_tx(&sm.fullK[sl], 2 * bytes);              // bytes of both CTAs
      }
      __syncwarp();
      // this CTA's half of the piece's keys: boxes [rank * nb, rank * nb + nb) of the piece
      const int nb = bytes / BOXB, i0 = pc * (256 / kBoxRows) + (int)rank * nb;
      if (gather) {
        if (lane * 512 < bytes) tma_gather4(slot + lane * 512, &maps.row[kcode.x >> 30], dk * 64, kcode, fb_leader);
      } else if (consecutive(i0, nb)) {                                             // nb = 4 (128 rows) or 2 (64 rows)
        if (lane == 0) { const uint32_t bx = sm.box[i0]; tma_box2(slot, &maps.src[bx >> 30][nb == 4 ? 2 : 1], dk * 64, (int)(bx & 0x3FFFFFFFu), fb_leader); }
      } else if (lane < nb) {
        const uint32_t bx = sm.box[i0 + lane];
        tma_box2(slot + lane * BOXB, &maps.src[bx >> 30][0], dk * 64, (int)(bx & 0x3FFFFFFFu), fb_leader);
      }
      __syncwarp();
    };
    if (pw == 0) {
      for (int i = 0; i < 4; ++i) { issue_q(2 * i); issue_q(2 * i + 1); issue_k(2 * i + 1); }
      for (int gk = 9; gk < NKST; gk += 2) issue_k(gk);
    } else {
      for (int gk = 0; gk < NKST; gk += 2) issue_k(gk);
    }
    // V stages reuse the whole staging area: they start when the last S product is complete (the softmax of the last
    // piece is still to come, so the ring is full by the time the PV products start)
    if (lane == 0 && !fail && !mbar_wait(&sm.acc_ev[npc - 1], 0)) fail = 1;
    __syncwarp();
    {
      int part = 0, kb = pw;
      while (kb >= nvb) { kb -= nvb; ++part; }
      for (int gv = pw; gv < NVST; gv += NPROD) {
        const int sl = gv % NSX, use = gv / NSX;
        const uint32_t slot = ring + (uint32_t)sl * SLOTP;
        const uint32_t fb_leader = map_to_rank(smem_u32(&sm.fullV[sl]), 0);
        uint4 vcode = make_uint4(0u, 0u, 0u, 0u);                 // (fetched before the wait for the slot)
        if (gather) vcode = codes_at(NQ == 2 ? kb * 64 + 4 * (lane & 15) : kb * 128 + 4 * lane);
        if (lane == 0) {
          if (use > 0 && !fail && !mbar_wait(&sm.emptyV[sl], (uint32_t)(use - 1) & 1u)) fail = 1;
          if (rank == 0) mbar_expect_tx(&sm.fullV[sl], 2 * SLOTP);
        }
        __syncwarp();
        if (gather) {             // NQ == 2: 16 row groups x 2 slices of 64 dims; else 32 row groups x this CTA's 64 dims
          if (NQ == 2) tma_gather4(slot + (lane >> 4) * 8192 + (lane & 15) * 512, &maps.row[vcode.x >> 30], (part * 4 + (int)rank * 2 + (lane >> 4)) * 64, vcode, fb_leader);
          else tma_gather4(slot + lane * 512, &maps.row[vcode.x >> 30], (part * 2 + (int)rank) * 64, vcode, fb_leader);
        } else if (NQ == 2) {     // 64 keys x this CTA's 128 dims: key boxes i = 0..1, 64-wide slices j = 0..1
          const int i0 = kb * (64 / kBoxRows);
          if (consecutive(i0, 2)) {
            if (lane < 2) { const uint32_t bx = sm.box[i0]; tma_box2(slot + lane * 8192, &maps.src[bx >> 30][1], (part * 4 + (int)rank * 2 + lane) * 64, (int)(bx & 0x3FFFFFFFu), fb_leader); }
          } else if (lane < 4) {
            const int i = lane >> 1, j = lane & 1;
            const uint32_t bx = sm.box[i0 + i];
            tma_box2(slot + j * 8192 + i * BOXB, &maps.src[bx >> 30][0], (part * 4 + (int)rank * 2 + j) * 64, (int)(bx & 0x3FFFFFFFu), fb_leader);
          }
        } else {                  // 128 keys x this CTA's 64 dims: key boxes 0..3
          const int i0 = kb * (128 / kBoxRows);
          if (consecutive(i0, 4)) {
            if (lane == 0) { const uint32_t bx = sm.box[i0]; tma_box2(slot, &maps.src[bx >> 30][2], (part * 2 + (int)rank) * 64, (int)(bx & 0x3FFFFFFFu), fb_leader); }
          } else if (lane < 4) {
            const uint32_t bx = sm.box[i0 + lane];
            tma_box2(slot + lane * BOXB, &maps.src[bx >> 30][0], (part * 2 + (int)rank) * 64, (int)(bx & 0x3FFFFFFFu), fb_leader);
          }
        }
        kb += NPROD;
        while (kb >= nvb) { kb -= nvb; ++part; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc_k256 = make_idesc2(256, 0), idesc_k128 = make_idesc2(128, 0), idesc_v = make_idesc2(OW, 1);
      auto need_ev = [&](int e) { if (!fail && !mbar_wait(&sm.cmp_ev[e], 0)) fail = 1; };
      // The issuing thread is the pacemaker of the tensor pipe: stages are walked with counters (no divisions), and the
      // descriptors of a stage are the slot-0 descriptor plus a multiple of the slot size (the address field counts
      // 16-byte units and cannot overflow within the ring).
      const uint64_t dk0 = make_desc(ring, 16, 1024), dv0 = make_desc(ring, NQ == 2 ? 8192 : 16384, 1024);
      // S, piece after piece (the softmax of a piece runs while the tensor core works on the next one): per piece the
      // eight slices of d, Q slice from its resident slot, K stage from the ring
      int sl = 0; uint32_t kph = 0;                      // slot and parity of the next K stage
      for (int pc = 0; pc < npc; ++pc) {
        if (pc == 2) need_ev(1);                         // piece 2 reuses the S columns of piece 1
        const uint32_t scol = tm + (pc == 0 ? 0 : 256);
        const uint32_t idesc = CL - pc * 256 >= 256 ? idesc_k256 : idesc_k128;
        for (int dk = 0; dk < 8; ++dk) {
          if (pc == 0 && !fail && !mbar_wait(&sm.fullQ[dk], 0)) fail = 1;
          if (!fail && !mbar_wait(&sm.fullK[sl], kph)) fail = 1;
          fence_after();
          const uint64_t qd = dk0 + (uint64_t)(dk * (SLOTP >> 4)), kd = dk0 + (uint64_t)((NQS + sl) * (SLOTP >> 4));
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) mma2_ss(scol, qd + 2 * ks, kd + 2 * ks, idesc, (dk | ks) != 0);
          mma2_commit(&sm.emptyK[sl]);
          if (++sl == NKS) { sl = 0; kph ^= 1u; }
        }
        mma2_commit(&sm.acc_ev[pc]);                     // S of the piece is complete
      }
      sl = 0;
      uint32_t ph = 0;                                   // slot and parity of the next V stage
      for (int part = 0; part < NQ; ++part) {
        need_ev(part == 0 ? npc - 1 : 3 + part - 1);     // all of P is in TMEM / the previous part of O has been read out
        for (int kb = 0; kb < nvb; ++kb) {
          if (!fail && !mbar_wait(&sm.fullV[sl], ph)) fail = 1;
          fence_after();
          const uint64_t vd = dv0 + (uint64_t)(sl * (SLOTP >> 4));
          if (NQ == 2) {          // per CTA: 64 keys x 128 dims = two [64 x 64] tiles
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) mma2_ts(tm + OCOL, tm + kb * 32 + ks * 8, vd + ks * (2048 >> 4), idesc_v, (kb | ks) != 0);
          } else {                // per CTA: 128 keys x 64 dims = one [128 x 64] tile
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) mma2_ts(tm + OCOL, tm + kb * 64 + ks * 8, vd + ks * (2048 >> 4), idesc_v, (kb | ks) != 0);
          }
          mma2_commit(&sm.emptyV[sl]);
          if (++sl == NSX) { sl = 0; ph ^= 1u; }
        }
        mma2_commit(&sm.acc_ev[3 + part]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (8 warps)
    const int q4 = warp & 3, hh = (warp - 2) >> 2;
    const int row = q4 * 32 + lane;
    const uint32_t tlane = tm + ((uint32_t)(q4 * 32) << 16);
    const uint32_t mybit = 1u << ((int)rank * (BM / s.H) + row / s.H);      // node of this row within the pair's plan tile
    const float scale2 = s.sm_scale * 1.4426950408889634f;
    float m_run = -INFINITY;                         // reference max of the row (log2 units)
    float lp[4] = {0.f, 0.f, 0.f, 0.f};              // this thread's share of the row sum, four independent chains

    // The softmax code works on slabs of 32 keys in short loops: the kernel passes through it once per piece, so long
    // unrolled code would be fetched cold every time.
    //
    // Visibility of a slab for this warp's rows, 32 keys per word (bit t = key t of the slab).  The 32 rows of a warp
    // belong to one node (H >= 32 on this path), so one ballot over the keys' node masks gives the word.
    auto slab_vis = [&](int pc, int c) { return __ballot_sync(0xffffffffu, sm.kmask[pc * 256 + hh * 128 + c * 32 + lane] & mybit); };
    // masked maximum of one slab of S (fp32 columns [col, col + 32))
    auto slab_max = [&](uint32_t col, uint32_t vis, float mx) {
      uint32_t sv[32];
      tmem_ld32(col, sv);
      float mc[4] = {mx, -INFINITY, -INFINITY, -INFINITY};
      if (vis == 0xffffffffu) {
#pragma unroll
        for (int t = 0; t < 32; ++t) mc[t & 3] = fmaxf(mc[t & 3], __uint_as_float(sv[t]));
      } else {
#pragma unroll
        for (int t = 0; t < 32; ++t) if ((vis >> t) & 1u) mc[t & 3] = fmaxf(mc[t & 3], __uint_as_float(sv[t]));
      }
      return fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
    };
    // P of one slab: 32 S values -> 16 bf16 pairs (low half = even key) stored at P columns [pcol, pcol + 16); the row
    // sum shares go to lp
    auto slab_exp = [&](const uint32_t* sv, uint32_t vis, float moff, uint32_t pcol) {
      uint32_t pk[16];
      if (vis == 0xffffffffu) {
#pragma unroll
        for (int t = 0; t < 32; t += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(sv[t]), scale2, -moff));
          const float p1 = ex2(fmaf(__uint_as_float(sv[t + 1]), scale2, -moff));
          lp[(t >> 1) & 3] += p0 + p1;
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          pk[t >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
        }
      } else {
#pragma unroll
        for (int t = 0; t < 32; t += 2) {
          const float p0 = ((vis >> t) & 1u) ? ex2(fmaf(__uint_as_float(sv[t]), scale2, -moff)) : 0.f;
          const float p1 = ((vis >> (t + 1)) & 1u) ? ex2(fmaf(__uint_as_float(sv[t + 1]), scale2, -moff)) : 0.f;
          lp[(t >> 1) & 3] += p0 + p1;
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          pk[t >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
        }
      }
      tmem_st16(pcol, pk);
    };
    auto p_stored = [&](int pc) {                    // this warp's P of piece pc is in TMEM: tell the leader's MMA warp
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&sm.cmp_ev[pc]), 0));
    };
    auto block_mine = [&](int pc) { return hh * 128 < min(256, CL - pc * 256); };

    // The pieces arrive one after the other (the tensor core computes S of the next piece meanwhile).  The first piece sets
    // the reference maximum of the row; a later piece keeps it unless it exceeds it by more than RESCALE_GAP (weights up
    // to 2^16 are harmless in bf16/fp32), else the P written so far and the sums are rescaled.
    //
    // Where P lands: piece pc -> columns [128 pc, 128 pc + 128), the warps with hh = 0 write the lower 64 (keys of their S
    // block, the piece's first 128), the warps with hh = 1 the upper 64.  P of pieces 0 and 2 overlays the first half of the
    // piece's own S: a warp with hh = 0 writes behind its own reads (slab c -> P columns 16 c.. below the 32 c.. it has
    // read), but the warps with hh = 1 write over S slabs 2 and 3 of their hh = 0 neighbours, so those are read into
    // registers first; a barrier of the eight warps follows.  P of piece 1 overlays S of piece 0, which every warp
    // has finished with when it passes the barrier of piece 1's maximum exchange.
#pragma unroll 1
    for (int pc = 0; pc < npc; ++pc) {
      if (!fail && !mbar_wait(&sm.acc_ev[pc], 0)) fail = 1;
      fence_after();
      const bool mine = block_mine(pc);
      const uint32_t scol = tlane + (pc == 0 ? 0 : 256) + hh * 128, pcol = tlane + pc * 128 + hh * 64;
      float mx = -INFINITY;
      if (mine) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) mx = slab_max(scol + c * 32, slab_vis(pc, c), mx);
      }
      sm.xch[hh][row] = mx;
      compute_sync();
      const float m_pass = fmaxf(sm.xch[0][row], sm.xch[1][row]) * scale2;
      float factor = 1.f;
      if (m_pass > m_run + RESCALE_GAP || m_run == -INFINITY) {
        if (m_run != -INFINITY) factor = ex2(m_run - m_pass);
        m_run = m_pass;
      }
      if (pc && __any_sync(0xffffffffu, factor != 1.f)) {  // warp-uniform: tcgen05.ld/st are warp-collective
#pragma unroll 1
        for (int v = 0; v < 2 * pc; ++v) {           // this thread's P columns of the earlier pieces
          const uint32_t qcol = tlane + (v >> 1) * 128 + hh * 64 + (v & 1) * 32;
          uint32_t r[32];
          tmem_ld32(qcol, r);
#pragma unroll
          for (int t = 0; t < 32; ++t) {
            float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&r[t]));
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(f.x * factor, f.y * factor);
            r[t] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          tmem_st16(qcol, r);
          tmem_st16(qcol + 16, r + 16);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) lp[c] *= factor;
      }
      const float moff = (m_run == -INFINITY) ? 0.f : m_run;
      {
        uint32_t hold[64];
        if (hh == 0) {
          if (mine) {
            tmem_ld32_nowait(scol + 64, hold);
            tmem_ld32_nowait(scol + 96, hold + 32);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            tmem_regs_ready(hold);
            tmem_regs_ready(hold + 32);
          }
          fence_before();
        }
        // all eight warps meet: the neighbours' slabs are in registers, and everybody has read the exchanged maxima (the
        // exchange buffer is written again for the next piece)
        asm volatile("bar.sync 2, 256;" ::: "memory");
        if (hh) fence_after();
        if (mine) {
          const int nstream = hh == 0 ? 2 : 4;
#pragma unroll 1
          for (int c = 0; c < nstream; ++c) {
            uint32_t sv[32];
            tmem_ld32(scol + c * 32, sv);
            slab_exp(sv, slab_vis(pc, c), moff, pcol + c * 16);
          }
          if (hh == 0) {
            slab_exp(hold, slab_vis(pc, 2), moff, pcol + 32);
            slab_exp(hold + 32, slab_vis(pc, 3), moff, pcol + 48);
          }
        }
        // the MMA warp waits for the last piece only (and, with three pieces, for piece 1 before it overwrites that
        // piece's S columns); the wait for the stores of a later piece covers the earlier ones
        if (pc == npc - 1 || (npc == 3 && pc == 1)) p_stored(pc);
      }
    }
    const float l_part = (lp[0] + lp[1]) + (lp[2] + lp[3]);
    sm.xch[hh][row] = l_part;
    compute_sync();
    const float l_row = sm.xch[0][row] + sm.xch[1][row];

    const bool rowok = row0 + row < rows_seq;
    const bool full_tile = row0 + BM <= rows_seq;     // whole tile inside the sequence: rows may be stored as 32-row boxes
    const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
    const int cw = OW / 2;                            // columns of the part this thread handles: 128 or 64
    const uint32_t stage = ring + (uint32_t)NSX * SLOTP + (uint32_t)(warp - 2) * 4096;   // this warp's 32 rows x 64 columns (bf16)
    bool store_pending = false;
    for (int part = 0; part < NQ; ++part) {
      if (!fail && !mbar_wait(&sm.acc_ev[3 + part], 0)) fail = 1;
      fence_after();
      // the thread's columns of the part (128 or 64) go to registers at once, so that the MMA may overwrite the part
      // while the values are normalised and stored
      uint32_t ro[128];
#pragma unroll
      for (int c = 0; c < 4; ++c) if (c * 32 < cw) tmem_ld32_nowait(tlane + OCOL + hh * cw + c * 32, ro + c * 32);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_regs_ready(ro + c * 32);
      if (part < NQ - 1) {
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&sm.cmp_ev[3 + part]), 0));
      }
#pragma unroll
      for (int cg = 0; cg < 2; ++cg) {
        const int c0 = cg * 64;
        if (c0 >= cw) break;
        const uint32_t* r0 = ro + cg * 64;
        const uint32_t* r1 = ro + cg * 64 + 32;
        const int col = part * OW + hh * cw + c0;
        const bool many = GENERAL && nch > 1;
        if ((nch == 1 && full_tile) || many) {
          // stage the 32 x 64 bf16 tile in the 128-byte swizzle pattern and store it with one TMA request: into the output,
          // or (multi-chunk tiles, where a merge kernel follows) into the chunk's tile of normalised partial outputs, which a merge kernel
          // combines with the chunks' (max, sum)
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
            const CUtensorMap* omap = many ? &maps.part : &maps.out;
            // (a chunk's bf16 tile lies at the start of the chunk's slot for an fp32 tile: 2 BM rows of 1 KiB per slot)
            const int orow = many ? (int)((rix * pl.tc_chmax + chunk) * 2 * BM) + q4 * 32 : b * rows_seq + row0 + q4 * 32;
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(omap)), "r"(col), "r"(orow), "r"(stage) : "memory");
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
          float* po = reinterpret_cast<float*>(ws + pl.off_tpo) + ((rix * pl.tc_chmax + chunk) * BM + row) * DH + col;
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
        reinterpret_cast<float2*>(ws + pl.off_tpml)[(rix * pl.tc_chmax + chunk) * BM + row] = make_float2(m_run, l_row);
    }
    if (store_pending && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (!GENERAL && nch > 1) {
      // Tiles of two chunks where nothing longer can occur: each chunk leaves its unnormalised part of O with (max, sum)
      // per row; the CTA that finishes a 128-row tile last merges the parts (fixed order, so the result does not depend
      // on who was last).  (In general a merge kernel follows: one CTA would take too long over many chunks.)
      __threadfence();
      compute_sync();
      if (warp == 2 && lane == 0) {
        int32_t* cnt = reinterpret_cast<int32_t*>(ws + pl.off_tcnt) + rix;
        const int done = atomicAdd(cnt, 1);
        sm.merge_here = done == nch - 1;
      }
      compute_sync();
      if (sm.merge_here) {
        __threadfence();
        bf16* orow0 = reinterpret_cast<bf16*>(out_) + ((size_t)b * rows_seq + row0) * DH;
        const float* po = reinterpret_cast<const float*>(ws + pl.off_tpo) + rix * pl.tc_chmax * BM * DH;
        const float2* pml = reinterpret_cast<const float2*>(ws + pl.off_tpml) + rix * pl.tc_chmax * BM;
        // One CTA merges a whole 128-row tile, so global latency has to be covered inside the thread: a warp takes 16 rows
        // (w, w + 8, ...), first the rows' reference maxima and sums (lane j < 16 for row w + 8 j, one round of loads), then
        // four rows at a time with all their loads of a chunk pair in flight; a lane owns columns 4 (l + 32 k) .. + 3.
        const int w = warp - 2;
        float m_row = -INFINITY, inv_row = 0.f;
        if (lane < 16) {
          const int r = w + 8 * lane;
          float l = 0.f;
          for (int ch = 0; ch < nch; ++ch) { const float2 ml = __ldcg(pml + ch * BM + r); if (ml.y > 0.f) m_row = fmaxf(m_row, ml.x); }
          for (int ch = 0; ch < nch; ++ch) { const float2 ml = __ldcg(pml + ch * BM + r); if (ml.y > 0.f) l = fmaf(ml.y, exp2f(ml.x - m_row), l); }
          inv_row = l > 0.f ? 1.f / l : 0.f;
        }
#pragma unroll 1
        for (int step = 0; step < 4; ++step) {
          float4 acc[4][4];
          float mj[4], invj[4];
#pragma unroll
          for (int jx = 0; jx < 4; ++jx) {
            mj[jx] = __shfl_sync(0xffffffffu, m_row, 4 * step + jx);
            invj[jx] = __shfl_sync(0xffffffffu, inv_row, 4 * step + jx);
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[jx][k] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll 2
          for (int ch = 0; ch < nch; ++ch) {
            float2 ml[4];
            float4 v[4][4];
#pragma unroll
            for (int jx = 0; jx < 4; ++jx) {
              const int r = w + 8 * (4 * step + jx);
              ml[jx] = __ldcg(pml + ch * BM + r);
              const float4* p4 = reinterpret_cast<const float4*>(po + ((size_t)ch * BM + r) * DH);
#pragma unroll
              for (int k = 0; k < 4; ++k) v[jx][k] = __ldcg(p4 + lane + 32 * k);
            }
#pragma unroll
            for (int jx = 0; jx < 4; ++jx) {
              const float wgt = ml[jx].y > 0.f ? exp2f(ml[jx].x - mj[jx]) : 0.f;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                acc[jx][k].x = fmaf(v[jx][k].x, wgt, acc[jx][k].x); acc[jx][k].y = fmaf(v[jx][k].y, wgt, acc[jx][k].y);
                acc[jx][k].z = fmaf(v[jx][k].z, wgt, acc[jx][k].z); acc[jx][k].w = fmaf(v[jx][k].w, wgt, acc[jx][k].w);
              }
            }
          }
#pragma unroll
          for (int jx = 0; jx < 4; ++jx) {
            const int r = w + 8 * (4 * step + jx);
            if (row0 + r >= rows_seq) continue;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[jx][k].x * invj[jx], acc[jx][k].y * invj[jx]);
              const __nv_bfloat162 hi = __floats2bfloat162_rn(acc[jx][k].z * invj[jx], acc[jx][k].w * invj[jx]);
              uint2 o2;
              o2.x = *reinterpret_cast<const uint32_t*>(&lo); o2.y = *reinterpret_cast<const uint32_t*>(&hi);
              *reinterpret_cast<uint2*>(orow0 + (size_t)r * DH + 4 * (lane + 32 * k)) = o2;
            }
          }
        }
      }
    }
  }
  if (fail) atomicOr(status + b, TSV_ST_INTERNAL);
  fence_before();
  __syncthreads();
  cluster_sync_all();                                            // neither CTA leaves while the other may still signal it or read its memory
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tm) : "memory");
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

bool tva_tc_pair_usable(const tsv_cache& c) { return c.csa_rows > 0 && encode_fn() != nullptr; }

static_assert(sizeof(pair::MapSet) <= sizeof(TvaTcPrep::maps), "tensor-map block of TvaTcPrep too small");

// Everything of the paired kernel's launch that can fail on the host, done before any kernel of the call is enqueued:
// the tensor maps and the kernel's shared-memory attribute.
int prepare_tva_tc_pair(const tsv_shape& s, const TvaPlan& p, const tsv_cache& c, const tsv_nodes& nd, void* out, char* ws, TvaTcPrep& prep) {
  pair::MapSet& ms = *reinterpret_cast<pair::MapSet*>(prep.maps);
  // (a layer without HCA entries has no HCA array to map: its map is never used and stands in as a copy of the CSA one)
  const bool has_hca = c.hca_rows > 0 && c.hca_kv;
  const void* bases[4] = {c.csa_kv, has_hca ? c.hca_kv : c.csa_kv, c.win_kv, ws + p.off_misc};
  const int64_t rows[4] = {c.csa_rows, has_hca ? c.hca_rows : c.csa_rows, c.page_table ? c.tok_rows : (int64_t)s.B * s.window, (int64_t)s.B * p.tc_misc_rows};
  bool ok = make_map(&ms.q, nd.q, (int64_t)s.B * s.D * s.H, 128) && make_map(&ms.out, out, (int64_t)s.B * s.D * s.H, 32);
  for (int a = 0; a < 4 && ok; ++a) {
    for (int k = 0; k < 3 && ok; ++k) ok = make_map(&ms.src[a][k], bases[a], rows[a], 32 << k);
    ok = ok && make_map(&ms.row[a], bases[a], rows[a], 1);
  }
  // partial outputs: per (128-row tile, chunk) a slot of 128 x 512 fp32 (used so by the instantiation that merges inside
  // the kernel); the general instantiation stores 128 x 512 bf16 at the start of the slot: as rows of 1 KiB the buffer
  // has 2 x 128 rows per slot
  if (p.tc_chmax > 1) ok = ok && make_map(&ms.part, ws + p.off_tpo, (int64_t)s.B * 2 * p.tc_nt * p.tc_chmax * 2 * tc::BM, 32);
  else ms.part = ms.out;                                                       // (never used: no tile has more than one chunk)
  if (!ok) {
    fprintf(stderr, "tsv: cuTensorMapEncodeTiled failed\n");
    return TSV_ERR_CUDA;
  }
  if (cudaFuncSetAttribute(tc_attn_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, pair::SMEM_X) != cudaSuccess ||
      cudaFuncSetAttribute(tc_attn_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, pair::SMEM_X) != cudaSuccess) {
    fprintf(stderr, "tsv: cannot set %d bytes of dynamic shared memory: %s\n", pair::SMEM_X, cudaGetErrorString(cudaGetLastError()));
    return TSV_ERR_CUDA;
  }
  TSV_PREP(tc_attn_pair_kernel<true>);
  TSV_PREP(tc_attn_pair_kernel<false>);
  return TSV_OK;
}

int launch_tva_tc_pair(const tsv_shape& s, const TvaPlan& p, const TvaTcPrep& prep, bool general, void* out, char* ws, int32_t* status, cudaStream_t st) {
  const pair::MapSet& ms = *reinterpret_cast<const pair::MapSet*>(prep.maps);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * p.tc_nt * s.B, p.tc_chmax, 1);
  cfg.blockDim = dim3(pair::TTHREADS, 1, 1);
  cfg.dynamicSmemBytes = pair::SMEM_X;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;          // may take its places under the plan kernel's tail (it waits inside)
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const cudaError_t le = general ? cudaLaunchKernelEx(&cfg, tc_attn_pair_kernel<true>, ms, s, p, out, ws, status)
                                 : cudaLaunchKernelEx(&cfg, tc_attn_pair_kernel<false>, ms, s, p, out, ws, status);
  if (le != cudaSuccess) {
    int ncl = -1;
    cudaOccupancyMaxActiveClusters(&ncl, tc_attn_pair_kernel<true>, &cfg);
    fprintf(stderr, "tsv: cluster launch failed: %s (max active clusters %d, grid %d x %d x %d)\n", cudaGetErrorString(le), ncl,
            cfg.gridDim.x, cfg.gridDim.y, cfg.gridDim.z);
  }
  count_launch();
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) fprintf(stderr, "tsv: launch of the paired attention kernel failed: %s\n", cudaGetErrorString(e));
  return e == cudaSuccess ? TSV_OK : TSV_ERR_CUDA;
}

}  // namespace tsv
