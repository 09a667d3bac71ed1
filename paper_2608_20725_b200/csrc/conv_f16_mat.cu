// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores:
// shifted-view kernel whose S tile is built by 8x8 matrix transposes.
//
// GEMM formulation (paper Algorithm 1, M x N x K = positions x Co x C*Kh*Kw): as in
// conv_f16_shift.cu every im2win column is staged once, S[row = virtual column][k2 = (c, u)],
// and the Kw kernel columns are Kw MMA groups against row-shifted views of that tile.
//
// What is new here is how S is built.  The shared-memory data pipe is the bottleneck of this
// kernel family (tensor-core operand reads, TMA writes and the producers' own loads/stores all
// go through it), so the re-layout from "channel planes of the window tensor" to "rows of S"
// must cost as few shared-memory wavefronts as possible:
//
//   * k order: k2 = (oct*Kh + u)*8 + e with channel c = 8*oct + e.  One 16-byte unit of an S
//     row then holds the 8 channels of an octet at one (column, u): an 8-vector ACROSS channel
//     planes, i.e. one row of a transposed 8x8 block of the raw data.
//   * raw stage: tiled TMA boxes [8*noct planes][136 halves] of the window tensor viewed as
//     [N][C][Ho*Kh*Wp]; boxes of a segment start 128 halves apart (the last 8 halves of a box
//     row only make the row pitch 272 bytes, which spreads the 8 planes of an octet over all
//     bank groups).  Channels beyond C are filled with zeros by the copy engine.
//   * re-layout: ONE ldmatrix.x4.trans (8 planes x 32 halves) and ONE stmatrix.x4 per 512
//     bytes: every lane computes one source address and one destination address, no data
//     shuffling in registers.
//   * S stage without swizzle: S[sub-tile][unit 0..7][row] 16 bytes each, so the address is
//     linear in the row and a view shifted by r rows starts 16*r bytes further (the MMA's
//     "no swizzle" K-major layout with 128 bytes between 8-row groups).  The rows per unit
//     plane, R, are chosen with R*Kh = 1 (mod 8) when Kh is odd, which makes the 8 destination
//     rows of one stmatrix matrix fall into 8 different bank groups.
//
//   * filter: packed as 8 KB images (64 output channels x 64 k2, already in the 128-byte-swizzled
//     order of a k-major MMA tile), so a filter tile is one contiguous run copied with 2 KB rows;
//     a filter stage holds all kernel columns of a k-block that fit, which keeps the MMA issuer's
//     barrier round trips at two waits and two commits per k-block.
//   * CTA pairs (tiles of 256 output channels): the two CTAs of a cluster share every MMA
//     (cta_group::2, M = 256), each staging its own 128 positions and half of the filter tile.
//
// Any stride s with Wp mod s = 0 (columns are de-interleaved into s sub-tiles as in
// conv_f16_shift.cu); the plane pitch of the window tensor must be a multiple of 16 bytes.
// Persistent CTAs, double-buffered accumulator in tensor memory, bounded mbarrier waits.
// Warp roles: 0-7 re-layout, 8 filter copies, 9 MMA issue (and tensor-memory allocation),
// 10-11 raw box copies, 12-15 epilogue.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;                       // 64 halves = 8 units per k-block
constexpr int REPACK_WARPS = 8;
constexpr int WARP_TMA = 8, WARP_MMA = 9, WARP_RAW = 10, WARP_EPI0 = 12;   // warps 10 and 11 load raw boxes
constexpr int NUM_WARPS = 16;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 6;
constexpr int SEG_MAX = 4;                           // images one tile may touch
constexpr int BOXW = 136;                            // halves per box row (272-byte pitch)
constexpr int BOXSTEP = 128;                         // halves of a box row that are used
constexpr int BATCH = 4;                             // direct path: re-layout tasks in flight per warp
constexpr int MAXBOX = 16;                           // boxes of one raw stage (per-lane table in registers)
constexpr int MAX_KB = 1024;                         // k-blocks (table in shared memory)

struct MatParams {
  float* __restrict__ y;
  uint32_t* status;
  int64_t VQ;
  int32_t C, N, Wq, Ho, Wo, HoWo, Co, Kh, Kw, s, num_kb;
  int32_t rows;             // virtual positions staged per tile: 128 + (Kw-1)/s
  int32_t R;                // rows per unit plane of an S sub-tile
  int32_t Cp8;              // channel octets
  int32_t nch_last;         // units of the last k-block (1..8)
  int32_t nplanes;          // planes per box
  int32_t box_bytes;        // nplanes * 272
  int32_t raw_stage_bytes;  // maxbox * box_bytes
  int32_t a_stage_bytes;    // s * 8 * R * 16, rounded up to 128
  uint32_t magic_kh, magic_s;   // floor(e / d) = (e * magic) >> 16 for e < 8192
  int32_t rs, sa, sb;       // ring depths
  int32_t vg;               // kernel columns per filter stage
  int32_t resident;         // 1: the filter ring holds the whole filter of the (only) channel tile: loaded once
  int32_t ntm, nwork;       // position tiles; work items = position tiles x channel tiles
  int32_t frows;            // 2 KB rows of the packed filter per (kernel column, k-block): 4 per 64 channels
};

struct Segment {            // the part of a tile that lies in one image
  int32_t n;                // image
  int32_t x0;               // first box column: the segment's first element rounded down to 8
  int32_t o0;               // offset of the segment's first element from x0 (0..7)
  int32_t row0;             // first S row of the segment
  int32_t elems;            // elements of one channel the segment covers: cnt * s * Kh
  int32_t box0, nbox;       // boxes [box0, box0 + nbox) of the raw stage belong to this segment
  int32_t pad_;
};

// Programmatic dependent launch: the convolution kernel is launched so that it may start while
// the filter pack (the kernel before it in the stream) is still running; its barrier setup, tensor
// memory allocation and descriptor fetches overlap the pack.  Every role that touches global memory
// first waits for the preceding kernel to have completed (and its writes to be visible).
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void let_next_kernel_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Splits the rows of the tile starting at virtual position q0 by image: within an image the
// columns of one channel are contiguous in the window tensor.  Returns the number of segments
// and, in *total_boxes, the boxes of one raw stage.
__device__ __forceinline__ int split_by_image(const MatParams& q, int q0, Segment* segs, int* total_boxes) {
  const int img_rows = q.Ho * q.Wq;              // VQ < 2^31 is a condition of this kernel
  int n = q0 / img_rows, a = q0 - n * img_rows;
  int remaining = q.rows, row0 = 0, box0 = 0, g = 0;
  const int per_row = q.s * q.Kh;
  while (remaining > 0 && n < q.N && g < SEG_MAX) {
    const int cnt = remaining < img_rows - a ? remaining : img_rows - a;
    const int f0 = a * per_row;                            // element offset inside the channel plane
    const int span = (f0 & 7) + cnt * per_row;
    segs[g].n = n;
    segs[g].x0 = f0 & ~7;
    segs[g].o0 = f0 & 7;
    segs[g].row0 = row0;
    segs[g].elems = cnt * per_row;
    segs[g].box0 = box0;
    segs[g].nbox = (span + BOXSTEP - 1) / BOXSTEP;
    box0 += segs[g].nbox;
    row0 += cnt;
    remaining -= cnt;
    a = 0;
    ++n;
    ++g;
  }
  *total_boxes = box0;
  return g;
}

// Kernel body.  PAIR = false: one CTA per work item (128 positions x BN channels).  PAIR = true:
// two CTAs of a cluster share every MMA (M = 256: 128 positions from each CTA, N = BN): each CTA
// stages its own S tile and HALF of the filter tile, the leader CTA (rank 0) issues the MMAs,
// the accumulator rows of a CTA's positions land in its own tensor memory.  Per CTA that halves
// the filter bytes written to and read from shared memory, which is what bounds the 1-CTA form.
// Barriers the leader's MMA warp waits on live in the leader CTA and collect arrivals from both
// CTAs; barriers signalled by MMA completion exist in both CTAs and are signalled together.
template <int BN, bool PAIR>
__device__ __forceinline__ void conv_f16_mat_body(const CUtensorMap& fmap, const CUtensorMap& wmap, const MatParams& q) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;            // filter rows (output channels) this CTA stages
  constexpr int B_TILE_BYTES = B_ROWS * KB * 2;         // one kernel column of one k-block
  const int B_STAGE_BYTES = q.vg * B_TILE_BYTES;        // a filter stage holds vg kernel columns
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int w_first = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[6 * MAX_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;
  __shared__ Segment seg_s[NUM_WARPS][SEG_MAX];     // each warp keeps its own copy of the tile's segments
  __shared__ __align__(16) unsigned char trash[512];   // destination of matrix rows that belong to no S unit

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // shared-memory map: filter ring (1024-byte aligned stages) | S ring | raw ring | k-block table
  const uint32_t b_ring = smem_u32(smem);
  const uint32_t a_ring = b_ring + q.sb * B_STAGE_BYTES;
  const uint32_t raw_ring = a_ring + q.sa * q.a_stage_bytes;
  uint32_t* kbinfo = reinterpret_cast<uint32_t*>(smem + q.sb * B_STAGE_BYTES + q.sa * q.a_stage_bytes +
                                                 q.rs * q.raw_stage_bytes);
  const uint32_t a_full0 = smem_u32(&bars[0]);
  const uint32_t a_empty0 = smem_u32(&bars[MAX_STAGES]);
  const uint32_t b_full0 = smem_u32(&bars[2 * MAX_STAGES]);
  const uint32_t b_empty0 = smem_u32(&bars[3 * MAX_STAGES]);
  const uint32_t r_full0 = smem_u32(&bars[4 * MAX_STAGES]);
  const uint32_t r_empty0 = smem_u32(&bars[5 * MAX_STAGES]);
  const uint32_t acc_full0 = smem_u32(&bars[6 * MAX_STAGES]);
  const uint32_t acc_empty0 = smem_u32(&bars[6 * MAX_STAGES + 2]);

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int i = 0; i < MAX_STAGES; ++i) {
      mbar_init(a_full0 + 8 * i, PAIR ? 2 * REPACK_WARPS : REPACK_WARPS);
      mbar_init(a_empty0 + 8 * i, 1);
      mbar_init(b_full0 + 8 * i, 1);
      mbar_init(b_empty0 + 8 * i, 1);
      mbar_init(r_full0 + 8 * i, 1);
      mbar_init(r_empty0 + 8 * i, REPACK_WARPS);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full0 + 8 * i, 1);
      mbar_init(acc_empty0 + 8 * i, PAIR ? 8 : 4);      // the four epilogue warps (of each CTA)
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) {
    if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_slot), 2 * BN);
    else tmem_alloc(smem_u32(&tmem_base_slot), 2 * BN);
  }
  // per k-block: first channel octet | octets << 16
  for (int kb = threadIdx.x; kb < q.num_kb; kb += NUM_THREADS) {
    const int oct_lo = (8 * kb) / q.Kh;
    int oct_hi = (8 * kb + 7) / q.Kh;
    if (oct_hi > q.Cp8 - 1) oct_hi = q.Cp8 - 1;
    kbinfo[kb] = (uint32_t)oct_lo | ((uint32_t)(oct_hi - oct_lo + 1) << 16);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();               // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  // where this CTA's arrivals for the MMA issuer go: the leader's barriers
  const uint32_t a_full_dst = PAIR ? mapa_shared(a_full0, 0) : a_full0;
  const uint32_t b_full_dst = PAIR ? mapa_shared(b_full0, 0) : b_full0;
  const uint32_t acc_empty_dst = PAIR ? mapa_shared(acc_empty0, 0) : acc_empty0;
  Segment* segs = seg_s[warp];

  if (warp < REPACK_WARPS) {
    // ---------------- re-layout: raw stage -> S stage ---------------------------
    // task = (box, octet of the k-block, group of 32 halves).  A warp owns one group of 32 halves
    // of every box and every second octet.  Where a lane's matrix row goes depends on the tile and
    // the box only, so it is worked out once per tile (boxinfo); per task only the unit of the
    // (octet, u) pair is added.
    bool ok = true;
    int st = 0, rst = 0;
    uint32_t ph = 0, rph = 0;
    const uint32_t trash_l = smem_u32(trash) + (lane >> 3) * 128;
    const uint32_t src_l = (uint32_t)(((lane & 7) * BOXW + (warp & 3) * 32 + (lane >> 3) * 8) * 2);
    const int m_l = (warp & 3) * 32 + lane;       // lane's matrix row = element m of the box row
    const int par = warp >> 2;                    // octets par, par + 2, ... (alternating with the box)
    const uint32_t r16 = (uint32_t)q.R * 16u;
    const bool use_table = q.num_kb > 2;
    TIMER_DECL;
    for (int w = w_first; w < q.nwork && ok; w += w_step) {
      const int q0 = (PAIR ? 2 * (w % q.ntm) + (int)rank : w % q.ntm) * TILE_M;
      int nseg = 0, total_boxes = 0;
      if (lane == 0) nseg = split_by_image(q, q0, segs, &total_boxes);
      nseg = __shfl_sync(0xffffffffu, nseg, 0);
      total_boxes = __shfl_sync(0xffffffffu, total_boxes, 0);
      __syncwarp();
      // boxinfo[b]: byte offset of (sub-tile, unit 0, this lane's S row) | u in the low 4 bits, or
      // bit 31 | bank group << 4 when the lane's element lies outside the segment
      uint32_t boxinfo[MAXBOX];
      if (use_table) {
        int g = 0, row0 = 0, seg_elems = segs[0].elems, seg_end = segs[0].nbox;
        int e0 = m_l - segs[0].o0;               // this lane's element in box 0 of the segment
#pragma unroll
        for (int b = 0; b < MAXBOX; ++b) {
          boxinfo[b] = 0x80000000u;
          if (b < total_boxes) {
            while (b >= seg_end) {
              ++g;
              row0 = segs[g].row0; seg_elems = segs[g].elems; seg_end = segs[g].box0 + segs[g].nbox;
              e0 = m_l - segs[g].o0 - segs[g].box0 * BOXSTEP;
            }
            const int e = b * BOXSTEP + e0;                                     // element of the segment
            boxinfo[b] = 0x80000000u | (uint32_t)(((q.R * e + row0) & 7) << 4);
            if ((unsigned)e < (unsigned)seg_elems) {
              const int col = (int)(((uint32_t)e * q.magic_kh) >> 16);
              const int u = e - col * q.Kh;
              const int vr = (int)(((uint32_t)col * q.magic_s) >> 16);
              const int sub = col - vr * q.s;
              boxinfo[b] = (uint32_t)((((sub << 3) * q.R + row0 + vr) << 4) | u);
            }
          }
        }
      }
      if (threadIdx.x == 0) TIMER_LAP(0);       // per-tile setup
      for (int kb = 0; kb < q.num_kb; ++kb) {
        if (lane == 0) {
          ok = mbar_wait(r_full0 + 8 * rst, rph, &abort_flag, q.status);
          if (threadIdx.x == 0) TIMER_LAP(1);   // wait for the raw stage
          if (ok) ok = mbar_wait(a_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          if (threadIdx.x == 0) TIMER_LAP(2);   // wait for a free S stage
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
        if (!ok) break;
        const uint32_t a_stage = a_ring + st * q.a_stage_bytes;
        const uint32_t raw_stage = raw_ring + rst * q.raw_stage_bytes + src_l;
        const uint32_t info = kbinfo[kb];
        const int oct_lo = (int)(info & 0xffffu), noct = (int)(info >> 16);
        const int nch = kb == q.num_kb - 1 ? q.nch_last : 8;
        const int unit0 = oct_lo * q.Kh - kb * 8;       // S unit of (first octet, u = 0); may be negative
        if (use_table) {
          // Four boxes (up to eight tasks) at a time: all matrix loads first, then the stores, so that
          // the loads' latencies overlap.  Within a box this warp takes octets o and o + 2.
          for (int oc = 0; oc < noct; oc += 4) {
  #pragma unroll
            for (int bg = 0; bg < MAXBOX; bg += 4) {
              if (bg < total_boxes) {
                uint32_t r[4][2][4];
  #pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int b = bg + i;
                  if (b < total_boxes) {
                    const int o = oc + ((par + b) & 1);
                    const uint32_t src = raw_stage + (uint32_t)(b * q.box_bytes + o * (8 * BOXW * 2));
                    if (o < noct) ldmatrix_x4_trans(src, r[i][0]);
                    if (o + 2 < noct) ldmatrix_x4_trans(src + 2 * (8 * BOXW * 2), r[i][1]);
                  }
                }
  #pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const int b = bg + i;
                  if (b < total_boxes) {
                    const int o = oc + ((par + b) & 1);
                    const uint32_t bi = boxinfo[b];
                    const uint32_t base = bi & 0x7ffffff0u;
                    const bool in_seg = (bi >> 31) == 0u;
                    const int unit_a = unit0 + o * q.Kh + (int)(bi & 15u);
                    // rows that belong to no S unit go to a scratch line, into the bank group the real
                    // destination would have had, so that the 8 rows of a matrix never collide
                    if (o < noct) {
                      const uint32_t ta = base + (uint32_t)unit_a * r16;
                      const uint32_t da =
                          (in_seg && (unsigned)unit_a < (unsigned)nch) ? a_stage + ta : trash_l + (ta & 0x70u);
                      stmatrix_x4(da, r[i][0]);
                    }
                    if (o + 2 < noct) {
                      const int unit_b = unit_a + 2 * q.Kh;
                      const uint32_t tb = base + (uint32_t)unit_b * r16;
                      const uint32_t db =
                          (in_seg && (unsigned)unit_b < (unsigned)nch) ? a_stage + tb : trash_l + (tb & 0x70u);
                      stmatrix_x4(db, r[i][1]);
                    }
                  }
                }
              }
            }
          }
        } else {
          // tiles with one or two k-blocks: the per-tile table would cost more than it saves;
          // warp w takes tasks w, w + 8, ... and works out each destination on the spot
          int o = warp >> 2, b = 0;
          while (o >= noct) { o -= noct; ++b; }
          // the current segment lives in registers; it changes at most SEG_MAX - 1 times per stage
          int g = 0, seg_o0 = segs[0].o0, seg_row0 = 0, seg_elems = segs[0].elems, seg_box0 = 0, seg_end = segs[0].nbox;
          while (b < total_boxes) {
            // BATCH tasks at a time: all matrix loads first, then the stores, so that the loads'
            // latencies overlap
            uint32_t r[BATCH][4], dst[BATCH];
            int cnt = 0;
  #pragma unroll
            for (int k = 0; k < BATCH; ++k) {
              if (b < total_boxes) {
                while (b >= seg_end) {
                  ++g;
                  seg_o0 = segs[g].o0; seg_row0 = segs[g].row0; seg_elems = segs[g].elems;
                  seg_box0 = segs[g].box0; seg_end = seg_box0 + segs[g].nbox;
                }
                ldmatrix_x4_trans(raw_stage + (uint32_t)(b * q.box_bytes + o * (8 * BOXW * 2)), r[k]);
                const int e = (b - seg_box0) * BOXSTEP + m_l - seg_o0;      // element of the segment
                const int ubase = unit0 + o * q.Kh;
                // rows that belong to no S unit go to a scratch line, into the bank group the real
                // destination would have had (R*e + const mod 8 when R*Kh = 1 mod 8), so that the 8
                // rows of a matrix never collide
                dst[k] = trash_l + (uint32_t)(((q.R * e + ubase * q.R + seg_row0) & 7) << 4);
                if ((unsigned)e < (unsigned)seg_elems) {
                  const int col = (int)(((uint32_t)e * q.magic_kh) >> 16);
                  const int u = e - col * q.Kh;
                  const int unit = ubase + u;
                  if ((unsigned)unit < (unsigned)nch) {
                    const int vr = (int)(((uint32_t)col * q.magic_s) >> 16);
                    const int sub = col - vr * q.s;
                    dst[k] = a_stage + (uint32_t)((((sub << 3) + unit) * q.R + seg_row0 + vr) << 4);
                  }
                }
                o += 2;
                while (o >= noct) { o -= noct; ++b; }
                cnt = k + 1;
              }
            }
  #pragma unroll
            for (int k = 0; k < BATCH; ++k)
              if (k < cnt) stmatrix_x4(dst[k], r[k]);
          }
        }
        if ((nch & 1) && kb == q.num_kb - 1) {
          // odd number of units: the last k step reads one more unit; make it zeros
          for (int sub = 0; sub < q.s; ++sub)
            for (int i = threadIdx.x; i < q.R; i += REPACK_WARPS * 32)
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(
                               a_stage + (uint32_t)((((sub << 3) + nch) * q.R + i) << 4)),
                           "r"(0u)
                           : "memory");
        }
        if (threadIdx.x == 0) TIMER_LAP(3);     // re-layout
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (PAIR) mbar_arrive_cluster(a_full_dst + 8 * st);
          else mbar_arrive(a_full0 + 8 * st);
          mbar_arrive(r_empty0 + 8 * rst);
        }
        if (threadIdx.x == 0) TIMER_LAP(4);     // fence + arrive
        if (++st == q.sa) { st = 0; ph ^= 1u; }
        if (++rst == q.rs) { rst = 0; rph ^= 1u; }
      }
    }
    if (threadIdx.x == 0) TIMER_FLUSH();
  } else if (warp == WARP_TMA) {
    // ---------------- TMA loader of the filter tiles ---------------------------
    wait_for_previous_kernel();
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0;
    for (int w = w_first; w < q.nwork && ok; w += w_step) {
      // first 2 KB row of this CTA's part of the channel tile in the packed filter (4 rows per 64 channels)
      const int row0 = ((w / q.ntm) * BN + (int)rank * B_ROWS) / 16;
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        for (int v0 = 0; v0 < q.Kw; v0 += q.vg) {
          const int nv = q.Kw - v0 < q.vg ? q.Kw - v0 : q.vg;      // kernel columns in this stage
          ok = mbar_wait(b_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (leader) {
            const uint32_t dst = b_ring + st * B_STAGE_BYTES;
            if (PAIR) {
              // the leader CTA announces both halves; each CTA's copies report to the leader's barrier
              if (rank == 0) mbar_arrive_expect_tx(b_full0 + 8 * st, (uint32_t)(2 * nv * B_TILE_BYTES));
              for (int i = 0; i < nv; ++i)
                tma_load_2d_pair(dst + i * B_TILE_BYTES, &fmap, 0, ((v0 + i) * q.num_kb + kb) * q.frows + row0,
                                 b_full_dst + 8 * st);
            } else {
              mbar_arrive_expect_tx(b_full0 + 8 * st, (uint32_t)(nv * B_TILE_BYTES));
              for (int i = 0; i < nv; ++i)
                tma_load_2d(dst + i * B_TILE_BYTES, &fmap, 0, ((v0 + i) * q.num_kb + kb) * q.frows + row0,
                            b_full0 + 8 * st);
            }
          }
          __syncwarp();
          if (++st == q.sb) { st = 0; ph ^= 1u; }
        }
      }
      if (q.resident) break;          // every stage now holds its k-block for good
    }
  } else if (warp == WARP_MMA && rank == 0) {
    // ---------------- MMA issuer (leader CTA of a pair) -------------------------
    constexpr uint32_t idesc = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, BN);
    const bool leader = elect_one();
    bool ok = true;
    int sta = 0, stb = 0;
    uint32_t pha = 0, phb = 0;
    uint32_t it = 0;                             // work items done by this CTA: accumulator buffer = it & 1
    const uint32_t a_lo0 = smem_desc_lo_noswz(a_ring, (uint32_t)q.R * 16u), b_lo0 = smem_desc_lo(b_ring);
    const uint32_t sub_units = 8u * (uint32_t)q.R;       // 16-byte units per sub-tile
    const uint32_t kstep_units = 2u * (uint32_t)q.R;     // 16-byte units per 16-element k step
    const int ks_last = (q.nch_last + 1) >> 1;
    TIMER_DECL;
    for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
      const uint32_t buf = it & 1u;
      TIMER_LAP(8);
      ok = PAIR ? mbar_wait_cluster(acc_empty0 + 8 * buf, ((it >> 1) & 1u) ^ 1u, &abort_flag, q.status)
                : mbar_wait(acc_empty0 + 8 * buf, ((it >> 1) & 1u) ^ 1u, &abort_flag, q.status);   // drained by the epilogue
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      TIMER_LAP(11);                             // MMA warp: wait for a free accumulator
      tc_fence_after();
      const uint32_t acc = tmem_acc + buf * (uint32_t)BN;
      uint32_t first = 0;
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        TIMER_LAP(8);
        ok = PAIR ? mbar_wait_cluster(a_full0 + 8 * sta, pha, &abort_flag, q.status)
                  : mbar_wait(a_full0 + 8 * sta, pha, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        TIMER_LAP(9);                            // MMA warp: wait for an S stage
        const uint32_t a_lo_stage = a_lo0 + (uint32_t)(sta * (q.a_stage_bytes >> 4));
        const int nks = kb == q.num_kb - 1 ? ks_last : KB / 16;
        uint32_t sub = 0, shift = 0;             // kernel column v reads sub-tile v mod s from row v div s on
        for (int v0 = 0; v0 < q.Kw; v0 += q.vg) {
          const int nv = q.Kw - v0 < q.vg ? q.Kw - v0 : q.vg;
          TIMER_LAP(8);
          if (!(q.resident && it > 0)) {       // a resident filter is complete after the first work item
            ok = PAIR ? mbar_wait_cluster(b_full0 + 8 * stb, phb, &abort_flag, q.status)
                      : mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          TIMER_LAP(10);                         // MMA warp: wait for a filter stage
          tc_fence_after();
          uint32_t b_lo = b_lo0 + (uint32_t)(stb * (B_STAGE_BYTES >> 4));
          if (leader) {
            for (int i = 0; i < nv; ++i) {
              const uint32_t a_lo = a_lo_stage + sub * sub_units + shift;
#pragma unroll 1
              for (int j = 0; j < nks; ++j) {
                if (PAIR)
                  umma_f16_ab_pair(acc, a_lo + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128, b_lo + 2 * j,
                                   kSmemDescHiSw128, idesc, first | (uint32_t)j);
                else
                  umma_f16_ab(acc, a_lo + (uint32_t)j * kstep_units, kSmemDescHiNoSwz128, b_lo + 2 * j,
                              kSmemDescHiSw128, idesc, first | (uint32_t)j);
              }
              first = 1u;
              b_lo += (uint32_t)(B_TILE_BYTES >> 4);
              if (++sub == (uint32_t)q.s) { sub = 0; ++shift; }
            }
            if (!q.resident) {
              if (PAIR) umma_commit_pair(b_empty0 + 8 * stb);
              else umma_commit(b_empty0 + 8 * stb);
            }
          }
          __syncwarp();
          if (++stb == q.sb) { stb = 0; phb ^= 1u; }
        }
        if (ok && leader) {
          if (PAIR) umma_commit_pair(a_empty0 + 8 * sta);
          else umma_commit(a_empty0 + 8 * sta);
        }
        __syncwarp();
        if (++sta == q.sa) { sta = 0; pha ^= 1u; }
      }
      if (ok && leader) {
        if (PAIR) umma_commit_pair(acc_full0 + 8 * buf);
        else umma_commit(acc_full0 + 8 * buf);
      }
      __syncwarp();
    }
    if (leader) { TIMER_LAP(8); TIMER_FLUSH(); }
  } else if (warp == WARP_RAW || warp == WARP_RAW + 1) {
    // ---------------- raw loaders: tiled TMA loads of the channel planes ---------
    // two warps share the boxes of a stage (even / odd): issuing a copy costs a few hundred
    // cycles and the stage is only complete when its last box has been requested
    const int half = warp - WARP_RAW;
    wait_for_previous_kernel();
    const bool leader = elect_one();
    bool ok = true;
    int rst = 0;
    uint32_t rph = 0;
    TIMER_DECL;
    for (int w = w_first; w < q.nwork && ok; w += w_step) {
      const int q0 = (PAIR ? 2 * (w % q.ntm) + (int)rank : w % q.ntm) * TILE_M;
      int nseg = 0, total_boxes = 0;
      if (lane == 0) nseg = split_by_image(q, q0, segs, &total_boxes);
      nseg = __shfl_sync(0xffffffffu, nseg, 0);
      total_boxes = __shfl_sync(0xffffffffu, total_boxes, 0);
      __syncwarp();
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        if (leader) TIMER_LAP(6);              // raw loader: issuing copies
        ok = mbar_wait(r_empty0 + 8 * rst, rph ^ 1u, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (leader) TIMER_LAP(5);              // raw loader: wait for a free raw stage
        const uint32_t bar = r_full0 + 8 * rst;
        const int c_lo = (int)(kbinfo[kb] & 0xffffu) * 8;
        const uint32_t stage = raw_ring + rst * q.raw_stage_bytes;
        if (leader) {
          if (half == 0) mbar_arrive_expect_tx(bar, (uint32_t)(total_boxes * q.box_bytes));
          for (int g = 0; g < nseg; ++g)
            for (int j = 0; j < segs[g].nbox; ++j)
              if (((segs[g].box0 + j) & 1) == half)
                tma_load_3d(stage + (segs[g].box0 + j) * q.box_bytes, &wmap, segs[g].x0 + j * BOXSTEP, c_lo,
                            segs[g].n, bar);
        }
        __syncwarp();
        if (++rst == q.rs) { rst = 0; rph ^= 1u; }
      }
    }
    if (leader) { TIMER_LAP(6); TIMER_FLUSH(); }
  } else if (warp >= WARP_EPI0) {
    // ---------------- epilogue: tensor memory -> NCHW output --------------------
    const int lq = warp & 3;                     // tensor-memory lane quadrant this warp may read
    wait_for_previous_kernel();                  // before the first store to y
    bool ok = true;
    uint32_t it = 0;
    for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
      const uint32_t buf = it & 1u;
      const int q0 = (PAIR ? 2 * (w % q.ntm) + (int)rank : w % q.ntm) * TILE_M;
      const int n0 = (w / q.ntm) * BN;
      const int vq = q0 + lq * 32 + lane;        // accumulator row = virtual position
      bool valid = false;
      float* yrow = q.y;
      if (vq < (int)q.VQ) {
        const int sg = vq / q.Wq;
        const int kq = vq - sg * q.Wq;
        const int n = sg / q.Ho;
        const int ho = sg - n * q.Ho;
        valid = kq < q.Wo;                       // trailing columns of a strip are no output
        yrow += ((int64_t)n * q.Co) * q.HoWo + ho * q.Wo + kq;
      }
      if (lane == 0) ok = mbar_wait(acc_full0 + 8 * buf, (it >> 1) & 1u, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if (!ok) break;
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + buf * (uint32_t)BN + ((uint32_t)(lq * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (n0 + c0 >= q.Co) break;
        uint32_t v[32];
        tmem_ld32(lane_base + (uint32_t)c0, v);
        if (valid) store_strided32(yrow + (int64_t)(n0 + c0) * q.HoWo, q.HoWo, v, q.Co - n0 - c0);
      }
      // the buffer may be overwritten once all four warps have read it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(acc_empty_dst + 8 * buf);
        else mbar_arrive(acc_empty0 + 8 * buf);
      }
    }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (PAIR) cluster_sync_all();               // no CTA leaves while its peer may still signal or read it
  if (warp == WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_acc, 2 * BN);
    else tmem_dealloc(tmem_acc, 2 * BN);
  }
}

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_f16_mat_kernel(const __grid_constant__ CUtensorMap fmap, const __grid_constant__ CUtensorMap wmap, MatParams q) {
  conv_f16_mat_body<BN, false>(fmap, wmap, q);
}

// CTA-pair form: clusters of two CTAs share every MMA (half as many MMA instructions per tile,
// half the filter tile per CTA).
template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
conv_f16_mat_pair_kernel(const __grid_constant__ CUtensorMap fmap, const __grid_constant__ CUtensorMap wmap, MatParams q) {
  conv_f16_mat_body<BN, true>(fmap, wmap, q);
}

// Filter pack for this kernel (paper Section "Im2win Convolution": height before width; here
// additionally grouped by channel octets): k2 = (oct*Kh + u)*8 + e, c = 8*oct + e.  The packed
// filter is a sequence of 8 KB images, one per (kernel column v, k-block kb, group of 64 output
// channels), each laid out exactly as the MMA wants a k-major tile with the 128-byte swizzle in
// shared memory (row = channel, 128 bytes; 16-byte chunk index XOR row mod 8), so that a filter
// tile is ONE contiguous run and can be copied with 2 KB rows (the copy engine spends about a
// cycle per row on top of the bytes).  Padded k2 and channels >= Co hold zeros.  Block (0,0,0)
// also clears the status block.
// One block handles one output channel and `noct` consecutive channel octets: their source halves
// ((co*C + c)*Kh + u)*Kw + v are one contiguous run of the OIHW filter, read coalesced into shared
// memory; every thread then assembles 16-byte units (8 channels of one (octet, u, v)) and stores
// them at their place in the tile images.
__global__ void pack_f16_mat_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp, uint32_t* status,
                                    int C, int Co, int Kh, int Kw, int K2p, int ncog, int noct) {
  extern __shared__ __align__(16) uint16_t pack_s[];
  let_next_kernel_start();
  const size_t f_total = (size_t)Co * C * Kh * Kw;
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int num_kb = K2p / KB;
  const int T = Kh * Kw;
  const int oct_a = blockIdx.x * noct;
  const int units_total = K2p / 8;                       // units per (co, v), padding included
  const int unit_a = oct_a * Kh;
  // the last block also covers the padded units beyond the last octet
  const int unit_b = (blockIdx.x == gridDim.x - 1) ? units_total : (oct_a + noct) * Kh;
  const int c_a = oct_a * 8;
  int nsrc = (C - c_a < noct * 8 ? C - c_a : noct * 8) * T;    // source halves that exist
  if (nsrc < 0) nsrc = 0;
  for (int co = blockIdx.y; co < ncog * 64; co += gridDim.y) {
    // The run is read with 16-byte loads from the 16-byte boundary at or before its start; run
    // element i then sits at run[i] = pack_s[i + mis].
    const size_t start = ((size_t)co * C + c_a) * T;
    const int mis = (int)(start & 7);
    __syncthreads();
    if (co < Co) {
      for (int vec = threadIdx.x; vec * 8 < mis + nsrc; vec += blockDim.x) {
        const size_t i0 = start - mis + (size_t)vec * 8;
        if (i0 + 8 <= f_total) {
          reinterpret_cast<uint4*>(pack_s)[vec] = __ldg(reinterpret_cast<const uint4*>(f + i0));
        } else {
          for (int h = 0; h < 8; ++h) pack_s[vec * 8 + h] = i0 + h < f_total ? f[i0 + h] : (uint16_t)0;
        }
      }
    }
    __syncthreads();
    const uint16_t* run = pack_s + mis;
    const int r = co & 63;
    const int nunits = unit_b - unit_a;
    for (int i = threadIdx.x; i < nunits * Kw; i += blockDim.x) {
      const int v = i / nunits;
      const int unit = unit_a + (i - v * nunits);
      const int oct = unit / Kh, u = unit - oct * Kh;
      uint32_t w[4];
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        uint32_t pair = 0;
#pragma unroll
        for (int lo = 0; lo < 2; ++lo) {
          const int e = 2 * h + lo;
          const int idx = ((oct - oct_a) * 8 + e) * T + u * Kw + v;     // (c - c_a)*T + u*Kw + v
          const uint32_t val = (co < Co && idx < nsrc && oct < oct_a + noct) ? run[idx] : 0u;
          pair |= val << (16 * lo);
        }
        w[h] = pair;
      }
      const int kb = unit >> 3, chunk = unit & 7;
      const size_t image = ((size_t)v * num_kb + kb) * ncog + (co >> 6);
      *reinterpret_cast<uint4*>(fp + image * 4096 + (size_t)r * 64 + (size_t)((chunk ^ (r & 7)) << 3)) =
          make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

constexpr int kSmemMax = 227 * 1024;

int tile_bn(const Geometry& g) { return g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256); }

// Ring depths that fit: S ring 2, raw ring 2, a filter stage of as many kernel columns as fit
// twice (every barrier round trip and commit costs the MMA issuer time, so fewer, larger filter
// stages are better), filter ring as deep as fits (<= 6), then a third raw stage if there is room.
// Narrow tiles try to fit two CTAs on an SM first.
bool choose_rings(int bn, int b_rows, int kw, int nct, const MatPlan& plan, int* rs, int* sa, int* sb, int* vg,
                  int* resident, int* smem_bytes) {
  const int fixed = plan.num_kb * 4;
  const int a = plan.a_stage_bytes, r = plan.raw_stage_bytes, tile = b_rows * KB * 2;
  *resident = 0;
  for (int half = (bn <= 128 ? 1 : 0); half >= 0; --half) {
    // dynamic shared memory left after the alignment slack, the static part (barriers, segment
    // copies) and, for two CTAs per SM, the 1 KB the runtime reserves per CTA
    const int budget = (half ? kSmemMax / 2 : kSmemMax) - 1024 - 4096;
    // One channel tile and a filter small enough: keep all of it in shared memory (loaded once per
    // CTA instead of once per work item).
    if (nct == 1 && plan.num_kb <= MAX_STAGES) {
      const int b = kw * tile;
      if (2 * a + 2 * r + plan.num_kb * b + fixed <= budget) {
        const int rr = (2 * a + 3 * r + plan.num_kb * b + fixed <= budget) ? 3 : 2;
        const int aa = (3 * a + rr * r + plan.num_kb * b + fixed <= budget) ? 3 : 2;
        *rs = rr; *sa = aa; *sb = plan.num_kb; *vg = kw; *resident = 1;
        *smem_bytes = aa * a + rr * r + plan.num_kb * b + fixed + 1024;
        return true;
      }
    }
    for (int g = kw; g >= 1; --g) {
      const int b = g * tile;
      if (2 * a + 2 * r + 2 * b + fixed > budget) continue;
      const int rr = (2 * a + 3 * r + 2 * b + fixed <= budget) ? 3 : 2;
      int bb = 2;
      while (bb < MAX_STAGES && (bb + 1) * g <= 12 && 2 * a + rr * r + (bb + 1) * b + fixed <= budget) ++bb;
      *rs = rr; *sa = 2; *sb = bb; *vg = g;
      *smem_bytes = 2 * a + rr * r + bb * b + fixed + 1024;
      return true;
    }
  }
  return false;
}

template <int BN>
cudaError_t launch_bn(const CUtensorMap& fmap, const CUtensorMap& wmap, MatParams q, const MatPlan& plan, int co,
                      cudaStream_t stream) {
  int smem_bytes = 0;
  if (!choose_rings(BN, BN, q.Kw, (co + BN - 1) / BN, plan, &q.rs, &q.sa, &q.sb, &q.vg, &q.resident, &smem_bytes))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(conv_f16_mat_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int64_t ntm = (plan.VQ + TILE_M - 1) / TILE_M;
  const int64_t nwork = ntm * ((co + BN - 1) / BN);
  if (nwork >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  q.ntm = (int32_t)ntm;
  q.nwork = (int32_t)nwork;
  const int per_sm = (BN <= 128 && smem_bytes + 1024 <= kSmemMax / 2) ? 2 : 1;
  const int slots = 148 * per_sm;                      // persistent CTAs
  const unsigned grid = (unsigned)(nwork < slots ? nwork : slots);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, conv_f16_mat_kernel<BN>, fmap, wmap, q);
}

// CTA-pair launch: clusters of two CTAs, as many as can be resident at once.
template <int BN>
cudaError_t launch_pair(const CUtensorMap& fmap, const CUtensorMap& wmap, MatParams q, const MatPlan& plan, int co,
                        cudaStream_t stream) {
  int smem_bytes = 0;
  if (!choose_rings(256, BN / 2, q.Kw, (co + BN - 1) / BN, plan, &q.rs, &q.sa, &q.sb, &q.vg, &q.resident, &smem_bytes))
    return cudaErrorInvalidValue;
  cudaError_t e =
      cudaFuncSetAttribute(conv_f16_mat_pair_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int64_t ntm = (plan.VQ + TILE_M - 1) / TILE_M;
  const int64_t ntp = (ntm + 1) / 2;                   // pairs of position tiles
  const int64_t nwork = ntp * ((co + BN - 1) / BN);
  if (nwork >= ((int64_t)1 << 30)) return cudaErrorInvalidValue;
  q.ntm = (int32_t)ntp;
  q.nwork = (int32_t)nwork;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(148, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&clusters, conv_f16_mat_pair_kernel<BN>, &cfg);
  if (e != cudaSuccess) return e;
  if (clusters < 1) return cudaErrorInvalidValue;
  if (clusters > 74) clusters = 74;
  if ((int64_t)clusters > nwork) clusters = (int)nwork;
  cudaLaunchAttribute lattr[2];
  lattr[0] = attr[0];
  lattr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  lattr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(2 * clusters, 1, 1);
  cfg.attrs = lattr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, conv_f16_mat_pair_kernel<BN>, fmap, wmap, q);
}

uint32_t magic16(int d) { return (uint32_t)(65536 / d + 1); }

}  // namespace

MatPlan plan_f16_mat(const Geometry& g) {
  MatPlan p{};
  p.eligible = false;
  if (g.Wp % g.s != 0) return p;
  if ((g.chan_stride * 2) % 16 != 0) return p;            // TMA needs a plane pitch that is a multiple of 16 bytes
  if (g.Kh > 16 || g.s > 8) return p;
  p.Wq = g.Wp / g.s;
  p.rows = TILE_M + (g.Kw - 1) / g.s;
  // rows per unit plane: R*Kh = 1 (mod 8) for odd Kh (conflict-free matrix stores), odd otherwise
  p.R = p.rows;
  while ((g.Kh & 1) ? ((p.R * g.Kh) & 7) != 1 : (p.R & 1) == 0) ++p.R;
  // the kernel divides by Kh and s with 16-bit reciprocals: check them over the ranges it uses
  for (int e = 0; e < p.rows * g.s * g.Kh + 8; ++e)
    if ((int)(((uint32_t)e * magic16(g.Kh)) >> 16) != e / g.Kh) return p;
  for (int c = 0; c < p.rows * g.s + 8; ++c)
    if ((int)(((uint32_t)c * magic16(g.s)) >> 16) != c / g.s) return p;
  p.Cp8 = (g.C + 7) / 8;
  const int64_t units = (int64_t)p.Cp8 * g.Kh;
  p.K2p = (units * 8 + KB - 1) / KB * KB;
  p.num_kb = (int32_t)(p.K2p / KB);
  if (p.num_kb > MAX_KB) return p;
  p.nch_last = (int32_t)(units - 8 * (int64_t)(p.num_kb - 1));
  p.VQ = (int64_t)g.N * g.Ho * p.Wq;
  if (p.VQ >= ((int64_t)1 << 31) - 4 * TILE_M) return p;    // the kernel indexes virtual positions with 32 bits
  const int64_t img_rows = (int64_t)g.Ho * p.Wq;
  const int64_t segmax = (p.rows - 2) / img_rows + 2;     // images a tile can touch
  if (segmax > SEG_MAX) return p;
  if (g.chan_stride >= ((int64_t)1 << 31)) return p;
  int noct = 1;
  for (int kb = 0; kb < p.num_kb && kb < 64; ++kb) {      // the pattern repeats after Kh k-blocks
    int hi = (8 * kb + 7) / g.Kh;
    if (hi > p.Cp8 - 1) hi = p.Cp8 - 1;
    const int n = hi - (8 * kb) / g.Kh + 1;
    if (n > noct) noct = n;
  }
  p.nplanes = 8 * noct;
  p.box_bytes = p.nplanes * BOXW * 2;
  // boxes one stage can need: the exact maximum over the tile start positions (period <= img_rows tiles)
  int maxbox = 1;
  {
    const int per_row = g.s * g.Kh;
    const int64_t ntiles = (p.VQ + TILE_M - 1) / TILE_M;
    const int64_t probe = ntiles < img_rows ? ntiles : img_rows;
    for (int64_t t = 0; t < probe && t < 65536; ++t) {
      int64_t a = (t * TILE_M) % img_rows;
      int remaining = p.rows, boxes = 0;
      while (remaining > 0) {
        const int cnt = (int)(remaining < img_rows - a ? remaining : img_rows - a);
        const int span = (int)((a * per_row) & 7) + cnt * per_row;
        boxes += (span + BOXSTEP - 1) / BOXSTEP;
        remaining -= cnt;
        a = 0;
      }
      if (boxes > maxbox) maxbox = boxes;
    }
    if (probe > 65536) maxbox += (int)segmax;   // unprobed phases: leave room for one more box per image
  }
  if (maxbox > MAXBOX) return p;
  p.raw_stage_bytes = maxbox * p.box_bytes;
  p.a_stage_bytes = (g.s * 8 * p.R * 16 + 127) / 128 * 128;
  if ((p.VQ + TILE_M - 1) / TILE_M * ((g.Co + 63) / 64) >= ((int64_t)1 << 31)) return p;
  p.scratch_bytes = (size_t)kStatusBytes + (size_t)p.K2p * ((g.Co + 63) / 64 * 64) * g.Kw * 2;
  int rs, sa, sb, vg, resident, smem;
  if (!choose_rings(tile_bn(g), tile_bn(g), g.Kw, 2, p, &rs, &sa, &sb, &vg, &resident, &smem)) return p;
  p.eligible = true;
  return p;
}

cudaError_t launch_pack_f16_mat(const uint16_t* filter, void* scratch, const Geometry& g, cudaStream_t stream) {
  const MatPlan plan = plan_f16_mat(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  uint16_t* fp = reinterpret_cast<uint16_t*>(base + kStatusBytes);
  const int ncog = (g.Co + 63) / 64;                    // groups of 64 output channels
  int noct = 4096 / (8 * g.T);                          // octets per block: staging of <= 4096 halves
  if (noct < 1) noct = 1;
  if (noct > plan.Cp8) noct = plan.Cp8;
  const size_t smem = ((size_t)noct * 8 * g.T + 16) * sizeof(uint16_t);
  if (smem > 48 * 1024) return cudaErrorInvalidValue;
  dim3 grid((unsigned)((plan.Cp8 + noct - 1) / noct), (unsigned)(ncog * 64 < 32768 ? ncog * 64 : 32768));
  pack_f16_mat_kernel<<<grid, 256, smem, stream>>>(filter, fp, reinterpret_cast<uint32_t*>(base), g.C, g.Co, g.Kh, g.Kw,
                                                   (int)plan.K2p, ncog, noct);
  return cudaGetLastError();
}

cudaError_t launch_conv_f16_mat(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                cudaStream_t stream) {
  const MatPlan plan = plan_f16_mat(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  uint16_t* fp = reinterpret_cast<uint16_t*>(base + kStatusBytes);
  const int bn = tile_bn(g);
  const char* pair_env = debug_getenv("IM2WIN_F16_PAIR");     // testing aid: 0 = never pair CTAs
  // measured: pairing pays for 256-channel tiles (the filter tile halves); narrow tiles gain nothing
  const bool pair = bn == 256 && !(pair_env && pair_env[0] == '0');
  const int ncog = (g.Co + 63) / 64;                    // groups of 64 output channels

  // Packed filter as a 2-D array of 2 KB rows (256 eight-byte elements); one box = this CTA's
  // rows of one (v, k-block): 128 bytes per output channel.
  CUtensorMap fmap;
  const int b_rows = pair ? bn / 2 : bn;
  const cuuint64_t frows_total = (cuuint64_t)g.Kw * plan.num_kb * ncog * 4;
  const cuuint64_t dims[2] = {256, frows_total};
  const cuuint64_t strides[1] = {2048};
  const cuuint32_t box[2] = {256, (cuuint32_t)(b_rows / 16)};
  const cuuint32_t estr[2] = {1, 1};
  CUresult cr = encode(&fmap, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, fp, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;

  // Window tensor as [N][C][chan_stride halves]; one box = 136 halves of nplanes channel planes of one image.
  CUtensorMap wmap;
  {
    const cuuint64_t wd[3] = {(cuuint64_t)g.chan_stride, (cuuint64_t)g.C, (cuuint64_t)g.N};
    const cuuint64_t ws[2] = {(cuuint64_t)g.chan_stride * 2, (cuuint64_t)g.img_stride * 2};
    const cuuint32_t wb[3] = {(cuuint32_t)BOXW, (cuuint32_t)plan.nplanes, 1};
    const cuuint32_t we[3] = {1, 1, 1};
    cr = encode(&wmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<uint16_t*>(window), wd, ws, wb, we,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }

  MatParams q;
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.VQ = plan.VQ;
  q.C = g.C; q.N = g.N; q.Wq = plan.Wq; q.Ho = g.Ho; q.Wo = g.Wo; q.HoWo = g.Ho * g.Wo; q.Co = g.Co;
  q.Kh = g.Kh; q.Kw = g.Kw; q.s = g.s; q.num_kb = plan.num_kb;
  q.rows = plan.rows; q.R = plan.R; q.Cp8 = plan.Cp8; q.nch_last = plan.nch_last;
  q.nplanes = plan.nplanes; q.box_bytes = plan.box_bytes;
  q.raw_stage_bytes = plan.raw_stage_bytes; q.a_stage_bytes = plan.a_stage_bytes;
  q.magic_kh = magic16(g.Kh); q.magic_s = magic16(g.s);
  q.rs = q.sa = q.sb = 2;
  q.vg = 1;
  q.resident = 0;
  q.ntm = q.nwork = 0;
  q.frows = ncog * 4;
  if (pair) return launch_pair<256>(fmap, wmap, q, plan, g.Co, stream);
  if (bn == 64) return launch_bn<64>(fmap, wmap, q, plan, g.Co, stream);
  if (bn == 128) return launch_bn<128>(fmap, wmap, q, plan, g.Co, stream);
  return launch_bn<256>(fmap, wmap, q, plan, g.Co, stream);
}

}  // namespace im2win
