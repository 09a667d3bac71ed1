// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores:
// shifted-view kernel with bulk-copied window runs (stride 1, 128-position tiles).
//
// Same GEMM formulation as conv_f16_shift.cu (paper Algorithm 1 with the S tile
// of im2win columns and Kw row-shifted views of it), but the S tile is no longer
// gathered from global memory with 2-byte loads.  For one channel the columns a
// tile needs are ONE contiguous run of the window tensor (rows x Kh halves, per
// image the tile touches).  The window tensor is a 2-D array [N*C channel planes]
// [Ho*Kh*Wp halves] to TMA (the plane pitch must be a multiple of 16 bytes), so a
// loader warp brings the runs of the ~22 channels of a k-block into a "raw"
// shared-memory stage with a handful of tiled TMA loads (boxes of 128 halves x
// nslot planes, starting on 8-element boundaries and overlapping by 8 so that
// every Kh-element record lies inside one box), several stages ahead: HBM/L2
// latency is hidden by the copy engine and no load/store-unit request is spent on
// global memory.  (One untiled bulk copy per channel was tried first: ~120 cycles
// of issue per copy made the loader the bottleneck.)  The producer warps only
// re-lay a raw stage into the k-major swizzled S stage (2-byte shared loads,
// 16-byte shared stores), which is latency-free work.
//
//   raw stage:  [box][slot = channel - first channel of the k-block][128 halves];
//               one more, all-zero slot per box serves padded k2.
//   S stage:    [row][64 halves], 128-byte swizzle            (as in conv_f16_shift.cu)
//
// Roles (16 warps): 8 repack warps, filter-TMA warp, MMA warp, raw-loader warp, 4 epilogue
// warps.  The kernel is persistent with a double-buffered accumulator in tensor memory, so
// that the epilogue of one tile overlaps the main loop of the next.  Rings: raw stages, S
// stages, filter stages.  All mbarrier waits are bounded.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;
constexpr int PRODUCER_WARPS = 8;
constexpr int PRODUCER_THREADS = PRODUCER_WARPS * 32;
constexpr int WARP_TMA = 8, WARP_MMA = 9, WARP_RAW = 10, WARP_EPI0 = 12;   // warp 11 idles
constexpr int NUM_WARPS = 16;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 6;
constexpr int SEG_MAX = 4;                           // images one tile may touch
constexpr int ITEMS = 5;                             // 16-byte chunks per producer thread and stage (<= 160 rows)

struct RawParams {
  const uint16_t* __restrict__ win;
  const uint32_t* __restrict__ rawtab;   // k2 -> slot*256 + u*2 ; padded k2 -> the zero slot
  float* __restrict__ y;
  uint32_t* status;
  int64_t VQ, img_stride, chan_stride, window_elems;
  int32_t C, N, Wq, Ho, Wo, HoWo, Co, Kh, Kw, num_kb;
  int32_t rows;             // rows of the S tile: 128 + halo, multiple of 8
  int32_t nslot;            // channel planes per box (without the zero slot)
  int32_t box_bytes;        // (nslot + 1) * 256
  int32_t raw_stage_bytes;  // maxbox * box_bytes
  int32_t a_stage_bytes;    // rows * 128
  int32_t rs, sa, sb;       // ring depths
  int32_t ntm, nwork;       // position tiles; work items = position tiles x channel tiles
};

constexpr int BOXW = 128;   // halves per box row
constexpr int BOXSTEP = 120;  // boxes of one segment start 120 halves apart (overlap 8 >= Kh - 1)

struct Segment {            // the part of a tile that lies in one image
  int32_t plane0;           // first channel plane of the image: n * C
  int32_t x0;               // first box column: the segment's first element rounded down to 8
  int32_t o0;               // offset of the segment's first element from x0 (0..7)
  int32_t row0, cnt;        // tile rows [row0, row0 + cnt)
  int32_t box0, nbox;       // boxes [box0, box0 + nbox) of the raw stage belong to this segment
  int32_t pad_;
};

// Splits the rows of the tile starting at virtual position q0 by image: within an image the
// columns of one channel are contiguous in the window tensor.  Lane g of the calling warp works out
// segment g (the segments after the first start on image boundaries, so there is no loop; a lone
// lane walking them cost the re-layout warps a quarter of their time on layers with three k-blocks);
// every lane gets the number of segments.
__device__ __forceinline__ int split_by_image(const RawParams& q, int q0, Segment* segs, int lane) {
  const int img_rows = q.Ho * q.Wq;               // VQ < 2^31 is a condition of this kernel
  const int n0 = q0 / img_rows, a0 = q0 - n0 * img_rows;
  const int first_cnt = q.rows < img_rows - a0 ? q.rows : img_rows - a0;
  const int n = n0 + lane;
  const int a = lane == 0 ? a0 : 0;
  const int row0 = lane == 0 ? 0 : first_cnt + (lane - 1) * img_rows;
  int cnt = q.rows - row0;
  if (cnt > img_rows - a) cnt = img_rows - a;
  const bool valid = lane < SEG_MAX && row0 < q.rows && n < q.N;
  const int f0 = a * q.Kh;                               // element offset inside the channel plane
  const int span = (f0 & 7) + cnt * q.Kh;
  const int nbox = !valid ? 0 : (span <= BOXW ? 1 : (span - (BOXW - BOXSTEP) + BOXSTEP - 1) / BOXSTEP);
  int incl = nbox;                                       // inclusive prefix sum over the first SEG_MAX lanes
  int t = __shfl_up_sync(0xffffffffu, incl, 1);
  if (lane >= 1) incl += t;
  t = __shfl_up_sync(0xffffffffu, incl, 2);
  if (lane >= 2) incl += t;
  if (valid) {
    segs[lane].plane0 = n * q.C;
    segs[lane].x0 = f0 & ~7;
    segs[lane].o0 = f0 & 7;
    segs[lane].row0 = row0;
    segs[lane].cnt = cnt;
    segs[lane].box0 = incl - nbox;
    segs[lane].nbox = nbox;
  }
  __syncwarp();
  return __popc(__ballot_sync(0xffffffffu, valid));
}

// Persistent kernel: every CTA walks work items w = blockIdx.x, blockIdx.x + gridDim.x, ...
// (w -> position tile w mod ntm, channel tile w div ntm).  The rings and their phases run on
// across work items; the accumulator is double buffered in tensor memory so that the epilogue
// warps drain one tile while the MMA warp already fills the next.
template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, (BN <= 128 ? 2 : 1))
conv_f16_raw_kernel(const __grid_constant__ CUtensorMap fmap, const __grid_constant__ CUtensorMap wmap, RawParams q) {
  constexpr int B_STAGE_BYTES = BN * KB * 2;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[6 * MAX_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;
  __shared__ Segment seg_s[NUM_WARPS][SEG_MAX];     // each warp keeps its own copy of the tile's segments

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // shared-memory map: S ring | filter ring | raw ring | k2 table
  const uint32_t a_ring = smem_u32(smem);
  const uint32_t b_ring = a_ring + q.sa * q.a_stage_bytes;
  const uint32_t raw_ring = b_ring + q.sb * B_STAGE_BYTES;
  unsigned char* raw_ptr = smem + q.sa * q.a_stage_bytes + q.sb * B_STAGE_BYTES;
  uint32_t* tab_s = reinterpret_cast<uint32_t*>(raw_ptr + q.rs * q.raw_stage_bytes);
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
      mbar_init(a_full0 + 8 * i, PRODUCER_WARPS);
      mbar_init(a_empty0 + 8 * i, 1);
      mbar_init(b_full0 + 8 * i, 1);
      mbar_init(b_empty0 + 8 * i, 1);
      mbar_init(r_full0 + 8 * i, 1);
      mbar_init(r_empty0 + 8 * i, PRODUCER_WARPS);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full0 + 8 * i, 1);
      mbar_init(acc_empty0 + 8 * i, 4);      // the four epilogue warps
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) tmem_alloc(smem_u32(&tmem_base_slot), 2 * BN);
  // k2 table into shared memory; zero slot of every raw stage
  for (int i = threadIdx.x; i < q.num_kb * KB; i += NUM_THREADS) tab_s[i] = __ldg(q.rawtab + i);
  for (int r = 0; r < q.rs * (q.raw_stage_bytes / q.box_bytes); ++r) {
    uint32_t* z = reinterpret_cast<uint32_t*>(raw_ptr + r * q.box_bytes + q.nslot * 256);
    for (int i = threadIdx.x; i < 64; i += NUM_THREADS) z[i] = 0u;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  Segment* segs = seg_s[warp];

  if (warp < PRODUCER_WARPS) {
    // ---------------- repack: raw stage -> S stage ------------------------------
    // item = (row, 16-byte chunk), item = chunk * rows + row (lanes on consecutive rows): fixed
    // per thread.  Per tile: rbase = byte offset of the row's data inside a raw slot (segment
    // offset + rows before it) | the segment's 16-byte phase for channel 0 << 24; bit 3 of meta
    // marks rows inside the tensor.
    uint32_t rbase[ITEMS], meta[ITEMS];
    int irow[ITEMS];
    const int n_items = q.rows * 8;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int item = threadIdx.x + it * PRODUCER_THREADS;
      meta[it] = 0xffffffffu;
      irow[it] = 0;
      if (item < n_items) {
        const int ch = item / q.rows;
        const int i = item - ch * q.rows;
        irow[it] = i;
        meta[it] = (uint32_t)(i * 128 + ((ch ^ (i & 7)) << 4)) | (uint32_t)ch;
      }
    }
    bool ok = true;
    int st = 0, rst = 0;
    uint32_t ph = 0, rph = 0;
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
      const int q0 = (w % q.ntm) * TILE_M;
      const int nseg = split_by_image(q, q0, segs, lane);
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        rbase[it] = 0;
        meta[it] &= ~8u;
        if (meta[it] == 0xfffffff7u) meta[it] = 0xffffffffu;   // "no such item" stays
        for (int g = 0; g < nseg; ++g) {
          const int i = irow[it];
          if (meta[it] != 0xffffffffu && i >= segs[g].row0 && i < segs[g].row0 + segs[g].cnt) {
            const int o = segs[g].o0 + (i - segs[g].row0) * q.Kh;   // offset of the row's record from x0
            int j = o / BOXSTEP;                                    // the box that holds the whole record
            if (j > segs[g].nbox - 1) j = segs[g].nbox - 1;
            rbase[it] = (uint32_t)((segs[g].box0 + j) * q.box_bytes + (o - j * BOXSTEP) * 2);
            meta[it] |= 8u;
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
        const uint32_t raw_stage = raw_ring + rst * q.raw_stage_bytes;
        const uint4* kt = reinterpret_cast<const uint4*>(tab_s + kb * KB);
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
          if (meta[it] == 0xffffffffu) continue;
          const int ch = (int)(meta[it] & 7u);
          const uint4 t0 = kt[ch * 2], t1 = kt[ch * 2 + 1];
          const uint32_t t[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
          uint32_t h[8];
          const uint32_t base = raw_stage + rbase[it];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            uint16_t v;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(base + t[e]));
            h[e] = v;
          }
          const bool live = (meta[it] & 8u) != 0;   // rows beyond the tensor contribute zeros
          const uint32_t w0 = live ? (h[0] | (h[1] << 16)) : 0u, w1 = live ? (h[2] | (h[3] << 16)) : 0u;
          const uint32_t w2 = live ? (h[4] | (h[5] << 16)) : 0u, w3 = live ? (h[6] | (h[7] << 16)) : 0u;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_stage + (meta[it] & ~15u)), "r"(w0),
                       "r"(w1), "r"(w2), "r"(w3)
                       : "memory");
        }
        if (threadIdx.x == 0) TIMER_LAP(3);     // repack
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(a_full0 + 8 * st);
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
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
      const int n0 = (w / q.ntm) * BN;
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        for (int v = 0; v < q.Kw; ++v) {
          ok = mbar_wait(b_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const uint32_t bar = b_full0 + 8 * st;
          if (leader) {
            mbar_arrive_expect_tx(bar, B_STAGE_BYTES);
            tma_load_3d(b_ring + st * B_STAGE_BYTES, &fmap, kb * KB, n0, v, bar);
          }
          __syncwarp();
          if (++st == q.sb) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == WARP_MMA) {
    // ---------------- MMA issuer ------------------------------------------------
    constexpr uint32_t idesc = instr_desc_f16(TILE_M, BN);
    const bool leader = elect_one();
    bool ok = true;
    int sta = 0, stb = 0;
    uint32_t pha = 0, phb = 0;
    uint32_t it = 0;                             // work items done by this CTA: accumulator buffer = it & 1
    const uint32_t a_lo0 = smem_desc_lo(a_ring), b_lo0 = smem_desc_lo(b_ring);
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x, ++it) {
      const uint32_t buf = it & 1u;
      TIMER_LAP(8);
      ok = mbar_wait(acc_empty0 + 8 * buf, ((it >> 1) & 1u) ^ 1u, &abort_flag, q.status);   // drained by the epilogue
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      TIMER_LAP(11);                             // MMA warp: wait for a free accumulator
      tc_fence_after();
      const uint32_t acc = tmem_acc + buf * (uint32_t)BN;
      uint32_t first = 0;
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        TIMER_LAP(8);
        ok = mbar_wait(a_full0 + 8 * sta, pha, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        TIMER_LAP(9);                            // MMA warp: wait for an S stage
        const uint32_t a_lo_stage = a_lo0 + (uint32_t)(sta * (q.a_stage_bytes >> 4));
        for (int v = 0; v < q.Kw; ++v) {
          TIMER_LAP(8);
          ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          TIMER_LAP(10);                         // MMA warp: wait for a filter stage
          tc_fence_after();
          const uint32_t b_lo = b_lo0 + (uint32_t)(stb * (B_STAGE_BYTES >> 4));
          const uint32_t a_lo = a_lo_stage + (uint32_t)v * 8u;   // kernel column v: the view starts v rows further down
          if (leader) {
#pragma unroll
            for (int j = 0; j < KB / 16; ++j) umma_f16_lohi(acc, a_lo + 2 * j, b_lo + 2 * j, idesc, first | (uint32_t)j);
            umma_commit(b_empty0 + 8 * stb);
          }
          __syncwarp();
          first = 1u;
          if (++stb == q.sb) { stb = 0; phb ^= 1u; }
        }
        if (ok && leader) umma_commit(a_empty0 + 8 * sta);
        __syncwarp();
        if (++sta == q.sa) { sta = 0; pha ^= 1u; }
      }
      if (ok && leader) umma_commit(acc_full0 + 8 * buf);
      __syncwarp();
    }
    if (leader) { TIMER_LAP(8); TIMER_FLUSH(); }
  } else if (warp == WARP_RAW) {
    // ---------------- raw loader: tiled TMA loads of the channel runs -----------
    const bool leader = elect_one();
    bool ok = true;
    int rst = 0;
    uint32_t rph = 0;
    TIMER_DECL;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x) {
      const int q0 = (w % q.ntm) * TILE_M;
      const int nseg = split_by_image(q, q0, segs, lane);
      int nbox = 0;
      for (int g = 0; g < nseg; ++g) nbox += segs[g].nbox;
      // box b of the stage: its segment and its place in it (lane b issues the copy)
      int bg = 0, bj = lane;
      while (bg < nseg - 1 && bj >= segs[bg].nbox) { bj -= segs[bg].nbox; ++bg; }
      const int bx = segs[bg].x0 + bj * BOXSTEP, by = segs[bg].plane0;
      for (int kb = 0; kb < q.num_kb && ok; ++kb) {
        if (leader) TIMER_LAP(6);              // raw loader: issuing copies
        ok = mbar_wait(r_empty0 + 8 * rst, rph ^ 1u, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (leader) TIMER_LAP(5);              // raw loader: wait for a free raw stage
        const uint32_t bar = r_full0 + 8 * rst;
        const int c_lo = (kb * KB) / q.Kh;
        const uint32_t stage = raw_ring + rst * q.raw_stage_bytes;
        // one lane announces the bytes, then every lane issues its box (issuing a copy costs a lone
        // lane several hundred cycles; a stage has up to a dozen)
        if (leader) mbar_arrive_expect_tx(bar, (uint32_t)(nbox * q.nslot * 256));
        __syncwarp();
        for (int b = lane; b < nbox; b += 32) {
          if (b == lane) {
            tma_load_2d(stage + b * q.box_bytes, &wmap, bx, by + c_lo, bar);
          } else {                                 // more than 32 boxes: beyond what the plan allows, kept for safety
            int g = 0, j = b;
            while (g < nseg - 1 && j >= segs[g].nbox) { j -= segs[g].nbox; ++g; }
            tma_load_2d(stage + b * q.box_bytes, &wmap, segs[g].x0 + j * BOXSTEP, segs[g].plane0 + c_lo, bar);
          }
        }
        __syncwarp();
        if (++rst == q.rs) { rst = 0; rph ^= 1u; }
      }
    }
    if (leader) { TIMER_LAP(6); TIMER_FLUSH(); }
  } else if (warp >= WARP_EPI0) {
    // ---------------- epilogue: tensor memory -> NCHW output --------------------
    const int lq = warp & 3;                     // tensor-memory lane quadrant this warp may read
    bool ok = true;
    uint32_t it = 0;
    for (int w = blockIdx.x; w < q.nwork && ok; w += gridDim.x, ++it) {
      const uint32_t buf = it & 1u;
      const int q0 = (w % q.ntm) * TILE_M;
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
      if (lane == 0) mbar_arrive(acc_empty0 + 8 * buf);
    }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_acc, 2 * BN);
  }
}

// ------------------------------------------------------------------- host side
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

// Ring depths that fit: S ring 2, raw ring 3 (2 if tight), filter ring as deep as fits (<= 4).
bool choose_rings(int bn, const RawPlan& plan, int* rs, int* sa, int* sb, int* smem_bytes) {
  // dynamic shared memory left after the alignment slack, the static part (barriers, segment
  // copies) and, for two CTAs per SM, the 1 KB the runtime reserves per CTA
  const int budget = (bn <= 128 ? kSmemMax / 2 : kSmemMax) - 1024 - 4096;
  const int fixed = (int)plan.K2p * 4;
  const int a = plan.a_stage_bytes, r = plan.raw_stage_bytes, b = bn * KB * 2;
  for (int rr = 3; rr >= 2; --rr)
    for (int bb = 4; bb >= 2; --bb)
      if (2 * a + rr * r + bb * b + fixed <= budget && (bb >= 3 || rr == 2)) {
        *rs = rr; *sa = 2; *sb = bb;
        *smem_bytes = 2 * a + rr * r + bb * b + fixed + 1024;
        return true;
      }
  return false;
}

template <int BN>
cudaError_t launch_bn(const CUtensorMap& fmap, const CUtensorMap& wmap, RawParams q, const RawPlan& plan, int co,
                      cudaStream_t stream) {
  int smem_bytes = 0;
  if (!choose_rings(BN, plan, &q.rs, &q.sa, &q.sb, &smem_bytes)) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(conv_f16_raw_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int64_t ntm = (plan.VQ + TILE_M - 1) / TILE_M;
  const int64_t nwork = ntm * ((co + BN - 1) / BN);
  if (nwork >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  q.ntm = (int32_t)ntm;
  q.nwork = (int32_t)nwork;
  const int slots = 148 * (BN <= 128 ? 2 : 1);        // persistent CTAs: one (two for narrow tiles) per SM
  const unsigned grid = (unsigned)(nwork < slots ? nwork : slots);
  conv_f16_raw_kernel<BN><<<grid, NUM_THREADS, smem_bytes, stream>>>(fmap, wmap, q);
  return cudaGetLastError();
}

}  // namespace

RawPlan plan_f16_raw(const Geometry& g) {
  RawPlan p{};
  p.eligible = false;
  if (g.s != 1) return p;
  if (g.Kw >= 5) return p;                         // wide kernels: filter-bound, tall tiles of the gather path win
  p.Wq = g.Wp;
  const int halo = g.Kw - 1;
  p.rows = TILE_M + (halo + 7) / 8 * 8;
  if (p.rows * 8 > ITEMS * PRODUCER_THREADS) return p;
  p.K2 = (int64_t)g.C * g.Kh;
  p.K2p = (p.K2 + KB - 1) / KB * KB;
  p.VQ = (int64_t)g.N * g.Ho * p.Wq;
  if (p.VQ >= ((int64_t)1 << 31) - 4 * TILE_M) return p;    // the kernel indexes virtual positions with 32 bits
  const int64_t img_rows = (int64_t)g.Ho * p.Wq;
  const int64_t segmax = (p.rows - 2) / img_rows + 2;     // images a tile can touch
  if (segmax > SEG_MAX) return p;
  if (g.Kh > 8) return p;                                 // a record must fit the 8-element box overlap
  if ((g.chan_stride * 2) % 16 != 0) return p;            // TMA needs a plane pitch that is a multiple of 16 bytes
  if ((int64_t)g.N * g.C >= ((int64_t)1 << 31)) return p;
  p.nslot = (KB - 1 + g.Kh - 1) / g.Kh + 1;               // channels a 64-wide k2 block can touch
  if (p.nslot > g.C) p.nslot = g.C;
  if (p.nslot > 256) return p;
  p.pitch = 256;
  // boxes one stage can need: the exact maximum over the tile start positions (period <= img_rows tiles)
  int maxbox = 1;
  {
    const int64_t ntiles = (p.VQ + TILE_M - 1) / TILE_M;
    const int64_t probe = ntiles < img_rows ? ntiles : img_rows;
    for (int64_t t = 0; t < probe && t < 65536; ++t) {
      int64_t a = (t * TILE_M) % img_rows;
      int remaining = p.rows, boxes = 0;
      while (remaining > 0) {
        const int cnt = (int)(remaining < img_rows - a ? remaining : img_rows - a);
        const int span = (int)((a * g.Kh) & 7) + cnt * g.Kh;
        boxes += span <= BOXW ? 1 : (span - (BOXW - BOXSTEP) + BOXSTEP - 1) / BOXSTEP;
        remaining -= cnt;
        a = 0;
      }
      if (boxes > maxbox) maxbox = boxes;
    }
    if (probe > 65536) maxbox += (int)segmax;   // unprobed phases: leave room for one more box per image
  }
  p.raw_stage_bytes = maxbox * (p.nslot + 1) * 256;
  p.a_stage_bytes = p.rows * 128;
  if (p.K2p * 4 > 24 * 1024) return p;
  if ((p.VQ + TILE_M - 1) / TILE_M * ((g.Co + 63) / 64) >= ((int64_t)1 << 31)) return p;
  int rs, sa, sb, smem;
  const int bn = g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256);
  if (!choose_rings(bn, p, &rs, &sa, &sb, &smem)) return p;
  p.eligible = true;
  return p;
}

cudaError_t launch_conv_f16_raw(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                const ScratchLayout& l, cudaStream_t stream) {
  const RawPlan plan = plan_f16_raw(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  const int bn = g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256);

  // Filter as Fp2[v][co][k2p] halves: a 3-D tensor (k2 fastest), one box = 64 k2 x BN channels of one v.
  CUtensorMap fmap;
  const cuuint64_t dims[3] = {(cuuint64_t)plan.K2p, (cuuint64_t)g.Co, (cuuint64_t)g.Kw};
  const cuuint64_t strides[2] = {(cuuint64_t)plan.K2p * 2, (cuuint64_t)plan.K2p * 2 * (cuuint64_t)g.Co};
  const cuuint32_t box[3] = {(cuuint32_t)KB, (cuuint32_t)bn, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult cr = encode(&fmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base + l.filter_off, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;

  // Window tensor as [N*C planes][chan_stride halves]; one box = 128 halves of nslot planes.
  CUtensorMap wmap;
  {
    const cuuint64_t wd[2] = {(cuuint64_t)g.chan_stride, (cuuint64_t)g.N * (cuuint64_t)g.C};
    const cuuint64_t ws[1] = {(cuuint64_t)g.chan_stride * 2};
    const cuuint32_t wb[2] = {(cuuint32_t)BOXW, (cuuint32_t)plan.nslot};
    const cuuint32_t we[2] = {1, 1};
    cr = encode(&wmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint16_t*>(window), wd, ws, wb, we,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }

  RawParams q;
  q.win = window;
  q.rawtab = reinterpret_cast<const uint32_t*>(base + l.koff_off);
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.VQ = plan.VQ; q.img_stride = g.img_stride; q.chan_stride = g.chan_stride; q.window_elems = g.window_elems;
  q.C = g.C; q.N = g.N; q.Wq = plan.Wq; q.Ho = g.Ho; q.Wo = g.Wo; q.HoWo = g.Ho * g.Wo; q.Co = g.Co;
  q.Kh = g.Kh; q.Kw = g.Kw; q.num_kb = (int32_t)(plan.K2p / KB);
  q.rows = plan.rows; q.nslot = plan.nslot; q.box_bytes = (plan.nslot + 1) * 256;
  q.raw_stage_bytes = plan.raw_stage_bytes; q.a_stage_bytes = plan.a_stage_bytes;
  q.rs = q.sa = q.sb = 2;
  if (bn == 64) return launch_bn<64>(fmap, wmap, q, plan, g.Co, stream);
  if (bn == 128) return launch_bn<128>(fmap, wmap, q, plan, g.Co, stream);
  return launch_bn<256>(fmap, wmap, q, plan, g.Co, stream);
}

}  // namespace im2win
