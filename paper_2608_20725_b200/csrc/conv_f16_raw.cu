// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores:
// shifted-view kernel with bulk-copied window runs (stride 1, 128-position tiles).
//
// Same GEMM formulation as conv_f16_shift.cu (paper Algorithm 1 with the S tile
// of im2win columns and Kw row-shifted views of it), but the S tile is no longer
// gathered from global memory with 2-byte loads.  For one channel the columns a
// tile needs are ONE contiguous run of the window tensor (rows x Kh halves, per
// image the tile touches).  A loader warp therefore brings the runs of the ~22
// channels of a k-block into a "raw" shared-memory stage with untiled bulk copies
// (cp.async.bulk, 16-byte-aligned supersets of the runs, completion on an
// mbarrier), several stages ahead; HBM/L2 latency is hidden by the copy engine
// and no load/store-unit request is spent on global memory.  The producer warps
// only re-lay a raw stage into the k-major swizzled S stage (2-byte shared loads,
// 16-byte shared stores), which is latency-free work.
//
//   raw stage:  [slot = channel - first channel of the k-block][PITCH bytes]
//               slot layout: segment g (one per image) at soff_g, data starting
//               at its 16-byte phase;  a last all-zero slot serves padded k2.
//   S stage:    [row][64 halves], 128-byte swizzle            (as in conv_f16_shift.cu)
//
// Roles (11 warps): 8 repack/epilogue warps, filter-TMA warp, MMA warp, raw-loader
// warp.  Rings: raw stages, S stages, filter stages.  All mbarrier waits are bounded.
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
constexpr int NUM_THREADS = PRODUCER_THREADS + 96;   // + filter-TMA warp + MMA warp + raw-loader warp
constexpr int MAX_STAGES = 6;
constexpr int SEG_MAX = 4;                           // images one tile may touch
constexpr int ITEMS = 5;                             // 16-byte chunks per producer thread and stage (<= 160 rows)

struct RawParams {
  const uint16_t* __restrict__ win;
  const uint32_t* __restrict__ rawtab;   // k2 -> (slot*pitch + u*2) | ((c*cs16)&15) << 20 ; padded k2 -> zero slot
  float* __restrict__ y;
  uint32_t* status;
  int64_t VQ, img_stride, chan_stride, window_elems;
  int32_t C, N, Wq, Ho, Wo, HoWo, Co, Kh, Kw, num_kb;
  int32_t rows;             // rows of the S tile: 128 + halo, multiple of 8
  int32_t pitch, nslot;     // raw slot pitch in bytes; slots per stage (without the zero slot)
  int32_t raw_stage_bytes;  // (nslot + 1) * pitch
  int32_t a_stage_bytes;    // rows * 128
  int32_t cs16;             // (chan_stride * 2) & 15: how the 16-byte phase moves from channel to channel
  int32_t rs, sa, sb;       // ring depths
};

struct Segment {            // the part of a tile that lies in one image
  int64_t elem0;            // element offset of (image, channel 0, first row of the segment)
  int32_t row0, cnt;        // tile rows [row0, row0 + cnt)
  int32_t soff;             // byte offset of the segment inside a raw slot (multiple of 16)
};

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, (BN <= 128 ? 2 : 1))
conv_f16_raw_kernel(const __grid_constant__ CUtensorMap fmap, RawParams q) {
  constexpr int B_STAGE_BYTES = BN * KB * 2;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[6 * MAX_STAGES + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;
  __shared__ Segment segs[SEG_MAX];
  __shared__ int nseg_s;

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
  const uint32_t acc_bar = smem_u32(&bars[6 * MAX_STAGES]);

  const int64_t q0 = (int64_t)blockIdx.x * TILE_M;   // first virtual position of the tile
  const int n0 = blockIdx.y * BN;
  const int64_t img_rows = (int64_t)q.Ho * q.Wq;     // virtual positions per image

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
    mbar_init(acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // Split the tile's rows by image: within an image the columns of one channel are contiguous.
    int64_t n = q0 / img_rows, a = q0 - n * img_rows;
    int remaining = q.rows, row0 = 0, soff = 0, g = 0;
    while (remaining > 0 && n < q.N && g < SEG_MAX) {
      const int cnt = (int)(remaining < img_rows - a ? remaining : img_rows - a);
      segs[g].elem0 = n * q.img_stride + a * q.Kh;
      segs[g].row0 = row0;
      segs[g].cnt = cnt;
      segs[g].soff = soff;
      soff += (cnt * q.Kh * 2 + 16 + 15) & ~15;
      row0 += cnt;
      remaining -= cnt;
      a = 0;
      ++n;
      ++g;
    }
    nseg_s = g;
  }
  if (warp == PRODUCER_WARPS + 1) tmem_alloc(smem_u32(&tmem_base_slot), BN);
  // k2 table into shared memory; zero slot of every raw stage
  for (int i = threadIdx.x; i < q.num_kb * KB; i += NUM_THREADS) tab_s[i] = __ldg(q.rawtab + i);
  for (int r = 0; r < q.rs; ++r) {
    uint32_t* z = reinterpret_cast<uint32_t*>(raw_ptr + r * q.raw_stage_bytes + q.nslot * q.pitch);
    for (int i = threadIdx.x; i < q.pitch / 4; i += NUM_THREADS) z[i] = 0u;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  const int nseg = nseg_s;

  if (warp < PRODUCER_WARPS) {
    // ---------------- repack: raw stage -> S stage ------------------------------
    // item = (row, 16-byte chunk), item = chunk * rows + row (lanes on consecutive rows).
    // rbase = byte offset of the row's data inside a raw slot (segment offset + rows before it
    // + the segment's 16-byte phase for channel 0); meta = swizzled S offset | chunk | valid << 3.
    uint32_t rbase[ITEMS], meta[ITEMS];
    const int n_items = q.rows * 8;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int item = threadIdx.x + it * PRODUCER_THREADS;
      rbase[it] = 0;
      meta[it] = 0xffffffffu;
      if (item < n_items) {
        const int ch = item / q.rows;
        const int i = item - ch * q.rows;
        meta[it] = (uint32_t)(i * 128 + ((ch ^ (i & 7)) << 4)) | (uint32_t)ch;
        for (int g = 0; g < nseg; ++g) {
          if (i >= segs[g].row0 && i < segs[g].row0 + segs[g].cnt) {
            const uint32_t m0 = (uint32_t)((segs[g].elem0 * 2) & 15);
            rbase[it] = (uint32_t)(segs[g].soff + (i - segs[g].row0) * q.Kh * 2) | (m0 << 24);
            meta[it] |= 8u;
          }
        }
      }
    }
    const bool phase_moves = q.cs16 != 0;   // channel stride not a multiple of 16 bytes

    bool ok = true;
    int st = 0, rst = 0;
    uint32_t ph = 0, rph = 0;
    TIMER_DECL;
    if (threadIdx.x == 0) TIMER_LAP(0);
    for (int kb = 0; kb < q.num_kb; ++kb) {
      if (lane == 0) {
        ok = mbar_wait(r_full0 + 8 * rst, rph, &abort_flag, q.status);
        if (threadIdx.x == 0) TIMER_LAP(1);   // wait for the raw stage
        if (ok) ok = mbar_wait(a_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
        if (threadIdx.x == 0) TIMER_LAP(2);   // wait for a free S stage
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
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
        if (!phase_moves) {
          const uint32_t base = raw_stage + (rbase[it] & 0xffffffu) + (rbase[it] >> 24);
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            uint16_t v;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(base + t[e]));
            h[e] = v;
          }
        } else {
          const uint32_t base = raw_stage + (rbase[it] & 0xffffffu);
          const uint32_t m0 = rbase[it] >> 24;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            uint16_t v;
            const uint32_t mis = (m0 + (t[e] >> 20)) & 15u;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(base + (t[e] & 0xfffffu) + mis));
            h[e] = v;
          }
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

    // ---------------- epilogue --------------------------------------------------
    if (ok && lane == 0) ok = mbar_wait(acc_bar, 0u, &abort_flag, q.status);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    if (threadIdx.x == 0) TIMER_LAP(5);        // wait for the accumulator
    if (ok) {
      tc_fence_after();
      const int lq = warp & 3;                 // tensor-memory lane quadrant this warp may read
      const int chalf = warp >> 2;             // which half of the channel tile
      const int64_t vq = q0 + lq * 32 + lane;  // accumulator row = virtual position
      bool valid = false;
      float* yrow = q.y;
      if (vq < q.VQ) {
        const int64_t sg = vq / q.Wq;
        const int kq = (int)(vq - sg * q.Wq);
        const int64_t n = sg / q.Ho;
        const int ho = (int)(sg - n * q.Ho);
        valid = kq < q.Wo;                     // trailing columns of a strip are no output
        yrow += (n * q.Co) * q.HoWo + ho * q.Wo + kq;
      }
      const uint32_t lane_base = tmem_acc + ((uint32_t)(lq * 32) << 16);
#pragma unroll 1
      for (int c0 = chalf * (BN / 2); c0 < (chalf + 1) * (BN / 2); c0 += 32) {
        if (n0 + c0 >= q.Co) break;
        uint32_t v[32];
        tmem_ld32(lane_base + (uint32_t)c0, v);
        if (valid) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int co = n0 + c0 + j;
            if (co < q.Co) yrow[(int64_t)co * q.HoWo] = __uint_as_float(v[j]);
          }
        }
      }
    }
    if (threadIdx.x == 0) { TIMER_LAP(6); TIMER_FLUSH(); }   // epilogue
  } else if (warp == PRODUCER_WARPS) {
    // ---------------- TMA loader of the filter tiles ---------------------------
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0;
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
  } else if (warp == PRODUCER_WARPS + 1) {
    // ---------------- MMA issuer ------------------------------------------------
    constexpr uint32_t idesc = instr_desc_f16(TILE_M, BN);
    const bool leader = elect_one();
    bool ok = true;
    int sta = 0, stb = 0;
    uint32_t pha = 0, phb = 0, first = 0;
    const uint32_t a_lo0 = smem_desc_lo(a_ring), b_lo0 = smem_desc_lo(b_ring);
    TIMER_DECL;
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
          for (int j = 0; j < KB / 16; ++j) umma_f16_lohi(tmem_acc, a_lo + 2 * j, b_lo + 2 * j, idesc, first | (uint32_t)j);
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
    if (ok && leader) umma_commit(acc_bar);
    __syncwarp();
    if (leader) { TIMER_LAP(8); TIMER_FLUSH(); }
  } else {
    // ---------------- raw loader: bulk copies of the channel runs ---------------
    // Lane l serves slots l, l + 32, ... of a stage: for every image the tile touches, one
    // bulk copy of the 16-byte-aligned superset of (rows x Kh) halves of that channel.
    bool ok = true;
    int rst = 0;
    uint32_t rph = 0;
    const int64_t win_bytes = q.window_elems * 2;
    const int64_t win_bytes16 = win_bytes & ~(int64_t)15;
    for (int kb = 0; kb < q.num_kb && ok; ++kb) {
      ok = mbar_wait(r_empty0 + 8 * rst, rph ^ 1u, &abort_flag, q.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t bar = r_full0 + 8 * rst;
      const int c_lo = (kb * KB) / q.Kh;
      int c_hi = (kb * KB + KB - 1) / q.Kh;
      if (c_hi >= q.C) c_hi = q.C - 1;
      unsigned char* stage_ptr = raw_ptr + rst * q.raw_stage_bytes;
      for (int c = c_lo + lane; c <= c_hi; c += 32) {
        const int slot = c - c_lo;
        for (int g = 0; g < nseg; ++g) {
          const int64_t byte0 = (segs[g].elem0 + (int64_t)c * q.chan_stride) * 2;
          const int64_t beg = byte0 & ~(int64_t)15;
          const int64_t want_end = byte0 + (int64_t)segs[g].cnt * q.Kh * 2;
          int64_t end = (want_end + 15) & ~(int64_t)15;
          if (end > win_bytes16) end = win_bytes16;       // never read past the tensor
          unsigned char* dst = stage_ptr + slot * q.pitch + segs[g].soff;
          if (end > beg) {
            mbar_expect_tx(bar, (uint32_t)(end - beg));
            bulk_load(smem_u32(dst), reinterpret_cast<const unsigned char*>(q.win) + beg, (uint32_t)(end - beg), bar);
          }
          // the last (< 16) bytes of the whole tensor, if this run needs them, by plain loads
          for (int64_t b = (end > beg ? end : beg); b < want_end && b < win_bytes; b += 2)
            *reinterpret_cast<uint16_t*>(dst + (b - beg)) = __ldg(reinterpret_cast<const uint16_t*>(
                reinterpret_cast<const unsigned char*>(q.win) + b));
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);   // the one pending arrival: the phase completes when the bytes have landed
      if (++rst == q.rs) { rst = 0; rph ^= 1u; }
    }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == PRODUCER_WARPS + 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_acc, BN);
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
  const int budget = (bn <= 128 ? kSmemMax / 2 : kSmemMax) - 1024 - 512;
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
cudaError_t launch_bn(const CUtensorMap& fmap, RawParams q, const RawPlan& plan, int co, cudaStream_t stream) {
  int smem_bytes = 0;
  if (!choose_rings(BN, plan, &q.rs, &q.sa, &q.sb, &smem_bytes)) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(conv_f16_raw_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  dim3 grid((unsigned)((plan.VQ + TILE_M - 1) / TILE_M), (unsigned)((co + BN - 1) / BN));
  conv_f16_raw_kernel<BN><<<grid, NUM_THREADS, smem_bytes, stream>>>(fmap, q);
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
  const int64_t img_rows = (int64_t)g.Ho * p.Wq;
  const int64_t segmax = (p.rows - 2) / img_rows + 2;     // images a tile can touch
  if (segmax > SEG_MAX) return p;
  p.nslot = (KB - 1 + g.Kh - 1) / g.Kh + 1;               // channels a 64-wide k2 block can touch
  if (p.nslot > g.C) p.nslot = g.C;
  p.pitch = ((p.rows * g.Kh * 2 + 15) & ~15) + 32 * (int)segmax;
  if ((int64_t)(p.nslot + 1) * p.pitch >= (1 << 20)) return p;   // table entries keep 20 bits of offset
  p.raw_stage_bytes = (p.nslot + 1) * p.pitch;
  p.a_stage_bytes = p.rows * 128;
  if (p.K2p * 4 > 24 * 1024) return p;
  if ((p.VQ + TILE_M - 1) / TILE_M >= ((int64_t)1 << 31)) return p;
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

  RawParams q;
  q.win = window;
  q.rawtab = reinterpret_cast<const uint32_t*>(base + l.koff_off);
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.VQ = plan.VQ; q.img_stride = g.img_stride; q.chan_stride = g.chan_stride; q.window_elems = g.window_elems;
  q.C = g.C; q.N = g.N; q.Wq = plan.Wq; q.Ho = g.Ho; q.Wo = g.Wo; q.HoWo = g.Ho * g.Wo; q.Co = g.Co;
  q.Kh = g.Kh; q.Kw = g.Kw; q.num_kb = (int32_t)(plan.K2p / KB);
  q.rows = plan.rows; q.pitch = plan.pitch; q.nslot = plan.nslot;
  q.raw_stage_bytes = plan.raw_stage_bytes; q.a_stage_bytes = plan.a_stage_bytes;
  q.cs16 = (int32_t)((g.chan_stride * 2) & 15);
  q.rs = q.sa = q.sb = 2;
  if (bn == 64) return launch_bn<64>(fmap, q, plan, g.Co, stream);
  if (bn == 128) return launch_bn<128>(fmap, q, plan, g.Co, stream);
  return launch_bn<256>(fmap, q, plan, g.Co, stream);
}

}  // namespace im2win
