// Channel-innermost (NHWC) form of the im2win path on the sm_100a tensor cores: transform,
// filter pack and fp16-input / fp32-accumulate convolution.
//
// The paper's tensor-core kernel works on NHWC data (Section "Im2win Convolution on Tensor
// Cores").  With the channel innermost the im2win tensor is
//     win[n][ho][k][u][c] = xpad[n][c][ho*s + u][k],  k in [0, Wp), u in [0, Kh), c in [0, Cp),
// (Eq. 2 with the channel moved to the fastest position; Cp = C rounded up to 8, the extra
// channels are zeros), so the window of output (ho, wo) is ONE contiguous run of K = Kw*Kh*Cp
// halves that starts (wo*s)*Kh*Cp halves into strip (n, ho), and the next window starts s*Kh*Cp
// halves (a multiple of 16 bytes) later.  In the GEMM view of Algorithm 1 (M x N x K = positions
// x Co x K) the activation operand is therefore a matrix whose rows OVERLAP: row (n, ho, wo)
// begins s*Kh*Cp halves after row (n, ho, wo-1).  A tiled TMA map describes exactly that (inner
// dimension K, second dimension wo with a stride SHORTER than the row, third dimension the strips),
// so one copy brings 128 positions x 64 k straight into the 128-byte-swizzled K-major tile the MMA
// reads: no re-layout through registers or shared memory, nothing expanded in HBM.
//
// Kernel: persistent CTAs; warp 0 issues the TMA copies of both operands into a ring of stages,
// warp 1 issues tcgen05.mma (M = 128, N = BN; or, as a pair of CTAs, cta_group::2 with M = 256 and
// each CTA holding its own 128 positions and half of the filter tile), four warps drain the
// double-buffered accumulator from tensor memory and apply the epilogue (bias, ReLU, fp32 or fp16
// store, NCHW or NHWC).  Small grids split K and add their partial sums with red.global.add.f32
// into an output that was cleared first.  Every mbarrier wait is bounded.
#include <cuda.h>
#include <cuda_fp16.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;                 // 64 halves = one 128-byte swizzle row
constexpr int WARP_TMA = 0, WARP_MMA = 1, WARP_EPI0 = 2;
constexpr int EPI_WARPS = 8;                   // two per tensor-memory lane quadrant: each takes half of the tile's channels
constexpr int NUM_WARPS = 2 + EPI_WARPS;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 8;
constexpr int A_SLOT_BYTES = TILE_M * KB * 2;  // 16 KB: room for 128 rows even when a tile holds fewer
constexpr int kSmemMax = 227 * 1024;
constexpr int MAX_ACC = 8;                     // accumulator buffers in tensor memory: 512 columns / BN, at most 8
__host__ __device__ constexpr int acc_buffers(int bn) { return 512 / bn < MAX_ACC ? 512 / bn : MAX_ACC; }
// Flag words of the hand-offs between CTAs that share a tile of a short last round: two per tile (shifted-view
// kernel, one per CTA of a pair) or two per CTA pair of the grid (overlapping-row kernel), compared with a
// value that differs from launch to launch.
constexpr int kTailFlagBytes = 2048;
// Partial sums of such tiles (overlapping-row kernel): one accumulator tile of 128 positions x 256 channels
// of fp32 per CTA of the grid.
constexpr size_t kPartialBytes = (size_t)148 * TILE_M * 256 * 4;

// What the epilogue needs to know about the output (shared by both kernels of this file).
struct EpiParams {
  void* y;
  const float* bias;
  int32_t relu, out16, y_nhwc, atomic;
  int32_t Ho, Wo, Co, HoWo;
  int32_t rows_total;        // N*Ho strips
};

struct NhwcParams {
  EpiParams e;
  uint32_t* status;
  int32_t bw, G, tw;         // tile = G strips x bw output columns; tw tiles along a strip
  int32_t num_kc;            // chunks of KSUB 64-wide k-blocks (one ring stage each)
  int32_t nks_last;          // 16-wide MMA steps of the last chunk
  int32_t ksplit, kc_per_split;
  int32_t ntn, nwork;        // channel tiles; work items = position tiles (pairs) x channel tiles x k parts
  int32_t stages;
  uint32_t a_bytes;          // bytes one activation copy brings: G*bw*128
  int32_t tail_halves;       // host only: the last round's tiles may be handed out as halves
  int32_t n_main;            // work items below this index are whole tiles; each whole tile above it is two
                             // items, one per half of its channels (fills the last, short round of tiles)
  // ... or, with stream_tiles > 0, the last round's tiles are handed out by reduction length: their
  // stream_tiles * num_kc chunks in order, stream_u to each of the first stream_ctas CTAs (pairs), so a CTA
  // holds the end of one tile's reduction and / or the start of the next one's.  The CTA that starts a tile
  // stores it; the others leave their partial sums in `partial` and raise their flag.
  int32_t stream_tiles, stream_u, stream_ctas;
  int32_t raster, ntm_eff;   // testing aid: 1 = items in channel-tile-major order (ntm_eff position tiles (pairs) per channel tile)
  float* partial;            // kPartialBytes
  uint32_t* flags;           // two words per CTA (pair) of the grid, compared with `epoch`
  uint32_t epoch;
};

// Programmatic dependent launch: the convolution may start while the kernel before it in the stream
// (the filter pack) is still running, so that its barrier set-up, tensor-memory allocation and
// descriptor fetches overlap that kernel; every role that touches global memory first waits for the
// preceding kernel to have completed.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void red_add_f32(float* p, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

// Epilogue of one accumulator row chunk: v[j] belongs to output channel c0 + j (j < cnt) of the
// row's position; `base` is the element index of channel c0 at that position and `cs` the element
// distance between channels (Ho*Wo for NCHW, 1 for NHWC).
__device__ __forceinline__ void store_chunk(const EpiParams& q, int64_t base, int64_t cs, const uint32_t (&v)[32],
                                            int cnt, bool vec_ok, bool add = false) {
  if (q.atomic || add) {
    float* p = reinterpret_cast<float*>(q.y) + base;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < cnt) red_add_f32(p + j * cs, __uint_as_float(v[j]));
  } else if (!q.out16) {
    float* p = reinterpret_cast<float*>(q.y) + base;
    if (!q.y_nhwc) {
      store_strided32(p, cs, v, cnt);
    } else if (vec_ok && cnt == 32) {
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        *reinterpret_cast<uint4*>(p + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j < cnt) p[j] = __uint_as_float(v[j]);
    }
  } else {
    __half* p = reinterpret_cast<__half*>(q.y) + base;
    if (!q.y_nhwc) {
      __half* p0 = p;
      __half* p1 = p + cs;
      const int64_t step = 2 * cs;
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        if (j < cnt) *p0 = __float2half_rn(__uint_as_float(v[j]));
        if (j + 1 < cnt) *p1 = __float2half_rn(__uint_as_float(v[j + 1]));
        p0 += step; p1 += step;
      }
    } else if (vec_ok && cnt == 32) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint32_t w[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const __half2 h = __floats2half2_rn(__uint_as_float(v[j + 2 * t]), __uint_as_float(v[j + 2 * t + 1]));
          w[t] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p + j) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j < cnt) p[j] = __float2half_rn(__uint_as_float(v[j]));
    }
  }
}

// Bias (first K part only), ReLU and store of 32 channels from c0 on of one accumulator row.
__device__ __forceinline__ void finish_chunk(const EpiParams& e, uint32_t (&v)[32], int c0, int n0, bool first_part,
                                             bool valid, int64_t base, int64_t cs, bool vec_ok, bool add = false,
                                             const float* bias_regs = nullptr) {
  const int cnt = e.Co - n0 - c0;                // channels left from c0 on
  if (cnt <= 0) return;
  if (bias_regs != nullptr) {
    // this warp's 32 bias values, loaded once before the first tile (zeros beyond Co)
    if (first_part) {
#pragma unroll
      for (int t = 0; t < 32; ++t) v[t] = __float_as_uint(__uint_as_float(v[t]) + bias_regs[t]);
    }
  } else if (e.bias != nullptr && first_part) {
    // every lane adds the same 32 channel values: uniform 16-byte loads (the bias is 16-byte aligned
    // and n0 + c0 a multiple of 32), element by element at the ragged end
    if (cnt >= 32) {
      const float4* b4 = reinterpret_cast<const float4*>(e.bias + n0 + c0);
#pragma unroll
      for (int t = 0; t < 32; t += 4) {
        const float4 b = __ldg(b4 + t / 4);
        v[t] = __float_as_uint(__uint_as_float(v[t]) + b.x);
        v[t + 1] = __float_as_uint(__uint_as_float(v[t + 1]) + b.y);
        v[t + 2] = __float_as_uint(__uint_as_float(v[t + 2]) + b.z);
        v[t + 3] = __float_as_uint(__uint_as_float(v[t + 3]) + b.w);
      }
    } else {
#pragma unroll
      for (int t = 0; t < 32; ++t)
        if (t < cnt) v[t] = __float_as_uint(__uint_as_float(v[t]) + __ldg(e.bias + n0 + c0 + t));
    }
  }
  if (e.relu) {
#pragma unroll
    for (int t = 0; t < 32; ++t) v[t] = __float_as_uint(fmaxf(__uint_as_float(v[t]), 0.0f));
  }
  if (valid) store_chunk(e, base + (int64_t)c0 * cs, cs, v, cnt < 32 ? cnt : 32, vec_ok, add);
}

// Tiles of 64 channels with one channel tile: an epilogue warp stores the same 32 channels for every
// tile, so it loads their bias once (with the largest shared-memory carve-out a global load per tile is
// an L2 round trip of 600-800 cycles on warps that bound these layers: measured 143 -> 189 us on a 7x7
// stem).  Returns whether breg is to be used.
template <int BN>
__device__ __forceinline__ bool hoist_bias(const EpiParams& e, int ntn, int warp, float (&breg)[32]) {
  if (BN != 64 || e.bias == nullptr || ntn != 1) return false;
  const int c0 = ((warp - WARP_EPI0) >> 2) * 32;
#pragma unroll
  for (int t = 0; t < 32; ++t) breg[t] = c0 + t < e.Co ? __ldg(e.bias + c0 + t) : 0.0f;
  return true;
}

// One epilogue warp's share of a finished accumulator: tensor-memory lane quadrant warp % 4, the
// lower (warps 2..5) or upper (warps 6..9) half of the tile's `cols` channels, 32 channels at a time:
// bias, ReLU, store.  The tensor-memory load of the next 32 channels is in flight while the current
// ones are stored (two register sets, taken in turn).  `base` is the element index of the tile's first
// channel at this lane's position, `cs` the element distance between channels.
__device__ __forceinline__ void drain_accumulator(const EpiParams& e, int cols, int warp, int lane, uint32_t lane_base,
                                                  bool valid, int64_t base, int64_t cs, int n0, bool first_part, bool vec_ok,
                                                  bool add = false, const float* bias_regs = nullptr) {
  const int CH = cols / 2;                       // a multiple of 32
  const int cbeg = ((warp - WARP_EPI0) >> 2) * CH;
  const int cend = cbeg + CH;
  uint32_t va[32], vb[32];
  tmem_ld32_issue(lane_base + (uint32_t)cbeg, va);
#pragma unroll 1
  for (int c0 = cbeg; c0 < cend; c0 += 64) {
    tmem_ld_wait_for(va);
    if (c0 + 32 < cend) tmem_ld32_issue(lane_base + (uint32_t)(c0 + 32), vb);
    finish_chunk(e, va, c0, n0, first_part, valid, base, cs, vec_ok, add, bias_regs);
    if (c0 + 32 >= cend) break;
    tmem_ld_wait_for(vb);
    if (c0 + 64 < cend) tmem_ld32_issue(lane_base + (uint32_t)(c0 + 64), va);
    finish_chunk(e, vb, c0 + 32, n0, first_part, valid, base, cs, vec_ok, add);
  }
}

// Bounded wait for a flag word to hold `value` (written with release semantics by another CTA).
__device__ __noinline__ bool wait_flag(const uint32_t* flag, uint32_t value, volatile uint32_t* abort_flag, uint32_t* status) {
  uint32_t limit = *reinterpret_cast<volatile uint32_t*>(status + 1);
  if (limit == 0u) limit = SPIN_LIMIT;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t i = 0; i < limit; ++i) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v == value) return true;
    if ((i & 255u) == 255u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > SPIN_TIME_NS) break;
    }
    __nanosleep(64);
  }
  *abort_flag = 1u;
  atomicExch(status, 1u);
  return false;
}

// The eight epilogue warps have stored their shares of a tile (or of its partial sums); one of them then
// raises a flag for other CTAs.  Every warp fences its stores and arrives on a CTA-local mbarrier; the first
// epilogue warp's lane 0 takes the BOUNDED wait for all eight arrivals before it publishes (a bar.sync here
// could wait for good if one warp had given up on an earlier wait and left the loop).  `phase` is the
// barrier's parity for this use (all warps count the uses alike).
__device__ __forceinline__ void publish_when_all_stored(uint32_t epi_bar, uint32_t phase, int warp, int lane, uint32_t* flag,
                                                        uint32_t epoch, volatile uint32_t* abort_flag, uint32_t* status) {
  __threadfence();
  __syncwarp();
  if (lane == 0) mbar_arrive(epi_bar);
  if (warp == WARP_EPI0 && lane == 0) {
    // (testing aid: with the marker in word 2 of the status block the flag stays down)
    if (mbar_wait(epi_bar, phase, abort_flag, status) && *reinterpret_cast<volatile uint32_t*>(status + 2) != kDebugDropFlag)
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(epoch) : "memory");
  }
}

// CTA `cta`'s two stream items (see NhwcParams): slot 0 is the part of its chunk range that does not start
// a tile (it ends the tile the CTA before it started), slot 1 the part that starts one.  Every CTA takes
// slot 0 first, so a partial sum is complete long before the tile's owner, in its slot 1, asks for it, and
// no item that waits is ever ahead of the item it waits for.  Returns false for an empty slot; else the
// tile (index among the last round's tiles) and its chunks [kc0, kc1).
__device__ __forceinline__ bool decode_stream_item(const NhwcParams& q, int cta, int slot, int* tile, int* kc0, int* kc1) {
  const int n = q.num_kc;
  const int total = q.stream_tiles * n;
  const int a = cta * q.stream_u;
  if (cta >= q.stream_ctas || a >= total) return false;
  const int b = a + q.stream_u < total ? a + q.stream_u : total;
  const int t1 = a / n, r = a - t1 * n;
  const int end1 = b < (t1 + 1) * n ? b - t1 * n : n;        // where the range leaves tile t1 (stream_u <= n)
  if (slot == 0) {
    if (r == 0) return false;
    *tile = t1; *kc0 = r; *kc1 = end1;
    return true;
  }
  if (r == 0) { *tile = t1; *kc0 = 0; *kc1 = end1; return true; }
  if (b <= (t1 + 1) * n) return false;
  *tile = t1 + 1; *kc0 = 0; *kc1 = b - (t1 + 1) * n;
  return true;
}

// A finished partial accumulator -> this CTA's slot of the partial-sum area, laid out
// [32-channel chunk][4-channel group][128 rows][4 floats]: the 32 lanes of a warp (32 consecutive rows)
// write, and the tile's owner later reads, 512 contiguous bytes per instruction.
__device__ __forceinline__ void dump_partial(int cols, int warp, int lane, uint32_t lane_base, float* slot) {
  const int CH = cols / 2;
  const int cbeg = ((warp - WARP_EPI0) >> 2) * CH;
  const int row = (warp & 3) * 32 + lane;
#pragma unroll 1
  for (int c0 = cbeg; c0 < cbeg + CH; c0 += 32) {
    uint32_t v[32];
    tmem_ld32_issue(lane_base + (uint32_t)c0, v);
    tmem_ld_wait_for(v);
    float4* p = reinterpret_cast<float4*>(slot + (size_t)(c0 >> 5) * (TILE_M * 32)) + row;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      __stcg(p + j * TILE_M, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                __uint_as_float(v[4 * j + 3])));
  }
}

// The owner's drain of a tile whose reduction other CTAs shared: accumulator + `count` partial tiles
// (`stride` floats apart from slot0 on), then bias, ReLU and store as for any tile.
__device__ __forceinline__ void drain_with_partials(const EpiParams& e, int cols, int warp, int lane, uint32_t lane_base,
                                                    bool valid, int64_t base, int64_t cs, int n0, bool vec_ok,
                                                    const float* slot0, size_t stride, int count) {
  const int CH = cols / 2;
  const int cbeg = ((warp - WARP_EPI0) >> 2) * CH;
  const int row = (warp & 3) * 32 + lane;
#pragma unroll 1
  for (int c0 = cbeg; c0 < cbeg + CH; c0 += 32) {
    uint32_t v[32];
    tmem_ld32_issue(lane_base + (uint32_t)c0, v);
    tmem_ld_wait_for(v);
    const float* s0 = slot0 + (size_t)(c0 >> 5) * (TILE_M * 32) + row * 4;
#pragma unroll 1
    for (int t = 0; t < count; ++t) {
      const float4* p = reinterpret_cast<const float4*>(s0 + (size_t)t * stride);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float4 a = __ldcg(p + j * TILE_M);
        v[4 * j] = __float_as_uint(__uint_as_float(v[4 * j]) + a.x);
        v[4 * j + 1] = __float_as_uint(__uint_as_float(v[4 * j + 1]) + a.y);
        v[4 * j + 2] = __float_as_uint(__uint_as_float(v[4 * j + 2]) + a.z);
        v[4 * j + 3] = __float_as_uint(__uint_as_float(v[4 * j + 3]) + a.w);
      }
    }
    finish_chunk(e, v, c0, n0, true, valid, base, cs, vec_ok);
  }
}

// Whole tile index -> (position tile (pair) mt, channel tile nt, K part ks).  Default order: nt and ks
// fastest, so that the CTAs that share an activation tile run at the same time; the other order (all
// position tiles of a channel tile, then the next channel tile) exists for the ablation only.
__device__ __forceinline__ void tile_coords(const NhwcParams& q, int whole, int* mt, int* nt, int* ks) {
  const int per_mt = q.ntn * q.ksplit;
  int rem;
  if (q.raster == 0) { *mt = whole / per_mt; rem = whole - *mt * per_mt; }
  else { rem = whole / q.ntm_eff; *mt = whole - rem * q.ntm_eff; }
  *nt = rem / q.ksplit;
  *ks = rem - *nt * q.ksplit;
}

// Work item w of the overlapping-row kernel -> whole tile index and which part of its channels:
// half = -1 the whole tile, 0 / 1 its lower / upper half.
__device__ __forceinline__ void decode_item(const NhwcParams& q, int w, int* whole, int* half) {
  if (w < q.n_main) { *whole = w; *half = -1; }
  else { const int t = w - q.n_main; *whole = q.n_main + (t >> 1); *half = t & 1; }
}

template <int BN, bool PAIR, int KSUB>
__device__ __forceinline__ void conv_nhwc_body(const CUtensorMap& amap, const CUtensorMap& bmap, const CUtensorMap& bmap_h,
                                               const NhwcParams& q) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;              // filter rows (output channels) this CTA stages
  constexpr int NACC = acc_buffers(BN);                   // accumulator ring: the epilogue's latency is hidden behind NACC - 1 tiles
  constexpr uint32_t B_BYTES = (uint32_t)B_ROWS * KB * 2;
  constexpr uint32_t SUB_BYTES = (uint32_t)A_SLOT_BYTES + B_BYTES;       // one 64-wide k-block of both operands
  constexpr uint32_t STAGE_BYTES = KSUB * SUB_BYTES;                     // a multiple of 1024
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int w_first = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 2 * MAX_ACC + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[MAX_STAGES]);
  const uint32_t acc_full0 = smem_u32(&bars[2 * MAX_STAGES]);
  const uint32_t acc_empty0 = smem_u32(&bars[2 * MAX_STAGES + MAX_ACC]);
  const uint32_t epi_bar = smem_u32(&bars[2 * MAX_STAGES + 2 * MAX_ACC]);   // rendezvous of the epilogue warps (publish_when_all_stored)

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int i = 0; i < MAX_STAGES; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, 1);
    }
    for (int i = 0; i < MAX_ACC; ++i) {
      mbar_init(acc_full0 + 8 * i, 1);
      mbar_init(acc_empty0 + 8 * i, PAIR ? 2 * EPI_WARPS : EPI_WARPS);   // the epilogue warps (of each CTA)
    }
    mbar_init(epi_bar, EPI_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) {
    if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_slot), NACC * BN);
    else tmem_alloc(smem_u32(&tmem_base_slot), NACC * BN);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();               // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  const uint32_t full_dst = PAIR ? mapa_shared(full0, 0) : full0;          // the leader's barriers
  const uint32_t acc_empty_dst = PAIR ? mapa_shared(acc_empty0, 0) : acc_empty0;

  // work item w -> (position tile (pair) mt, channel tile nt, k part ks): tile_coords.  K is walked in
  // chunks of KSUB 64-wide k-blocks: one ring stage, one pair of barrier operations per chunk.

  if (warp == WARP_TMA) {
    // ---------------- copies of both operands ------------------------------------
    {
      const bool leader = elect_one();
      wait_for_previous_kernel();                // the filter pack (and everything before it) is complete
      int st = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int w = w_first; w < q.nwork && ok; w += w_step) {
        int whole, half, kc0, kc1;
        if (BN >= 128 && q.stream_tiles > 0 && w >= q.n_main) {
          if (!decode_stream_item(q, w_first, (w - q.n_main) / w_step, &whole, &kc0, &kc1)) continue;
          whole += q.n_main; half = -1;
        } else {
          decode_item(q, w, &whole, &half);
          kc0 = -1;
        }
        int mt, nt, ks;
        tile_coords(q, whole, &mt, &nt, &ks);
        const int mti = PAIR ? 2 * mt + (int)rank : mt;
        const int rg = mti / q.tw, wt = mti - rg * q.tw;
        const int z = rg * q.G, yc = wt * q.bw;
        // filter rows of this CTA: its share of the tile's channels, or of one half of them
        const int brow = half < 0 ? nt * BN + (int)rank * B_ROWS : nt * BN + half * (BN / 2) + (int)rank * (B_ROWS / 2);
        const uint32_t b_bytes = half < 0 ? B_BYTES : B_BYTES / 2;
        const CUtensorMap* bm = half < 0 ? &bmap : &bmap_h;
        if (kc0 < 0) {
          kc0 = ks * q.kc_per_split;
          kc1 = kc0 + q.kc_per_split < q.num_kc ? kc0 + q.kc_per_split : q.num_kc;
        }
        for (int kc = kc0; kc < kc1; ++kc) {
          ok = mbar_wait(empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (leader) {
            const uint32_t dst = ring + (uint32_t)st * STAGE_BYTES;
            const uint32_t bar = full_dst + 8 * st;
            // k-blocks beyond K read as zeros (and cost no memory traffic), so every stage brings the
            // same number of bytes.  In a pair the leader CTA announces the bytes of both CTAs.
            if (!PAIR || rank == 0) mbar_arrive_expect_tx(full0 + 8 * st, (PAIR ? 2u : 1u) * KSUB * (q.a_bytes + b_bytes));
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub) {
              const int kx = (kc * KSUB + sub) * KB;
              if (PAIR) {
                tma_load_3d_pair(dst + sub * SUB_BYTES, &amap, kx, yc, z, bar);
                tma_load_2d_pair(dst + sub * SUB_BYTES + (uint32_t)A_SLOT_BYTES, bm, kx, brow, bar);
              } else {
                tma_load_3d(dst + sub * SUB_BYTES, &amap, kx, yc, z, bar);
                tma_load_2d(dst + sub * SUB_BYTES + (uint32_t)A_SLOT_BYTES, bm, kx, brow, bar);
              }
            }
          }
          __syncwarp();
          if (++st == q.stages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == WARP_MMA && rank == 0) {
    // ---------------- MMA issuer (leader CTA of a pair) -----------------------------
    // Every byte the MMAs read was written by the copy engine, whose completion the barrier's
    // transaction count tracks, so CTA-scope waits suffice also for the peer's half.
    constexpr uint32_t idesc_whole = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, BN);
    constexpr uint32_t idesc_half = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, BN / 2);
    {
      // the whole warp walks the loop and takes the waits, one elected lane issues (measured faster
      // than a lone lane, whose satisfied waits cost more)
      const bool leader = elect_one();
      int st = 0;
      uint32_t ph = 0, it = 0;
      bool ok = true;
      const uint32_t a_lo0 = smem_desc_lo(ring), b_lo0 = smem_desc_lo(ring + (uint32_t)A_SLOT_BYTES);
      for (int w = w_first; w < q.nwork && ok; w += w_step) {
        int whole, half, kc0, kc1;
        if (BN >= 128 && q.stream_tiles > 0 && w >= q.n_main) {
          if (!decode_stream_item(q, w_first, (w - q.n_main) / w_step, &whole, &kc0, &kc1)) continue;
          half = -1;
        } else {
          decode_item(q, w, &whole, &half);
          int mt, nt, ks;
          tile_coords(q, whole, &mt, &nt, &ks);
          kc0 = ks * q.kc_per_split;
          kc1 = kc0 + q.kc_per_split < q.num_kc ? kc0 + q.kc_per_split : q.num_kc;
        }
        const uint32_t idesc = half < 0 ? idesc_whole : idesc_half;
        const uint32_t buf = it % (uint32_t)NACC, aph = (it / (uint32_t)NACC) & 1u;
        ok = mbar_wait(acc_empty0 + 8 * buf, aph ^ 1u, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem_acc + buf * (uint32_t)BN;
        uint32_t accumulate = 0;
        for (int kc = kc0; kc < kc1; ++kc) {
          ok = mbar_wait(full0 + 8 * st, ph, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const uint32_t a_lo = a_lo0 + (uint32_t)st * (STAGE_BYTES >> 4);
          const uint32_t b_lo = b_lo0 + (uint32_t)st * (STAGE_BYTES >> 4);
          if (leader) {
            const int nks = kc != q.num_kc - 1 ? KSUB * (KB / 16) : q.nks_last;
#pragma unroll
            for (int j = 0; j < KSUB * (KB / 16); ++j) {
              if (j < nks) {
                const uint32_t off = (uint32_t)(j / 4) * (SUB_BYTES >> 4) + 2u * (uint32_t)(j % 4);
                if (PAIR) umma_f16_ab_pair(acc, a_lo + off, kSmemDescHiSw128, b_lo + off, kSmemDescHiSw128, idesc, accumulate);
                else umma_f16_lohi(acc, a_lo + off, b_lo + off, idesc, accumulate);
                accumulate = 1u;
              }
            }
            if (PAIR) umma_commit_pair(empty0 + 8 * st);
            else umma_commit(empty0 + 8 * st);
          }
          __syncwarp();
          if (++st == q.stages) { st = 0; ph ^= 1u; }
        }
        if (ok && leader) {
          if (PAIR) umma_commit_pair(acc_full0 + 8 * buf);
          else umma_commit(acc_full0 + 8 * buf);
        }
        __syncwarp();
        ++it;                                    // (empty stream slots take no accumulator)
      }
    }
  } else if (warp >= WARP_EPI0) {
    // ---------------- epilogue: tensor memory -> output -----------------------------
    const int lq = warp & 3;                     // tensor-memory lane quadrant this warp may read
    const EpiParams& e = q.e;
    const bool vec_ok = e.out16 ? (e.Co % 8 == 0) : (e.Co % 4 == 0);
    wait_for_previous_kernel();                  // before the first store to y
    float breg[32];
    const bool hoisted = hoist_bias<BN>(e, q.ntn, warp, breg);
    bool ok = true;
    uint32_t it = 0, epi_phase = 0;
    TIMER_DECL;
    for (int w = w_first; w < q.nwork && ok; w += w_step) {
      const uint32_t buf = it % (uint32_t)NACC, aph = (it / (uint32_t)NACC) & 1u;
      int whole, half;
      // stream items: frag 1 = a partial sum for another CTA's tile, 2 = the start of a tile others complete
      int frag = 0, fkc1 = 0, ftile = 0;
      if (BN >= 128 && q.stream_tiles > 0 && w >= q.n_main) {
        int fkc0;
        if (!decode_stream_item(q, w_first, (w - q.n_main) / w_step, &ftile, &fkc0, &fkc1)) continue;
        whole = ftile + q.n_main; half = -1;
        frag = fkc0 > 0 ? 1 : (fkc1 < q.num_kc ? 2 : 0);
      } else {
        decode_item(q, w, &whole, &half);
      }
      int mt, nt, ks;
      tile_coords(q, whole, &mt, &nt, &ks);
      const int mti = PAIR ? 2 * mt + (int)rank : mt;
      const int rg = mti / q.tw, wt = mti - rg * q.tw;
      const int n0 = nt * BN + (half > 0 ? BN / 2 : 0);
      const int cols = half < 0 ? BN : BN / 2;
      // accumulator row r = lane of tensor memory = (strip j of the tile, column i of the tile)
      const int r = lq * 32 + lane;
      const int j = r / q.bw, i = r - j * q.bw;
      const int strip = rg * q.G + j, wo = wt * q.bw + i;
      const bool valid = j < q.G && strip < e.rows_total && wo < e.Wo;
      int64_t base = 0, cs = 1;
      if (valid) {
        if (e.y_nhwc) {
          base = ((int64_t)strip * e.Wo + wo) * e.Co + n0;
        } else {
          const int n = strip / e.Ho, ho = strip - n * e.Ho;
          cs = e.HoWo;
          base = ((int64_t)n * e.Co + n0) * e.HoWo + ho * e.Wo + wo;
        }
      }
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(5);     // epilogue: draining and storing
      if (lane == 0) ok = mbar_wait(acc_full0 + 8 * buf, aph, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if (!ok) break;
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(6);     // epilogue: wait for a finished accumulator
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + buf * (uint32_t)BN + ((uint32_t)(lq * 32) << 16);
      if (BN < 128 || frag == 0) {
        drain_accumulator(e, cols, warp, lane, lane_base, valid, base, cs, n0, ks == 0, vec_ok, false, hoisted ? breg : nullptr);
      } else {
        constexpr int PER = PAIR ? 2 : 1;                    // slots and flag words per CTA (pair) of the grid
        constexpr size_t SLOT = (size_t)BN * TILE_M;         // floats of one CTA's partial tile
        if (frag == 1) {
          dump_partial(cols, warp, lane, lane_base, q.partial + (size_t)(PER * w_first + (int)rank) * SLOT);
          publish_when_all_stored(epi_bar, epi_phase, warp, lane, q.flags + PER * w_first + (int)rank, q.epoch, &abort_flag, q.status);
          epi_phase ^= 1u;
        } else {
          if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(5);
          // the CTAs after this one whose ranges reach into the tile
          int last = ((ftile + 1) * q.num_kc - 1) / q.stream_u;
          if (last > q.stream_ctas - 1) last = q.stream_ctas - 1;
          const int count = last - w_first;
          if (lane == 0)
            for (int t = 1; t <= count && ok; ++t) ok = wait_flag(q.flags + PER * (w_first + t) + (int)rank, q.epoch, &abort_flag, q.status);
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          __syncwarp();
          if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(8);   // epilogue: wait for the other CTAs' partial sums
          if (ok)
            drain_with_partials(e, cols, warp, lane, lane_base, valid, base, cs, n0, vec_ok,
                                q.partial + (size_t)(PER * (w_first + 1) + (int)rank) * SLOT, PER * SLOT, count);
        }
      }
      // the buffer may be overwritten once all four warps (of both CTAs) have read it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(acc_empty_dst + 8 * buf);
        else mbar_arrive(acc_empty0 + 8 * buf);
      }
      ++it;
    }
    if (threadIdx.x == WARP_EPI0 * 32 && blockIdx.x == 0) { TIMER_LAP(5); TIMER_FLUSH(); }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);     // copies in flight land before the CTA leaves
    __syncthreads();
  }
  if (PAIR) cluster_sync_all();               // no CTA leaves while its peer may still signal or read it
  if (warp == WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_acc, NACC * BN);
    else tmem_dealloc(tmem_acc, NACC * BN);
  }
}

template <int BN, int KSUB>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_f16_nhwc_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
                     const __grid_constant__ CUtensorMap bmap_h, NhwcParams q) {
  conv_nhwc_body<BN, false, KSUB>(amap, bmap, bmap_h, q);
}

template <int BN, int KSUB>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
conv_f16_nhwc_pair_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
                          const __grid_constant__ CUtensorMap bmap_h, NhwcParams q) {
  conv_nhwc_body<BN, true, KSUB>(amap, bmap, bmap_h, q);
}

// ------------------------------------------------------------------------------------------------
// Second kernel: shifted views.  The copies above bring every element of a strip into shared
// memory Kw/s times (the rows of the activation operand overlap).  The im2win layout lets the MMA
// use that overlap instead: stage every COLUMN of the strips once,
//     S[sub-tile t][row = virtual position q][64 halves of k2 = (u, c)],   column k = q*s + t,
// and multiply kernel column v against the view of sub-tile v mod s that starts v div s rows
// further down (the 128-byte swizzle is a function of the shared-memory address, so a view may start
// at any row).  One MMA row is one virtual position q = strip*Wq + i, Wq = Wp/s; positions with
// i >= Wo are computed and dropped (useful fraction Wo/Wq).  Per k2-block the activation bytes that
// cross from L2 to the SM shrink from Kw*16 KB to 16 KB + halo; the filter tiles (one per (k2-block,
// kernel column), streamed through their own ring, or resident when the layer's whole filter
// fits) stay as they were.  Needs s | Wp.  Of the s column classes only those some kernel column reads
// (min(s, Kw)) are copied; a 1x1 layer is then a plain product over full 128-position tiles.
constexpr int MAX_SA = 6, MAX_SB = 12;
constexpr int MAX_KW = 64;                     // kernel widths the shifted-view kernel takes
constexpr int WARP_BLOAD = 2 + EPI_WARPS;      // the filter-copy warp of this kernel
constexpr int SHIFT_THREADS = (NUM_WARPS + 1) * 32;

struct ShiftViewParams {
  EpiParams e;
  uint32_t* status;
  int64_t VQ;                // N*Ho*Wq virtual positions
  int32_t Wq;                // virtual positions per strip
  int32_t s, Kw;
  int32_t rows;              // rows of a sub-tile: 128 + (Kw-1)/s
  uint32_t subt_bytes;       // rows*128 rounded up to 1024
  uint32_t a_stage_bytes;    // s*subt_bytes
  int32_t nkb2;              // 64-wide blocks of k2 = Kh*Cp
  int32_t nks_last;          // 16-wide MMA steps of the last block
  int32_t bu;                // (k2-block, kernel column) units per filter stage
  int32_t sa, sb;            // ring depths
  int32_t resident;          // 1: the filter ring holds the layer's whole filter, loaded once per CTA
  int32_t ksplit, kb_per_split;
  int32_t ntn, nwork;
  int32_t bu_forced;         // testing aid: bu was given, do not choose it
  int32_t dual;              // 1: two MMA-issuing warps, each with half of the activation ring (resident filter only)
  int32_t n_main;            // work items below this index are whole tiles; each whole tile above it is handed out as
  int32_t tail_log2;         // 2^tail_log2 items of BN >> tail_log2 channels (fills the last, short round of tiles)
  int32_t tail_k;            // 1: the tail items split the reduction instead (tail_kb k2-blocks each, all channels):
  int32_t tail_kb;           //    part 0 stores, raises the tile's flag; the others wait for it and add atomically
  uint32_t* flags;           // two words per tail tile (one per CTA of a pair), compared with `epoch`
  uint32_t epoch;            // distinct per launch, so that flags need no clearing between launches
};

// k2-blocks [kb0, kb1) of an item: its K part (ks of q.ksplit), or for a tail part that splits the
// reduction its tail_kb blocks.
__device__ __forceinline__ void item_blocks(const ShiftViewParams& q, int ks, int part, int* kb0, int* kb1) {
  const int per = (part >= 0 && q.tail_k) ? q.tail_kb : q.kb_per_split;     // (part is the constant -1 in kernels without tail items)
  const int first = ((part >= 0 && q.tail_k) ? part : ks) * per;
  *kb0 = first;
  *kb1 = first + per < q.nkb2 ? first + per : q.nkb2;
}

// Work item w of the shifted-view kernel -> whole item index and which part of its channels
// (-1: all of them).
__device__ __forceinline__ void decode_shift_item(const ShiftViewParams& q, int w, int* whole, int* part) {
  if (w < q.n_main) { *whole = w; *part = -1; }
  else { const int t = w - q.n_main; *whole = q.n_main + (t >> q.tail_log2); *part = t & ((1 << q.tail_log2) - 1); }
}

// All MMAs of one full k2-block whose KW kernel columns sit in one filter stage, unrolled for a
// compile-time kernel width (view offsets from registers, filter tiles B16 sixteen-byte units apart):
// the issuing lane then spends a handful of instructions per MMA, which is what narrow tiles need
// (an N = 64 MMA occupies the tensor pipe for 48 cycles only).
template <int KW, bool PAIR>
__device__ __forceinline__ void issue_k2_block(uint32_t acc, uint32_t a_stage, uint32_t b_lo, const uint32_t (&tap)[7],
                                               uint32_t b16, uint32_t idesc, uint32_t& accumulate) {
#pragma unroll
  for (int v = 0; v < KW; ++v) {
#pragma unroll
    for (int t = 0; t < KB / 16; ++t) {
      if (PAIR) umma_f16_ab_pair(acc, a_stage + tap[v] + 2 * t, kSmemDescHiSw128, b_lo + v * b16 + 2 * t, kSmemDescHiSw128, idesc, accumulate);
      else umma_f16_lohi(acc, a_stage + tap[v] + 2 * t, b_lo + v * b16 + 2 * t, idesc, accumulate);
      accumulate = 1u;
    }
  }
}

// TAIL: the launch has items that are parts of a tile (a short last round, see decode_shift_item); without
// them every item is a whole tile and the part handling drops out of the code (layers with very short
// items, a 3x3 stem has six MMAs per item, pay for every instruction in the per-item paths).
template <int BN, bool PAIR, bool TAIL, bool HOIST>
__device__ __forceinline__ void conv_shift_body(const CUtensorMap& amap, const CUtensorMap& bmap, const CUtensorMap& bmap_h,
                                                const CUtensorMap& bmap_q, const ShiftViewParams& q) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  constexpr int NACC = acc_buffers(BN);
  constexpr uint32_t B_BYTES = (uint32_t)B_ROWS * KB * 2;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int w_first = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[2 * MAX_SA + 2 * MAX_SB + 2 * MAX_ACC + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;
  __shared__ uint32_t tap16[MAX_KW];           // view of kernel column v inside an activation stage, in 16-byte units

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t a_ring = smem_u32(smem);
  const uint32_t b_ring = a_ring + (uint32_t)q.sa * q.a_stage_bytes;
  const uint32_t b_stage_bytes = (uint32_t)q.bu * B_BYTES;
  const uint32_t a_full0 = smem_u32(&bars[0]);
  const uint32_t a_empty0 = smem_u32(&bars[MAX_SA]);
  const uint32_t b_full0 = smem_u32(&bars[2 * MAX_SA]);
  const uint32_t b_empty0 = smem_u32(&bars[2 * MAX_SA + MAX_SB]);
  const uint32_t acc_full0 = smem_u32(&bars[2 * MAX_SA + 2 * MAX_SB]);
  const uint32_t acc_empty0 = smem_u32(&bars[2 * MAX_SA + 2 * MAX_SB + MAX_ACC]);
  const uint32_t epi_bar = smem_u32(&bars[2 * MAX_SA + 2 * MAX_SB + 2 * MAX_ACC]);   // rendezvous of the epilogue warps

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    // kernel column v reads sub-tile v mod s from row v div s on
    for (int v = 0; v < q.Kw; ++v) tap16[v] = (uint32_t)(v % q.s) * (q.subt_bytes >> 4) + (uint32_t)(v / q.s) * (KB * 2 >> 4);
    for (int i = 0; i < MAX_SA; ++i) { mbar_init(a_full0 + 8 * i, 1); mbar_init(a_empty0 + 8 * i, 1); }
    for (int i = 0; i < MAX_SB; ++i) { mbar_init(b_full0 + 8 * i, 1); mbar_init(b_empty0 + 8 * i, 1); }
    for (int i = 0; i < MAX_ACC; ++i) {
      mbar_init(acc_full0 + 8 * i, 1);
      mbar_init(acc_empty0 + 8 * i, PAIR ? 2 * EPI_WARPS : EPI_WARPS);
    }
    mbar_init(epi_bar, EPI_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) {
    if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_slot), NACC * BN);
    else tmem_alloc(smem_u32(&tmem_base_slot), NACC * BN);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  const uint32_t a_full_dst = PAIR ? mapa_shared(a_full0, 0) : a_full0;     // the leader's barriers
  const uint32_t b_full_dst = PAIR ? mapa_shared(b_full0, 0) : b_full0;
  const uint32_t acc_empty_dst = PAIR ? mapa_shared(acc_empty0, 0) : acc_empty0;
  const int per_mt = q.ntn * q.ksplit;

  if (warp == WARP_TMA) {
    // ---------------- activation copies: s sub-tiles per k2-block -------------------
    // (the whole warp walks the loops and takes the waits, one elected lane issues)
    {
      const bool leader = elect_one();
      const int ncls = q.s < q.Kw ? q.s : q.Kw;   // column classes some kernel column reads
      wait_for_previous_kernel();
      // with two issuing warps the ring is two rings of half the stages: even items fill one, odd items the other
      const int nst = q.dual ? q.sa / 2 : q.sa;
      int st_even = 0, st_odd = 0;             // (scalars, not an array indexed by the ring: that would live in local memory)
      uint32_t ph_even = 0u, ph_odd = 0u;
      uint32_t it = 0;
      bool ok = true;
      TIMER_DECL;
      for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
        int whole = w, part = -1;
        if (TAIL) decode_shift_item(q, w, &whole, &part);
        const int mt = whole / per_mt, rem = whole - mt * per_mt;
        const int ks = rem % q.ksplit;
        const int q0 = (PAIR ? 2 * mt + (int)rank : mt) * TILE_M;
        int kb0, kb1;
        item_blocks(q, ks, part, &kb0, &kb1);
        const bool odd = q.dual && (it & 1u);
        int stl = odd ? st_odd : st_even;
        uint32_t phl = odd ? ph_odd : ph_even;
        for (int kb = kb0; kb < kb1; ++kb) {
          const int st = (odd ? nst : 0) + stl;
          if (lane == 0) TIMER_LAP(0);                   // activation copies: issuing
          ok = mbar_wait(a_empty0 + 8 * st, phl ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) TIMER_LAP(1);                   // activation copies: wait for a free stage
          if (leader) {
            const uint32_t dst = a_ring + (uint32_t)st * q.a_stage_bytes;
            const uint32_t bar = a_full_dst + 8 * st;
            if (!PAIR || rank == 0)
              mbar_arrive_expect_tx(a_full0 + 8 * st, (PAIR ? 2u : 1u) * (uint32_t)(ncls * q.rows * KB * 2));
            for (int t = 0; t < ncls; ++t) {
              if (PAIR) tma_load_3d_pair(dst + (uint32_t)t * q.subt_bytes, &amap, kb * KB, t, q0, bar);
              else tma_load_3d(dst + (uint32_t)t * q.subt_bytes, &amap, kb * KB, t, q0, bar);
            }
          }
          __syncwarp();
          if (++stl == nst) { stl = 0; phl ^= 1u; }
        }
        if (odd) { st_odd = stl; ph_odd = phl; } else { st_even = stl; ph_even = phl; }
      }
      if (lane == 0 && blockIdx.x == 0) { TIMER_LAP(0); TIMER_FLUSH(); }
    }
  } else if (warp == WARP_BLOAD) {
    // ---------------- filter copies: bu (k2-block, kernel column) units per stage ----
    {
      const bool leader = elect_one();
      wait_for_previous_kernel();
      int st = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int w = w_first; w < q.nwork && ok; w += w_step) {
        int whole = w, part = -1;
        if (TAIL) decode_shift_item(q, w, &whole, &part);
        const int rem = whole % per_mt;
        const int nt = rem / q.ksplit, ks = rem - nt * q.ksplit;
        // filter rows of this CTA: its share of the tile's channels, or of one part of them
        const bool npart = part >= 0 && !q.tail_k;       // a part of the channels (a K part keeps them all)
        const int brow = !npart ? nt * BN + (int)rank * B_ROWS
                                : nt * BN + part * (BN >> q.tail_log2) + (int)rank * (B_ROWS >> q.tail_log2);
        const uint32_t unit_bytes = !npart ? B_BYTES : B_BYTES >> q.tail_log2;
        const CUtensorMap* bm = !npart ? &bmap : (q.tail_log2 == 1 ? &bmap_h : &bmap_q);
        int kb0, kb1;
        item_blocks(q, ks, part, &kb0, &kb1);
        int kb = kb0, v = 0;
        for (int left = (kb1 - kb0) * q.Kw; left > 0 && ok; left -= q.bu) {
          const int nu = left < q.bu ? left : q.bu;             // units of this stage
          ok = mbar_wait(b_empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const uint32_t dst = b_ring + (uint32_t)st * b_stage_bytes;
          const uint32_t bar = b_full_dst + 8 * st;
          if (leader && (!PAIR || rank == 0))
            mbar_arrive_expect_tx(b_full0 + 8 * st, (PAIR ? 2u : 1u) * (uint32_t)nu * unit_bytes);
          for (int j = 0; j < nu; ++j) {
            if (leader) {
              if (PAIR) tma_load_3d_pair(dst + (uint32_t)j * B_BYTES, bm, kb * KB, v, brow, bar);
              else tma_load_3d(dst + (uint32_t)j * B_BYTES, bm, kb * KB, v, brow, bar);
            }
            if (++v == q.Kw) { v = 0; ++kb; }
          }
          __syncwarp();
          if (++st == q.sb) { st = 0; ph ^= 1u; }
        }
        if (q.resident) break;                   // every stage now holds its units for good
      }
    }
  }
  if ((warp == WARP_MMA || (warp == WARP_BLOAD && q.dual)) && rank == 0) {
    // ---------------- MMA issuer ------------------------------------------------------
    // The whole warp walks the loop (waits are taken by every lane), one elected lane issues the
    // MMAs and commits: measured faster than a lone lane, whose satisfied waits cost more.
    // With a resident filter the filter-copy warp is idle after the first item and becomes a second
    // issuer (q.dual): issuer 0 takes the even items, issuer 1 the odd ones, each with its own half of
    // the activation ring and its own accumulators (the accumulator ring has an even length), so the
    // two instruction streams are independent: while one issuer waits for its stages or an accumulator
    // the other keeps the tensor pipe fed (short items of 64-channel layers).
    constexpr uint32_t idesc_whole = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, BN);
    const uint32_t idesc_part = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, 0) | ((uint32_t)((BN >> q.tail_log2) >> 3) << 17);
    {
      const bool leader = elect_one();
      const int mid = warp == WARP_MMA ? 0 : 1;
      const int nroles = q.dual ? 2 : 1;
      const int nst = q.dual ? q.sa / 2 : q.sa;      // activation stages of this issuer
      const int abase = mid * nst;
      int sta = 0, stb = 0;
      uint32_t pha = 0, phb = 0, it = (uint32_t)mid;
      bool ok = true;
      const uint32_t a_lo0 = smem_desc_lo(a_ring), b_lo0 = smem_desc_lo(b_ring);
      const uint32_t astage16 = q.a_stage_bytes >> 4, bstage16 = b_stage_bytes >> 4;
      uint32_t tapr[7];                          // the first seven view offsets in registers (unrolled issue paths)
#pragma unroll
      for (int v = 0; v < 7; ++v) tapr[v] = v < q.Kw ? tap16[v] : 0u;
      TIMER_DECL;
      for (int w = w_first + mid * w_step; w < q.nwork && ok; w += nroles * w_step, it += (uint32_t)nroles) {
        int whole = w, part = -1;
        if (TAIL) decode_shift_item(q, w, &whole, &part);
        const uint32_t idesc = (part < 0 || q.tail_k) ? idesc_whole : idesc_part;
        const int rem = whole % per_mt;
        const int ks = rem % q.ksplit;
        int kb0, kb1;
        item_blocks(q, ks, part, &kb0, &kb1);
        const uint32_t buf = it % (uint32_t)NACC, aph = (it / (uint32_t)NACC) & 1u;
        const bool first_item = it < (uint32_t)nroles;   // this issuer's first item: a resident filter is still arriving
        if (lane == 0) TIMER_LAP(2);                     // MMA warp: issue and bookkeeping
        ok = mbar_wait(acc_empty0 + 8 * buf, aph ^ 1u, &abort_flag, q.status);   // drained by the epilogue
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) TIMER_LAP(3);                     // MMA warp: wait for a free accumulator
        tc_fence_after();
        const uint32_t acc = tmem_acc + buf * (uint32_t)BN;
        uint32_t accumulate = 0;
        if (q.resident) stb = 0;
        if (q.bu == q.Kw) {
          // one filter stage per k2-block (all its kernel columns): two waits and two commits per block
          for (int kb = kb0; kb < kb1; ++kb) {
            if (lane == 0) TIMER_LAP(2);
            ok = mbar_wait(a_full0 + 8 * (abase + sta), pha, &abort_flag, q.status);
            if (ok && !(q.resident && !first_item)) ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) TIMER_LAP(4);               // MMA warp: wait for the stages
            if (leader) {
              const uint32_t a_stage = a_lo0 + (uint32_t)(abase + sta) * astage16;
              uint32_t b_lo = b_lo0 + (uint32_t)stb * bstage16;
              if (kb != q.nkb2 - 1 || q.nks_last == KB / 16) {
                if (q.Kw == 3) issue_k2_block<3, PAIR>(acc, a_stage, b_lo, tapr, B_BYTES >> 4, idesc, accumulate);
                else if (q.Kw == 5) issue_k2_block<5, PAIR>(acc, a_stage, b_lo, tapr, B_BYTES >> 4, idesc, accumulate);
                else if (q.Kw == 7) issue_k2_block<7, PAIR>(acc, a_stage, b_lo, tapr, B_BYTES >> 4, idesc, accumulate);
                else {
                  for (int v = 0; v < q.Kw; ++v) {
                    const uint32_t a_lo = a_stage + tap16[v];
#pragma unroll
                    for (int t = 0; t < KB / 16; ++t) {
                      if (PAIR) umma_f16_ab_pair(acc, a_lo + 2 * t, kSmemDescHiSw128, b_lo + 2 * t, kSmemDescHiSw128, idesc, accumulate);
                      else umma_f16_lohi(acc, a_lo + 2 * t, b_lo + 2 * t, idesc, accumulate);
                      accumulate = 1u;
                    }
                    b_lo += B_BYTES >> 4;
                  }
                }
              } else {
                for (int v = 0; v < q.Kw; ++v) {
                  const uint32_t a_lo = a_stage + tap16[v];
                  for (int t = 0; t < q.nks_last; ++t) {
                    if (PAIR) umma_f16_ab_pair(acc, a_lo + 2 * t, kSmemDescHiSw128, b_lo + 2 * t, kSmemDescHiSw128, idesc, accumulate);
                    else umma_f16_lohi(acc, a_lo + 2 * t, b_lo + 2 * t, idesc, accumulate);
                    accumulate = 1u;
                  }
                  b_lo += B_BYTES >> 4;
                }
              }
              if (PAIR) umma_commit_pair(a_empty0 + 8 * (abase + sta));
              else umma_commit(a_empty0 + 8 * (abase + sta));
              if (!q.resident) {
                if (PAIR) umma_commit_pair(b_empty0 + 8 * stb);
                else umma_commit(b_empty0 + 8 * stb);
              }
            }
            __syncwarp();
            if (++sta == nst) { sta = 0; pha ^= 1u; }
            if (++stb == q.sb) { stb = 0; phb ^= 1u; }
          }
        } else {
        // the item's units (k2-block, kernel column) in order, bu per filter stage
        int kb = kb0, v = 0;
        uint32_t a_stage = 0;
        int nks = KB / 16;
        for (int left = (kb1 - kb0) * q.Kw; left > 0 && ok; left -= q.bu) {
          const int nu = left < q.bu ? left : q.bu;
          if (!(q.resident && !first_item)) {    // a resident filter is complete after the first item
            if (lane == 0) TIMER_LAP(2);
            ok = mbar_wait(b_full0 + 8 * stb, phb, &abort_flag, q.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) TIMER_LAP(7);                 // MMA warp: wait for a filter stage
          }
          uint32_t b_lo = b_lo0 + (uint32_t)stb * bstage16;
          for (int j = 0; j < nu; ++j) {
            if (v == 0) {
              if (lane == 0) TIMER_LAP(2);
              ok = mbar_wait(a_full0 + 8 * sta, pha, &abort_flag, q.status);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              if (lane == 0) TIMER_LAP(4);               // MMA warp: wait for an activation stage
              a_stage = a_lo0 + (uint32_t)sta * astage16;
              nks = kb == q.nkb2 - 1 ? q.nks_last : KB / 16;
            }
            if (leader) {
              const uint32_t a_lo = a_stage + tap16[v];
#pragma unroll
              for (int t = 0; t < KB / 16; ++t) {
                if (t < nks) {
                  if (PAIR) umma_f16_ab_pair(acc, a_lo + 2 * t, kSmemDescHiSw128, b_lo + 2 * t, kSmemDescHiSw128, idesc, accumulate);
                  else umma_f16_lohi(acc, a_lo + 2 * t, b_lo + 2 * t, idesc, accumulate);
                  accumulate = 1u;
                }
              }
            }
            b_lo += B_BYTES >> 4;
            if (++v == q.Kw) {
              v = 0; ++kb;
              if (leader) {
                if (PAIR) umma_commit_pair(a_empty0 + 8 * sta);
                else umma_commit(a_empty0 + 8 * sta);
              }
              if (++sta == q.sa) { sta = 0; pha ^= 1u; }
            }
          }
          if (!ok) break;
          if (leader && !q.resident) {
            if (PAIR) umma_commit_pair(b_empty0 + 8 * stb);
            else umma_commit(b_empty0 + 8 * stb);
          }
          __syncwarp();
          if (++stb == q.sb) { stb = 0; phb ^= 1u; }
        }
        }
        if (ok && leader) {
          if (PAIR) umma_commit_pair(acc_full0 + 8 * buf);
          else umma_commit(acc_full0 + 8 * buf);
        }
        __syncwarp();
      }
      if (lane == 0 && blockIdx.x == 0 && mid == 0) { TIMER_LAP(2); TIMER_FLUSH(); }
    }
  }
  if (warp >= WARP_EPI0 && warp < WARP_EPI0 + EPI_WARPS) {
    // ---------------- epilogue ----------------------------------------------------------
    const int lq = warp & 3;
    const EpiParams& e = q.e;
    const bool vec_ok = e.out16 ? (e.Co % 8 == 0) : (e.Co % 4 == 0);
    wait_for_previous_kernel();
    // HOIST (64-channel tiles, one channel tile, a bias): the warp's 32 bias values stay in registers.  A
    // kernel of its own: the same choice taken at run time cost the stems without a bias 8-15 %.
    float breg[HOIST ? 32 : 1];
    if (HOIST) {
      const int c0 = ((warp - WARP_EPI0) >> 2) * 32;
#pragma unroll
      for (int t = 0; t < (HOIST ? 32 : 1); ++t) breg[t] = c0 + t < e.Co ? __ldg(e.bias + c0 + t) : 0.0f;
    }
    bool ok = true;
    uint32_t it = 0, epi_phase = 0;
    TIMER_DECL;
    for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
      const uint32_t buf = it % (uint32_t)NACC, aph = (it / (uint32_t)NACC) & 1u;
      int whole = w, part = -1;
      if (TAIL) decode_shift_item(q, w, &whole, &part);
      const int mt = whole / per_mt, rem = whole - mt * per_mt;
      const int nt = rem / q.ksplit, ks = rem - nt * q.ksplit;
      const bool kpart = TAIL && q.tail_k && part >= 0;        // a tail item that holds one K part of all channels
      const int n0 = nt * BN + ((part > 0 && !kpart) ? part * (BN >> q.tail_log2) : 0);
      const int cols = (part < 0 || kpart) ? BN : BN >> q.tail_log2;
      // accumulator row = virtual position vq = strip*Wq + i; columns i >= Wo of a strip are no output
      const int64_t vq = (int64_t)(PAIR ? 2 * mt + (int)rank : mt) * TILE_M + lq * 32 + lane;
      bool valid = false;
      int64_t base = 0, cs = 1;
      if (vq < q.VQ) {
        const int strip = (int)(vq / q.Wq), i = (int)(vq - (int64_t)strip * q.Wq);
        valid = i < e.Wo;
        if (e.y_nhwc) {
          base = ((int64_t)strip * e.Wo + i) * e.Co + n0;
        } else {
          const int n = strip / e.Ho, ho = strip - n * e.Ho;
          cs = e.HoWo;
          base = ((int64_t)n * e.Co + n0) * e.HoWo + ho * e.Wo + i;
        }
      }
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(5);     // epilogue: draining and storing
      if (lane == 0) ok = mbar_wait(acc_full0 + 8 * buf, aph, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if (!ok) break;
      if (threadIdx.x == WARP_EPI0 * 32) TIMER_LAP(6);     // epilogue: wait for a finished accumulator
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + buf * (uint32_t)BN + ((uint32_t)(lq * 32) << 16);
      // K parts of a tail tile: part 0 stores (with the bias) and then raises this CTA's flag of the
      // tile; the other parts wait for that flag and add their sums with red.global.add.f32
      uint32_t* flag = q.flags + 2 * (whole - q.n_main) + (PAIR ? (int)rank : 0);
      const bool adds = kpart && part > 0;
      if (adds) {
        if (lane == 0) ok = wait_flag(flag, q.epoch, &abort_flag, q.status);
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        __syncwarp();
      }
      if (ok) drain_accumulator(e, cols, warp, lane, lane_base, valid, base, cs, n0, kpart ? part == 0 : ks == 0, vec_ok, adds,
                                HOIST ? breg : nullptr);
      if (kpart && part == 0) {
        publish_when_all_stored(epi_bar, epi_phase, warp, lane, flag, q.epoch, &abort_flag, q.status);
        epi_phase ^= 1u;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(acc_empty_dst + 8 * buf);
        else mbar_arrive(acc_empty0 + 8 * buf);
      }
    }
    if (threadIdx.x == WARP_EPI0 * 32 && blockIdx.x == 0) { TIMER_LAP(5); TIMER_FLUSH(); }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);     // copies in flight land before the CTA leaves
    __syncthreads();
  }
  if (PAIR) cluster_sync_all();
  if (warp == WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_acc, NACC * BN);
    else tmem_dealloc(tmem_acc, NACC * BN);
  }
}

template <int BN, bool TAIL, bool HOIST>
__global__ void __launch_bounds__(SHIFT_THREADS, 1)
conv_f16_nhwc_shift_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
                           const __grid_constant__ CUtensorMap bmap_h, const __grid_constant__ CUtensorMap bmap_q,
                           ShiftViewParams q) {
  conv_shift_body<BN, false, TAIL, HOIST>(amap, bmap, bmap_h, bmap_q, q);
}

template <int BN, bool TAIL, bool HOIST>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(SHIFT_THREADS, 1)
conv_f16_nhwc_shift_pair_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap,
                                const __grid_constant__ CUtensorMap bmap_h, const __grid_constant__ CUtensorMap bmap_q,
                                ShiftViewParams q) {
  conv_shift_body<BN, true, TAIL, HOIST>(amap, bmap, bmap_h, bmap_q, q);
}

// Filter pack (paper Section "Im2win Convolution": height before width; here with the channel below
// both): fp[co][(v*Kh + u)*Cp + c] = f[co][c][u][v], zeros for c >= C.  One block takes one output
// channel and a run of `cb` input channels: their cb*Kh*Kw halves are contiguous in the OIHW filter
// (coalesced reads into shared memory) and leave as Kh*Kw runs of cb channels (coalesced writes).
// Block (0, 0) also clears the status block.
__global__ void __launch_bounds__(256)
pack_f16_nhwc_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp, uint32_t* status, uint32_t* flags,
                     int C, int Cp, int Co, int Kh, int Kw, int cb) {
  extern __shared__ __align__(16) uint16_t pack_s[];   // [cb][T], after up to 8 halves of phase padding
  // the convolution that follows in the stream may be launched now: its set-up overlaps this kernel,
  // and every role of it that touches memory first waits for this grid to have completed
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    if (threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
    for (int i = threadIdx.x; i < kTailFlagBytes / 4; i += blockDim.x) flags[i] = 0u;
  }
  const int T = Kh * Kw;
  const int64_t K = (int64_t)T * Cp;
  const int c0 = blockIdx.x * cb;
  const int nc = Cp - c0 < cb ? Cp - c0 : cb;     // stored channels of this block (Cp and cb are multiples of 8)
  const int nreal = C - c0 < nc ? (C - c0 > 0 ? C - c0 : 0) : nc;
  const int pairs = nc / 2;
  int ncc_log2 = 0;
  while ((1 << ncc_log2) < pairs && (1 << ncc_log2) < (int)blockDim.x) ++ncc_log2;
  const int ncc = 1 << ncc_log2, ntt = (int)blockDim.x >> ncc_log2;   // blockDim.x is a power of two
  for (int co = blockIdx.y; co < Co; co += gridDim.y) {
    const uint16_t* src = f + ((int64_t)co * C + c0) * T;
    // the run is read with 16-byte loads from the first 16-byte boundary on (shared-memory copy kept at
    // the same phase), four loads in flight per thread; the ragged ends element by element
    const int n = nreal * T;
    const int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(src) & 15u)) & 15u) >> 1);   // halves before the boundary
    uint16_t* dst = pack_s + 8 - head;              // dst + head is 16-byte aligned (pack_s is)
    const int nvec = n > head ? (n - head) / 8 : 0;
    for (int i = threadIdx.x; i < (n < head ? n : head); i += blockDim.x) dst[i] = __ldg(src + i);
    for (int i = head + nvec * 8 + threadIdx.x; i < n; i += blockDim.x) dst[i] = __ldg(src + i);
    const uint4* vsrc = reinterpret_cast<const uint4*>(src + head);
    uint4* vdst = reinterpret_cast<uint4*>(dst + head);
    for (int i0 = threadIdx.x; i0 < nvec; i0 += 4 * blockDim.x) {
      uint4 r[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + j * (int)blockDim.x < nvec) r[j] = __ldg(vsrc + i0 + j * blockDim.x);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + j * (int)blockDim.x < nvec) vdst[i0 + j * blockDim.x] = r[j];
    }
    const uint16_t* ps = dst;                       // element i of the run is ps[i]
    __syncthreads();
    // 4-byte stores (a channel pair each), consecutive threads along c.  The threads form ntt rows of
    // ncc (a power of two): a row walks t = v*Kh + u in steps of ntt, its threads the channel pairs;
    // (v, u) advance by additions, so that the loop holds no division.
    {
      uint32_t* out_co = reinterpret_cast<uint32_t*>(fp + (int64_t)co * K + c0);
      const int tx = (int)threadIdx.x & (ncc - 1), ty = (int)threadIdx.x >> ncc_log2;
      const int dv = ntt / Kh, du = ntt - dv * Kh;
      int v = ty / Kh, u = ty - v * Kh;
      for (int t = ty; t < T; t += ntt) {
        const uint16_t* pt = ps + u * Kw + v;
        uint32_t* orow = out_co + ((t * Cp) >> 1);
        for (int cp2 = tx; cp2 < pairs; cp2 += ncc) {
          const int c = 2 * cp2;
          const uint32_t lo = c < nreal ? pt[c * T] : 0u;
          const uint32_t hi = c + 1 < nreal ? pt[(c + 1) * T] : 0u;
          orow[cp2] = lo | (hi << 16);
        }
        u += du; v += dv;
        if (u >= Kh) { u -= Kh; ++v; }
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------- transform ----
template <int VEC> struct VecType;
template <> struct VecType<8> { typedef uint4 type; };
template <> struct VecType<4> { typedef uint2 type; };
template <> struct VecType<2> { typedef uint32_t type; };
template <> struct VecType<1> { typedef uint16_t type; };

// x given NHWC: every (n, ho, k, u) of the window tensor is the channel vector of one input pixel
// (or zeros in the padding): 16-byte chunks, one per thread, consecutive threads along (k, u, c).
__global__ void transform_nhwc_from_nhwc_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ win, int C, int Cp,
                                                int H, int W, int Ho, int Wp, int Kh, int s, int p, int64_t chunks) {
  const int c8n = Cp / 8;
  const bool vec = (C % 8) == 0;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < chunks; idx += (int64_t)gridDim.x * blockDim.x) {
    int64_t t = idx;
    const int c8 = (int)(t % c8n); t /= c8n;
    const int u = (int)(t % Kh); t /= Kh;
    const int k = (int)(t % Wp); t /= Wp;
    const int ho = (int)(t % Ho);
    const int64_t n = t / Ho;
    const int h = ho * s + u - p, w = k - p;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (h >= 0 && h < H && w >= 0 && w < W) {
      const uint16_t* src = x + ((n * H + h) * W + w) * C + c8 * 8;
      if (vec) {
        val = __ldg(reinterpret_cast<const uint4*>(src));
      } else {
        uint16_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = c8 * 8 + i < C ? __ldg(src + i) : (uint16_t)0;
        val = make_uint4(e[0] | ((uint32_t)e[1] << 16), e[2] | ((uint32_t)e[3] << 16), e[4] | ((uint32_t)e[5] << 16),
                         e[6] | ((uint32_t)e[7] << 16));
      }
    }
    reinterpret_cast<uint4*>(win)[idx] = val;
  }
}

// x given NHWC: one block per strip (n, ho).  A thread takes 16-byte chunk i of the padded row (column
// k = i / c8n, channels 8 (i % c8n) ..) and copies it from each of the strip's Kh input rows to
// window[(k*Kh + u)*Cp + ...]: along a row the reads of consecutive threads are contiguous, the Kh loads of a
// thread are independent, and its Kh stores complete a run of Kh*Cp halves; the only index arithmetic per
// chunk is the split of i (a shift when Cp/8 is a power of two).  The chunk-per-thread kernel above pays five
// 64-bit divisions per chunk and reached 0.39-0.54 of the copy rate where this one is used now (C a multiple
// of 8: 0.65-0.87 on layers of 80 MB and more).
template <bool POW2>
__global__ void __launch_bounds__(256)
transform_nhwc_from_nhwc_strip_kernel(const uint16_t* __restrict__ x, uint4* __restrict__ win, int C, int c8n, int sh,
                                      int H, int W, int Ho, int Wp, int Kh, int s, int p) {
  const int strip = blockIdx.x;                  // n*Ho + ho
  const int n = strip / Ho, ho = strip - n * Ho;
  uint4* out = win + (int64_t)strip * Wp * Kh * c8n;
  const int row_chunks = Wp * c8n;
  const int h0 = ho * s - p;
  const uint16_t* ximg = x + (int64_t)n * H * W * C;
  for (int i = threadIdx.x; i < row_chunks; i += 256) {
    const int k = POW2 ? i >> sh : i / c8n;
    const int c8 = i - k * c8n;
    const int w = k - p;
    const bool colok = w >= 0 && w < W;
    uint4* o = out + (int64_t)k * Kh * c8n + c8;
#pragma unroll 4
    for (int u = 0; u < Kh; ++u) {
      const int h = h0 + u;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (colok && h >= 0 && h < H) {
        const uint16_t* src = ximg + ((int64_t)h * W + w) * C + c8 * 8;
        v = __ldg(reinterpret_cast<const uint4*>(src));
      }
      o[u * c8n] = v;
    }
  }
}

// x given NHWC with fewer than 8 channels (Cp = 8: every pixel becomes one 16-byte chunk): one block per
// strip.  The strip's Kh input rows (W*C halves each, contiguous) are staged in shared memory with coalesced
// 2-byte loads; then thread j builds chunk j = k*Kh + u of the strip from the C halves of pixel (u, k - p)
// and the block writes the strip as one contiguous run.
__global__ void __launch_bounds__(256)
transform_nhwc_from_nhwc_small_c_kernel(const uint16_t* __restrict__ x, uint4* __restrict__ win, int C, int H, int W,
                                        int Ho, int Wp, int Kh, int s, int p) {
  extern __shared__ __align__(16) uint16_t px_s[];        // [Kh][W*C]
  const int strip = blockIdx.x;
  const int n = strip / Ho, ho = strip - n * Ho;
  const int h0 = ho * s - p;
  const int row = W * C;
  for (int u = 0; u < Kh; ++u) {
    const int h = h0 + u;
    if (h < 0 || h >= H) continue;                 // (uniform per block; such rows are never read below)
    const uint16_t* src = x + ((int64_t)n * H + h) * row;
    for (int i = threadIdx.x; i < row; i += 256) px_s[u * row + i] = __ldg(src + i);
  }
  __syncthreads();
  uint4* out = win + (int64_t)strip * Wp * Kh;
  const int chunks = Wp * Kh;
  for (int j = threadIdx.x; j < chunks; j += 256) {
    const int k = j / Kh, u = j - k * Kh;
    const int w = k - p, h = h0 + u;
    uint16_t e[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (w >= 0 && w < W && h >= 0 && h < H) {
      const uint16_t* px = px_s + u * row + w * C;
#pragma unroll
      for (int t = 0; t < 8; ++t)
        if (t < C) e[t] = px[t];
    }
    out[j] = make_uint4(e[0] | ((uint32_t)e[1] << 16), e[2] | ((uint32_t)e[3] << 16), e[4] | ((uint32_t)e[5] << 16),
                        e[6] | ((uint32_t)e[7] << 16));
  }
}

// x given NCHW: a transposition.  One block takes one row h of the padded input of one image (all
// channels, a chunk of columns when the row is long): phase 1 reads it along w (coalesced) and
// stores it in shared memory as T[w][c] (pitch Cp + 2 halves = an odd number of words:
// conflict-free); phase 2 writes T to every place of the window tensor that holds this input row,
// i.e. once per (ho, u) with ho*s + u = h + p (Kh/s places): 16-byte chunks in output order (c
// fastest), so consecutive threads write consecutive bytes of a column.  Every input element is
// read once and transposed once; blocks of rows outside the image only write zeros.  Indices are
// kept in mixed-radix counters (no division per element).
// SWZ (Cp/8 a power of two): rows of T are Cp halves apart (no padding) and the 16-byte chunk c8 of row r sits at
// chunk c8 ^ ((r / VEC) & 7): the transposing stores of a warp (lanes on different column groups) still spread
// over the banks, and phase 2 reads a chunk with ONE 16-byte load and finds (k, chunk) with a shift and a mask
// (with the odd pitch Cp + 2 a chunk is only 4-byte aligned: four loads, and mixed-radix counters per chunk).
template <int VEC, bool SWZ>
__global__ void __launch_bounds__(256)
transform_nhwc_from_nchw_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ win, int C, int Cp, int H, int W,
                                int Ho, int Wp, int Kh, int s, int p, int kc, int kchunks, int R, int rgroups) {
  extern __shared__ __align__(16) uint16_t rows_s[];     // T[kc][Cp + 2], or (SWZ) T[kc][Cp] with swizzled chunks
  const int PC = SWZ ? Cp : Cp + 2;
  const int smask = SWZ ? ((Cp / 8 < 8 ? Cp / 8 : 8) - 1) : 0;
  // element index of channel c of row r in T
  auto tidx = [&](int r, int c) { return SWZ ? r * PC + ((((c >> 3) ^ ((r / VEC) & smask)) << 3) | (c & 7)) : r * PC + c; };
  // block -> (image n, group of R consecutive rows of the padded input, column chunk); 32-bit
  // arithmetic (the host keeps the block count below 2^31): the set-up is paid by every thread of
  // every block, and a block's own work is only a few instructions per thread and row
  uint32_t b = blockIdx.x;
  const int kci = (int)(b % (uint32_t)kchunks); b /= (uint32_t)kchunks;
  const int rg = (int)(b % (uint32_t)rgroups);
  const int64_t n = b / (uint32_t)rgroups;
  const int w0 = kci * kc;
  const int nw = W - w0 < kc ? W - w0 : kc;               // input columns of this block
  // its columns of the window tensor: k = w + p, plus the left padding for the first chunk and the
  // right padding for the last
  const int k_lo = kci == 0 ? 0 : w0 + p;
  const int k_hi = kci == kchunks - 1 ? Wp : w0 + nw + p; // exclusive
  const int step = (int)blockDim.x;
  // phase 1 counters: item -> (channel pair, group of VEC columns), columns fastest
  typedef typename VecType<VEC>::type V;
  const int nwi = nw / VEC;
  const int cpairs = (C + 1) / 2;
  const int items = cpairs * nwi;
  const int d_c = step / nwi, d_col = step - d_c * nwi;
  const int cp_first = (int)threadIdx.x / nwi, col_first = (int)threadIdx.x - cp_first * nwi;
  const int64_t cstride = (int64_t)H * W;
  // phase 2 counters: chunk j = (k - k_lo)*octs + oct
  const int octs = Cp / 8;
  const int chunks = (k_hi - k_lo) * octs;
  const int d_k = step / octs, d_o = step - d_k * octs;
  const int k_first = k_lo + (int)threadIdx.x / octs, oct_first = (int)threadIdx.x % octs;

  const int hp_end = (rg + 1) * R < H + 2 * p ? (rg + 1) * R : H + 2 * p;
  for (int hp = rg * R; hp < hp_end; ++hp) {              // row of the padded input
    const int h = hp - p;
    const bool row_ok = h >= 0 && h < H;
    // the strips that hold this row: ho*s + u = hp with 0 <= u < Kh
    const int ho_hi = hp / s < Ho - 1 ? hp / s : Ho - 1;
    const int ho_lo = hp - Kh + 1 > 0 ? (hp - Kh + 1 + s - 1) / s : 0;
    if (ho_lo > ho_hi) continue;                          // a row no window reaches (the same for every thread)
    __syncthreads();                                      // the row before has been written out
    if (row_ok) {
      if (Cp > C) {                                       // the zero channels C .. Cp-1 (an odd C's last pair store
                                                          // writes a zero to channel C as well: same value)
        const int extra = Cp - C;
        for (int i = threadIdx.x; i < nw * extra; i += step) {
          const int r = i / extra, e = i - r * extra;
          rows_s[tidx(r, C + e)] = 0;
        }
      }
      // phase 1 (W, w0 and nw are multiples of VEC): two VEC*2-byte loads (the second channel's only
      // when it exists), VEC transposing 4-byte stores of a channel pair each; two items in flight
      int cp = cp_first, col = col_first;
      const uint16_t* xrow = x + ((n * C) * H + h) * (int64_t)W + w0;    // channel c: + c*H*W
      for (int i0 = threadIdx.x; i0 < items; i0 += 2 * step) {
        V r0[2], r1[2];
        int dsts[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          dsts[j] = -1;
          if (i0 + j * step < items) {
            const int c = 2 * cp;
            dsts[j] = tidx(VEC * col, c);            // (rows VEC*col .. + VEC - 1 share the swizzle: + t*PC below)
            const uint16_t* src = xrow + c * cstride + VEC * col;
            r0[j] = __ldg(reinterpret_cast<const V*>(src));
            if (c + 1 < C) r1[j] = __ldg(reinterpret_cast<const V*>(src + cstride));
            else memset(&r1[j], 0, sizeof(V));
          }
          col += d_col; cp += d_c;
          if (col >= nwi) { col -= nwi; ++cp; }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          if (dsts[j] >= 0) {
            const uint16_t* e0 = reinterpret_cast<const uint16_t*>(&r0[j]);
            const uint16_t* e1 = reinterpret_cast<const uint16_t*>(&r1[j]);
#pragma unroll
            for (int t = 0; t < VEC; ++t)
              *reinterpret_cast<uint32_t*>(rows_s + dsts[j] + t * PC) = (uint32_t)e0[t] | ((uint32_t)e1[t] << 16);
          }
        }
      }
    }
    __syncthreads();
    // phase 2: for every (ho, u) that holds the row
    for (int ho = ho_lo; ho <= ho_hi; ++ho) {
      const int u = hp - ho * s;
      // chunk (k, oct) of strip (n, ho): ((k*Kh + u)*Cp + 8*oct) halves into the strip
      uint16_t* strip = win + ((n * Ho + ho) * (int64_t)Wp) * Kh * Cp + (int64_t)u * Cp;
      if (SWZ) {
        const int lo = 31 - __clz(octs);                  // octs is a power of two
        for (int j = threadIdx.x; j < chunks; j += step) {
          const int k = k_lo + (j >> lo), oct = j & (octs - 1);
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          const int r = k - p - w0;
          if (row_ok && r >= 0 && r < nw) v = *reinterpret_cast<const uint4*>(rows_s + tidx(r, 8 * oct));
          *reinterpret_cast<uint4*>(strip + (int64_t)k * Kh * Cp + 8 * oct) = v;
        }
      } else {
      int k = k_first, oct = oct_first;
      for (int j = threadIdx.x; j < chunks; j += step) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        const int w = k - p;
        if (row_ok && w >= w0 && w < w0 + nw) {
          const uint32_t* src = reinterpret_cast<const uint32_t*>(rows_s + (w - w0) * PC + 8 * oct);
          v = make_uint4(src[0], src[1], src[2], src[3]);
        }
        *reinterpret_cast<uint4*>(strip + (int64_t)k * Kh * Cp + 8 * oct) = v;
        oct += d_o; k += d_k;
        if (oct >= octs) { oct -= octs; ++k; }
      }
      }
    }
  }
}

// x given NCHW with at most 8 channels (Cp = 8, the 3-channel stems): a column of the window tensor is
// one 16-byte chunk per (k, u), and the per-row kernel above would scatter such chunks Kh*16 bytes
// apart.  Here one block builds one whole strip (n, ho) in shared memory in output order and writes
// it out as one contiguous run.  The input rows a strip needs are, per channel, one contiguous run
// of the input (rows ho*s - p .. + Kh - 1, clipped to the image): the C runs are brought into a
// staging area with 16-byte loads from their first 16-byte boundary on (all in flight together; a
// run is read by the Kh/s strips that hold its rows, from L2 after the first), then scattered inside
// shared memory to S[k][u][c]; everything else (padding, channels C..7) stays zero.  A column of S is
// PW = 4*Kh + 1 words apart, an odd number, so that the scatter and the read-out spread over the
// banks.
__global__ void __launch_bounds__(256)
transform_nhwc_strip_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ win, int C, int H, int W, int Ho,
                            int Wp, int Kh, int s, int p, int SP) {
  extern __shared__ __align__(16) uint32_t strip_s[];     // [Wp][PW] words, then the staging area [C][SP] halves
  const int PW = 4 * Kh + 1;
  const int strip_words = (Wp * PW + 3) & ~3;
  uint16_t* stage = reinterpret_cast<uint16_t*>(strip_s + strip_words);
  const int64_t n = blockIdx.x / Ho;
  const int ho = (int)(blockIdx.x - n * Ho);
  // rows of the image this strip holds: u_lo .. u_hi of its Kh rows
  const int h0 = ho * s - p;
  const int u_lo = h0 < 0 ? -h0 : 0;
  const int u_hi = h0 + Kh - 1 < H ? Kh - 1 : H - 1 - h0;
  const int L = (u_hi - u_lo + 1) * W;                    // halves per channel run (<= 0: none)
  const int NV = L > 0 ? L / 8 + 1 : 0;                   // 16-byte pieces a run may span after its head
  const int step = (int)blockDim.x;
  const uint16_t* run0 = x + ((n * C) * H + (h0 + u_lo)) * (int64_t)W;         // channel c: + c*H*W
  const int64_t cstride = (int64_t)H * W;
  // halves before the first 16-byte boundary of channel c's run
  const int ph0 = (int)((reinterpret_cast<uintptr_t>(run0) >> 1) & 7u), cs7 = (int)(cstride & 7);
  auto head_of = [&](int c) { return (8 - ((ph0 + c * cs7) & 7)) & 7; };
  if (L > 0) {
    // 16-byte pieces, four in flight per thread: item -> (c, piece)
    for (int i0 = threadIdx.x; i0 < C * NV; i0 += 4 * step) {
      uint4 r[4];
      int dsts[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        dsts[j] = -1;
        const int i = i0 + j * step;
        if (i < C * NV) {
          const int c = i / NV, v = i - c * NV;
          const uint16_t* src = run0 + c * cstride;
          const int head = head_of(c);
          if (head + 8 * v + 8 <= L) {
            dsts[j] = c * SP + 8 + 8 * v;                 // the staged run keeps the phase: element e at c*SP + 8 - head + e
            r[j] = __ldg(reinterpret_cast<const uint4*>(src + head + 8 * v));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (dsts[j] >= 0) *reinterpret_cast<uint4*>(stage + dsts[j]) = r[j];
    }
    // the ragged ends of every run, element by element: at most 7 + 7 halves per channel
    for (int i = threadIdx.x; i < C * 16; i += step) {
      const int c = i >> 4, e = i & 15;
      const uint16_t* src = run0 + c * cstride;
      const int head = head_of(c);
      const int nvec = L > head ? (L - head) / 8 : 0;
      int idx = -1;
      if (e < 8) { if (e < head && e < L) idx = e; }                        // before the boundary
      else { const int t = head + 8 * nvec + (e - 8); if (t < L && t >= head) idx = t; }   // after the last whole piece
      if (idx >= 0) stage[c * SP + 8 - head + idx] = __ldg(src + idx);
    }
  }
  {
    const int total = Wp * PW, quads = total / 4;
    for (int i = threadIdx.x; i < quads; i += step) reinterpret_cast<uint4*>(strip_s)[i] = make_uint4(0u, 0u, 0u, 0u);
    for (int i = 4 * quads + threadIdx.x; i < total; i += step) strip_s[i] = 0u;
  }
  __syncthreads();
  // scatter inside shared memory: a warp takes the rows (c, u) in turn, its lanes walk the columns
  if (L > 0) {
    uint16_t* sh = reinterpret_cast<uint16_t*>(strip_s);
    const int rows = u_hi - u_lo + 1;
    const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31, nwarps = step >> 5;
    for (int c = 0; c < C; ++c) {
      const uint16_t* src_c = stage + c * SP + 8 - head_of(c);       // element 0 of channel c's run
      for (int r = warp; r < rows; r += nwarps) {
        const uint16_t* src = src_c + r * W;
        uint16_t* dst = sh + (p * PW + 4 * (r + u_lo)) * 2 + c;
        for (int w = lane; w < W; w += 32) dst[w * PW * 2] = src[w];
      }
    }
  }
  __syncthreads();
  // read-out: chunk j = k*Kh + u of the strip, consecutive threads consecutive chunks
  {
    uint4* dst = reinterpret_cast<uint4*>(win + (n * Ho + ho) * (int64_t)Wp * Kh * 8);
    const int chunks = Wp * Kh;
    const int d_k = step / Kh, d_u = step - d_k * Kh;
    int k = (int)threadIdx.x / Kh, u = (int)threadIdx.x - k * Kh;
    for (int j = threadIdx.x; j < chunks; j += step) {
      const uint32_t* src = strip_s + k * PW + 4 * u;
      dst[j] = make_uint4(src[0], src[1], src[2], src[3]);
      u += d_u; k += d_k;
      if (u >= Kh) { u -= Kh; ++k; }
    }
  }
}

// ------------------------------------------------------------------- host side
// Testing aid: with IM2WIN_DEBUG and IM2WIN_VERBOSE set, a failed host-side step says what failed.
cudaError_t report(cudaError_t e, const char* what) {
  if (e != cudaSuccess && debug_getenv("IM2WIN_VERBOSE")) fprintf(stderr, "im2win nhwc: %s: %s\n", what, cudaGetErrorString(e));
  return e;
}

// A value no earlier launch of this process used (flag words are compared with it and need no clearing).
uint32_t next_epoch() {
  static std::atomic<uint32_t> launches{0};
  uint32_t e = ++launches;
  if (e == 0) e = ++launches;                   // 0 is what cleared flags hold
  return e;
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

// Overlapping-row kernel, a short last round of tiles: the reductions of its `tiles` tiles are laid end to
// end and cut into equal runs of `u` chunks (of ksub k-blocks), one per CTA (pair) for the first `ctas` of
// them.  The CTA that holds a tile's first chunk adds the others' partial sums (scratch area, one flag per
// CTA) and stores the tile, so bias, ReLU and the rounding store work as for whole tiles.  At most eight
// runs per tile (their sums are added one after another) and no run shorter than eight k-blocks.
// tiles == 0: not worth it; `rounds` is the estimated time of the launch in tile times.
struct RunPlan {
  int tiles, u, ctas;
  double rounds;
};

RunPlan plan_runs(int64_t nwork, int slots, int num_kc, int ksub, int bn) {
  RunPlan r{};
  bool on = bn >= 128;                                      // 64-channel tiles: items too short to share
  if (const char* v = debug_getenv("IM2WIN_NHWC_STREAM")) on = on && v[0] != '0';
  const int tail = (int)(nwork % slots);
  // what the round takes otherwise: a whole tile, or about 0.55 of one as half tiles
  const double alt = tail == 0 ? 0.0 : ((bn >= 128 && 2 * tail <= slots) ? 0.55 : 1.0);
  r.rounds = (double)(nwork / slots) + alt;
  if (!on || tail == 0) return r;
  const int min_run = (num_kc + 7) / 8 > 8 / ksub ? (num_kc + 7) / 8 : 8 / ksub;
  const int64_t total = (int64_t)tail * num_kc;
  if (total >= ((int64_t)1 << 30)) return r;             // (the kernel indexes the runs with 32-bit integers)
  int S = slots;
  if (total / S < min_run) S = (int)(total / min_run);
  if (S <= tail) return r;
  const int U = (int)((total + S - 1) / S);
  S = (int)((total + U - 1) / U);
  // Worth it when the run, plus the two drains that now follow one another at the end (a partial sum
  // written, then read by the tile's owner: measured about 24 k-blocks' time together), is clearly
  // shorter.  (Measured on 3x3 layers of 256 and 512 channels, 36 and 72 k-blocks per tile: 3 to 8 us
  // slower than half tiles; on 7x7 and 11x11 layers of 256 channels with a ReLU and a binary16 store:
  // 281 -> 258 us and 717 -> 626 us.)
  double margin = 24.0 / ((double)num_kc * ksub) + 0.05;
  if (const char* v = debug_getenv("IM2WIN_NHWC_STREAM_MARGIN")) margin = atof(v);
  if (U >= num_kc || (double)U / num_kc + margin >= alt) return r;
  r.tiles = tail; r.u = U; r.ctas = S;
  r.rounds = (double)(nwork / slots) + (double)U / num_kc + margin;
  return r;
}

template <int BN, bool PAIR, int KSUB>
cudaError_t launch_variant(const CUtensorMap& amap, const CUtensorMap& bmap, const CUtensorMap& bmap_h, NhwcParams q,
                           const NhwcPlan& plan, cudaStream_t stream) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  constexpr int STAGE = KSUB * (A_SLOT_BYTES + B_ROWS * KB * 2);
  int stages = (kSmemMax - 2048) / STAGE;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return cudaErrorInvalidValue;
  if (const char* v = debug_getenv("IM2WIN_NHWC_STAGES")) { const int n = atoi(v); if (n >= 2 && n < stages) stages = n; }   // ablation: ring depth
  q.stages = stages;
  // K in chunks of KSUB k-blocks; a K split hands out whole chunks
  q.num_kc = (plan.num_kb + KSUB - 1) / KSUB;
  q.nks_last = (int32_t)((plan.K - (int64_t)(q.num_kc - 1) * KSUB * KB + 15) / 16);
  q.kc_per_split = (q.num_kc + q.ksplit - 1) / q.ksplit;
  q.ksplit = (q.num_kc + q.kc_per_split - 1) / q.kc_per_split;
  const int64_t ntm_eff = PAIR ? (plan.ntm + 1) / 2 : plan.ntm;
  const int64_t nwork = ntm_eff * q.ntn * q.ksplit;
  if (nwork >= ((int64_t)1 << 30)) return cudaErrorInvalidValue;
  q.ntm_eff = (int32_t)ntm_eff;
  q.raster = 0;
  if (const char* v = debug_getenv("IM2WIN_NHWC_RASTER")) q.raster = v[0] == '1';     // ablation: item order
  q.nwork = (int32_t)nwork;
  q.n_main = q.nwork;
  int slots = PAIR ? 74 : 148;
  const int smem_bytes = stages * STAGE + 1024;
  // per device and kernel variant, done once: the shared-memory opt-in and the number of CTA pairs
  // that can be resident together (both are host-side queries that would otherwise sit between the
  // filter pack and this launch on every call)
  static int cached_clusters[64] = {};           // 0 = not yet asked
  static bool attr_done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  if (PAIR) {
    cudaError_t e = cudaSuccess;
    if (!attr_done[dev]) {
      e = cudaFuncSetAttribute(conv_f16_nhwc_pair_kernel<BN, KSUB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
      if (e != cudaSuccess) return e;
      attr_done[dev] = true;
    }
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(148, 1, 1);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = cached_clusters[dev];        // as many pairs as can be resident at once
    if (clusters == 0) {
      e = cudaOccupancyMaxActiveClusters(&clusters, conv_f16_nhwc_pair_kernel<BN, KSUB>, &cfg);
      if (e != cudaSuccess) return e;
      if (clusters < 1) return cudaErrorInvalidValue;
      cached_clusters[dev] = clusters;
    }
    if (clusters < slots) slots = clusters;
  } else if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(conv_f16_nhwc_kernel<BN, KSUB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  // The last round of tiles, when it is short, handed out as runs of its reduction (plan_runs)
  q.stream_tiles = 0;
  if (BN >= 128 && q.partial != nullptr && q.ksplit == 1 && q.tail_halves) {
    const RunPlan rp = plan_runs(q.nwork, slots, q.num_kc, KSUB, BN);
    if (rp.tiles > 0) {
      q.stream_tiles = rp.tiles; q.stream_u = rp.u; q.stream_ctas = rp.ctas;
      q.n_main = q.nwork - rp.tiles;
      q.nwork = q.n_main + 2 * slots;            // two stream items per CTA (either may be empty)
    }
  }
  // Else, when that round would fill at most half of the CTAs (or pairs), each of its tiles
  // is handed out as two items of half the channels, so the round takes half as long.  (Not with a K
  // split, whose parts already are the finer grain.)
  if (q.stream_tiles == 0 && BN >= 128 && q.ksplit == 1 && q.tail_halves) {
    const int tail = q.nwork % slots;
    if (tail > 0 && 2 * tail <= slots) {
      q.n_main = q.nwork - tail;
      q.nwork += tail;
    }
  }
  const int ctas = slots < q.nwork ? slots : q.nwork;
  if (PAIR) {
    cfg.gridDim = dim3(2 * ctas, 1, 1);
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, conv_f16_nhwc_pair_kernel<BN, KSUB>, amap, bmap, bmap_h, q);
  }
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)ctas, 1, 1);
  return cudaLaunchKernelEx(&cfg, conv_f16_nhwc_kernel<BN, KSUB>, amap, bmap, bmap_h, q);
}

template <int KSUB>
cudaError_t launch_ksub(const CUtensorMap& amap, const CUtensorMap& bmap, const CUtensorMap& bmap_h, const NhwcParams& q,
                        const NhwcPlan& plan, cudaStream_t stream) {
  if (plan.pair) {
    if (plan.bn == 256) return launch_variant<256, true, KSUB>(amap, bmap, bmap_h, q, plan, stream);
    if (plan.bn == 128) return launch_variant<128, true, KSUB>(amap, bmap, bmap_h, q, plan, stream);
    return launch_variant<64, true, KSUB>(amap, bmap, bmap_h, q, plan, stream);
  }
  if (plan.bn == 64) return launch_variant<64, false, KSUB>(amap, bmap, bmap_h, q, plan, stream);
  if (plan.bn == 128) return launch_variant<128, false, KSUB>(amap, bmap, bmap_h, q, plan, stream);
  return launch_variant<256, false, KSUB>(amap, bmap, bmap_h, q, plan, stream);
}

// Geometry of the shifted-view kernel for a layer (host side).
struct ShiftViewPlan {
  bool eligible;
  int32_t Wq, rows, nkb2, nks_last, bu;
  uint32_t subt_bytes, a_stage_bytes;
  int64_t VQ, K2;
  double m_eff;              // useful fraction of the MMA rows
};

ShiftViewPlan plan_shift_view(const Geometry& g, const NhwcPlan& plan) {
  ShiftViewPlan p{};
  p.eligible = false;
  if (g.Kw > MAX_KW || g.Wp % g.s != 0 || g.s > 16) return p;
  p.Wq = g.Wp / g.s;
  p.VQ = (int64_t)g.N * g.Ho * p.Wq;
  if (p.VQ >= ((int64_t)1 << 31) - 4 * TILE_M) return p;
  p.rows = TILE_M + (g.Kw - 1) / g.s;
  if (p.rows > 256) return p;
  p.subt_bytes = (uint32_t)((p.rows * KB * 2 + 1023) / 1024 * 1024);
  p.a_stage_bytes = (uint32_t)(g.s < g.Kw ? g.s : g.Kw) * p.subt_bytes;
  p.K2 = (int64_t)g.Kh * plan.Cp;
  p.nkb2 = (int32_t)((p.K2 + KB - 1) / KB);
  p.nks_last = (int32_t)((p.K2 - (int64_t)(p.nkb2 - 1) * KB + 15) / 16);
  p.bu = g.Kw % 3 == 0 ? 3 : 2;
  if (2 * (int64_t)p.a_stage_bytes + 2 * (int64_t)p.bu * 256 * KB * 2 / 2 > kSmemMax - 2048) return p;
  p.m_eff = (double)g.Wo / p.Wq;
  p.eligible = true;
  return p;
}

template <int BN, bool PAIR>
cudaError_t launch_shift_variant(const CUtensorMap& amap, const CUtensorMap& bmap, const CUtensorMap& bmap_h,
                                 const CUtensorMap& bmap_q, ShiftViewParams q, const NhwcPlan& plan,
                                 const ShiftViewPlan& sp, cudaStream_t stream) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  constexpr int B_BYTES = B_ROWS * KB * 2;
  const int budget = kSmemMax - 2048;
  // units per filter stage: all kernel columns of a k2-block when two such stages fit beside two
  // activation stages (the MMA warp then pays two waits and two commits per block); otherwise three,
  // or fewer when three stages of that size do not fit (wide tiles without pairing)
  const bool whole_blocks = 2 * (int64_t)sp.a_stage_bytes + 2 * (int64_t)q.Kw * B_BYTES <= budget;
  if (!q.bu_forced) q.bu = whole_blocks ? q.Kw : 3;
  if (!(whole_blocks && q.bu == q.Kw))
    while (q.bu > 1 && 2 * (int64_t)sp.a_stage_bytes + 3 * (int64_t)q.bu * B_BYTES > budget) --q.bu;
  const int b_stage = q.bu * B_BYTES;
  // K split: whole k2-blocks
  q.kb_per_split = (sp.nkb2 + q.ksplit - 1) / q.ksplit;
  q.ksplit = (sp.nkb2 + q.kb_per_split - 1) / q.kb_per_split;
  const int64_t ntm = (sp.VQ + TILE_M - 1) / TILE_M;
  const int64_t ntm_eff = PAIR ? (ntm + 1) / 2 : ntm;
  const int64_t nwork = ntm_eff * q.ntn * q.ksplit;
  if (nwork >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  q.nwork = (int32_t)nwork;
  // rings: the whole filter resident when the layer has one channel tile and it fits beside two
  // activation stages; otherwise two or three activation stages and the rest for filter stages
  const int groups = (sp.nkb2 * q.Kw + q.bu - 1) / q.bu;
  q.resident = 0;
  if (q.ntn == 1 && q.ksplit == 1 && groups <= MAX_SB &&
      (int64_t)groups * b_stage + 2 * (int64_t)sp.a_stage_bytes <= budget) {
    q.resident = 1;
    q.sb = groups;
    q.sa = (int)((budget - (int64_t)groups * b_stage) / sp.a_stage_bytes);
    if (q.sa > MAX_SA) q.sa = MAX_SA;
  } else {
    q.sa = sp.a_stage_bytes <= 20 * 1024 ? 3 : 2;
    q.sb = (int)((budget - (int64_t)q.sa * sp.a_stage_bytes) / b_stage);
    if (q.sb > MAX_SB) q.sb = MAX_SB;
    if (q.sb < 2) { q.sa = 2; q.sb = (int)((budget - 2 * (int64_t)sp.a_stage_bytes) / b_stage); }
    if (q.sb < 2) return report(cudaErrorInvalidValue, "rings do not fit (shifted view)");
  }
  // two MMA issuers (see the kernel): a resident filter held as whole k2-blocks, and for each issuer
  // activation stages for a whole item (measured: 2-5 % faster then, cfg3 148 -> 142 us, a 3x3 layer
  // with 56x56 images and 64 channels 90 -> 86; with half-item rings a 128-channel layer lost 27 %)
  // and items of 24 MMAs or more (a 3x3 stem, six MMAs per item and bound by its output stores, lost a third)
  q.dual = (q.resident && q.bu == q.Kw && q.sa / 2 >= sp.nkb2 && q.nwork >= 2 && sp.nkb2 * q.Kw * (KB / 16) >= 24) ? 1 : 0;
  if (const char* v = debug_getenv("IM2WIN_NHWC_DUAL")) q.dual = (q.dual && v[0] != '0') ? 1 : 0;
  const int smem_bytes = q.sa * (int)sp.a_stage_bytes + q.sb * b_stage + 1024;
  static int cached_clusters[64] = {};
  static int attr_bytes[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  // CTAs (pairs) that are resident together: the grid, and what "a round of tiles" means below.  The
  // items of a split last round wait for one another, so every one of them must have a CTA of its own.
  int slots = PAIR ? 74 : 148;
  // the variants of this tile width: with / without tile parts, with / without the bias in registers
  // (64-channel tiles with one channel tile only)
  using Kernel = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, ShiftViewParams);
  constexpr bool CAN_HOIST = BN == 64;
  const Kernel variants[2][2] = {
      {PAIR ? (Kernel)conv_f16_nhwc_shift_pair_kernel<BN, false, false> : (Kernel)conv_f16_nhwc_shift_kernel<BN, false, false>,
       PAIR ? (Kernel)conv_f16_nhwc_shift_pair_kernel<BN, false, CAN_HOIST> : (Kernel)conv_f16_nhwc_shift_kernel<BN, false, CAN_HOIST>},
      {PAIR ? (Kernel)conv_f16_nhwc_shift_pair_kernel<BN, true, false> : (Kernel)conv_f16_nhwc_shift_kernel<BN, true, false>,
       PAIR ? (Kernel)conv_f16_nhwc_shift_pair_kernel<BN, true, CAN_HOIST> : (Kernel)conv_f16_nhwc_shift_kernel<BN, true, CAN_HOIST>}};
  const bool hoist = CAN_HOIST && q.e.bias != nullptr && q.ntn == 1;
  if (attr_bytes[dev] < smem_bytes) {
    for (int t = 0; t < 2; ++t)
      for (int h = 0; h < 2; ++h) {
        const cudaError_t e = cudaFuncSetAttribute((const void*)variants[t][h], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax - 1024);
        if (e != cudaSuccess) return report(e, "shared-memory opt-in (shifted view)");
      }
    attr_bytes[dev] = kSmemMax - 1024;
  }
  if (PAIR) {
    int clusters = cached_clusters[dev];
    if (clusters == 0) {
      cudaLaunchConfig_t probe = {};
      cudaLaunchAttribute pattr[1];
      pattr[0].id = cudaLaunchAttributeClusterDimension;
      pattr[0].val.clusterDim.x = 2; pattr[0].val.clusterDim.y = 1; pattr[0].val.clusterDim.z = 1;
      probe.blockDim = dim3(SHIFT_THREADS, 1, 1);
      probe.gridDim = dim3(148, 1, 1);
      probe.dynamicSmemBytes = (size_t)(kSmemMax - 1024);   // the worst case: one CTA per SM either way
      probe.attrs = pattr;
      probe.numAttrs = 1;
      cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, (const void*)variants[1][CAN_HOIST ? 1 : 0], &probe);
      if (e != cudaSuccess) return e;
      if (clusters < 1) return cudaErrorInvalidValue;
      cached_clusters[dev] = clusters;
    }
    if (clusters < slots) slots = clusters;
  }
  // The last round of tiles: when it is short, each of its tiles is handed out as two or four items
  // of half or a quarter of the channels (at least 64), so that the round takes a fraction of a
  // tile's time.  Streamed filters only (a resident one is laid out for whole tiles), no K split.
  q.n_main = q.nwork;
  q.tail_log2 = 0;
  bool tail_parts = true;
  if (const char* v = debug_getenv("IM2WIN_NHWC_TAIL")) tail_parts = v[0] != '0';
  q.tail_k = 0;
  q.tail_kb = 0;
  if (tail_parts && !q.resident && q.ksplit == 1) {
    const int tail = q.nwork % slots;
    // Preferred: parts of the reduction (every MMA stays as wide as the tile; the parts meet through
    // the tile's flag and red.global.add.f32), up to eight per tile, each at least two k2-blocks long.
    // Not under a ReLU or a rounding store (partial sums cannot pass them): then, or when K is short,
    // parts of the channels.
    // (and only for long items, 96 (k2-block, kernel column) units or more: measured, the wait for part 0
    // and the atomics cost short items more than the narrower MMAs of channel parts do:
    // 5x5 on 96 channels 121 against 115 us, 3x3 on 256 channels 71 against 61; 7x7 on 256: 265 against 300)
    bool k_parts = !q.e.relu && !q.e.out16 && q.flags != nullptr && 2 * tail * (int)sizeof(uint32_t) <= kTailFlagBytes &&
                   sp.nkb2 * q.Kw >= 96;
    if (const char* v = debug_getenv("IM2WIN_NHWC_TAIL_K")) k_parts = k_parts && v[0] != '0';
    int lg = 0;
    if (tail > 0 && k_parts) {
      for (int c = 3; c >= 1; --c)
        if ((tail << c) <= slots && sp.nkb2 >= 2 * (1 << c)) { lg = c; break; }
      if (lg > 0) {
        q.tail_k = 1;
        q.tail_kb = (sp.nkb2 + (1 << lg) - 1) >> lg;
        if (((1 << lg) - 1) * q.tail_kb >= sp.nkb2) { q.tail_k = 0; lg = 0; }      // a part would be empty
      }
    }
    if (lg == 0 && tail > 0 && BN >= 128) {
      if (BN >= 256 && 4 * tail <= slots) lg = 2;
      else if (2 * tail <= slots) lg = 1;
    }
    if (lg > 0) {
      q.n_main = q.nwork - tail;
      q.nwork += tail * ((1 << lg) - 1);
      q.tail_log2 = lg;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(SHIFT_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  if (PAIR) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    const int clusters = slots < q.nwork ? slots : q.nwork;
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.numAttrs = 2;
    return report(cudaLaunchKernelEx(&cfg, variants[q.tail_log2 > 0][hoist], amap, bmap, bmap_h, bmap_q, q),
                  q.tail_log2 > 0 ? "pair launch (shifted view, parts)" : "pair launch (shifted view)");
  }
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)(slots < q.nwork ? slots : q.nwork), 1, 1);
  return report(cudaLaunchKernelEx(&cfg, variants[q.tail_log2 > 0][hoist], amap, bmap, bmap_h, bmap_q, q),
                q.tail_log2 > 0 ? "launch (shifted view, parts)" : "launch (shifted view)");
}

cudaError_t launch_shift_view(const uint16_t* window, const uint16_t* fp, void* y, uint32_t* status, uint32_t* flags,
                              const Geometry& g, const NhwcPlan& plan, const ShiftViewPlan& sp, const EpilogueArgs& epi,
                              bool split, EncodeTiledFn encode, cudaStream_t stream) {
  // Activation operand: (k2, column class t, virtual position q): column k = q*s + t of the flat
  // sequence of all strips' columns; filter: (k2, kernel column v, output channel).  Out-of-range
  // coordinates read as zeros.
  CUtensorMap amap, bmap, bmap_h, bmap_q;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)sp.K2, (cuuint64_t)g.s, (cuuint64_t)sp.VQ};
    const cuuint64_t strides[2] = {(cuuint64_t)sp.K2 * 2, (cuuint64_t)g.s * sp.K2 * 2};
    const cuuint32_t box[3] = {(cuuint32_t)KB, 1, (cuuint32_t)sp.rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult cr = encode(&amap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<uint16_t*>(window), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return report(cudaErrorInvalidValue, "activation tensor map (shifted view)");
  }
  const int b_rows = plan.pair ? plan.bn / 2 : plan.bn;
  // the filter with boxes of a CTA's whole share of a tile's channels, of half and of a quarter of it
  // (the last two for the items of a short last round)
  for (int lg = 0; lg < 3; ++lg) {
    const cuuint64_t dims[3] = {(cuuint64_t)sp.K2, (cuuint64_t)g.Kw, (cuuint64_t)g.Co};
    const cuuint64_t strides[2] = {(cuuint64_t)sp.K2 * 2, (cuuint64_t)g.Kw * sp.K2 * 2};
    const cuuint32_t box[3] = {(cuuint32_t)KB, 1, (cuuint32_t)(b_rows >> lg)};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult cr = encode(lg == 0 ? &bmap : (lg == 1 ? &bmap_h : &bmap_q), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                         const_cast<uint16_t*>(fp), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return report(cudaErrorInvalidValue, "filter tensor map (shifted view)");
  }
  ShiftViewParams q{};
  q.e.y = y; q.e.bias = epi.bias;
  q.e.relu = epi.relu; q.e.out16 = epi.out16; q.e.y_nhwc = epi.y_nhwc; q.e.atomic = split ? 1 : 0;
  q.e.Ho = g.Ho; q.e.Wo = g.Wo; q.e.Co = g.Co; q.e.HoWo = g.Ho * g.Wo;
  q.e.rows_total = g.N * g.Ho;
  q.status = status;
  q.VQ = sp.VQ; q.Wq = sp.Wq; q.s = g.s; q.Kw = g.Kw;
  q.rows = sp.rows; q.subt_bytes = sp.subt_bytes; q.a_stage_bytes = sp.a_stage_bytes;
  q.nkb2 = sp.nkb2; q.nks_last = sp.nks_last; q.bu = sp.bu;
  q.ksplit = split ? plan.ksplit : 1;
  q.ntn = plan.ntn;
  q.epoch = next_epoch();
  q.flags = flags;
  if (const char* v = debug_getenv("IM2WIN_NHWC_BU")) { const int bu = atoi(v); if (bu >= 1 && bu <= 8) { q.bu = bu; q.bu_forced = 1; } }
  if (plan.pair) {
    if (plan.bn == 256) return launch_shift_variant<256, true>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
    if (plan.bn == 128) return launch_shift_variant<128, true>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
    return launch_shift_variant<64, true>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
  }
  if (plan.bn == 64) return launch_shift_variant<64, false>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
  if (plan.bn == 128) return launch_shift_variant<128, false>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
  return launch_shift_variant<256, false>(amap, bmap, bmap_h, bmap_q, q, plan, sp, stream);
}

}  // namespace

NhwcPlan plan_nhwc(const Geometry& g) {
  NhwcPlan p{};
  p.eligible = false;
  p.Cp = (g.C + 7) / 8 * 8;
  p.K = (int64_t)g.Kw * g.Kh * p.Cp;
  const int64_t lim = (int64_t)1 << 31;
  if (p.K >= lim - 64) return p;
  p.num_kb = (int32_t)((p.K + KB - 1) / KB);
  p.strip = (int64_t)g.Wp * g.Kh * p.Cp;
  p.window_elems = (int64_t)g.N * g.Ho * p.strip;
  if ((int64_t)g.N * g.Ho >= lim || p.strip >= lim) return p;
  if ((int64_t)g.s * g.Kh * p.Cp * 2 >= ((int64_t)1 << 40) || p.strip * 2 >= ((int64_t)1 << 40)) return p;
  // the transform from NCHW stages at least eight columns of Cp + 2 channels in 48 KB of shared memory
  if ((int64_t)(p.Cp + 2) * 2 * 8 > 48 * 1024) return p;
  // position tiles: tw tiles along a strip of bw columns each (one when the strip fits 128 rows),
  // G whole strips per tile when a strip is short
  p.tw = (g.Wo + TILE_M - 1) / TILE_M;
  p.bw = (g.Wo + p.tw - 1) / p.tw;
  p.G = p.tw > 1 ? 1 : TILE_M / p.bw;
  if (p.G > 256) p.G = 256;
  const int64_t groups = ((int64_t)g.N * g.Ho + p.G - 1) / p.G;
  p.ntm = groups * p.tw;
  // channel tile: the narrowest MMA N that covers Co, at most 256; CTA pairs (cta_group::2, M = 256)
  p.bn = g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256);
  p.pair = p.ntm >= 2;       // pairs at every width: half the filter bytes per CTA and half the MMA instructions per flop
  p.ntn = (g.Co + p.bn - 1) / p.bn;
  p.ksplit = 1;
  const int64_t ntm_eff = p.pair ? (p.ntm + 1) / 2 : p.ntm;
  const int slots = p.pair ? 74 : 148;
  const int64_t tiles = ntm_eff * p.ntn;
  // K is split over several CTAs only where the parts stay long (48 k-blocks or more): the partial
  // sums are added with atomics, which was measured to cost more than the fuller waves gain unless
  // a long main loop of other items hides it.  Among the admissible splits the one with the best
  // wave efficiency wins.
  if (tiles < 4 * slots) {
    double best = 0.0;
    for (int ks = 1; ks <= 8; ++ks) {
      const int per = (p.num_kb + ks - 1) / ks;
      if (ks > 1 && per < 48) break;
      const int parts = (p.num_kb + per - 1) / per;
      const int64_t items = tiles * parts;
      const int64_t waves = (items + slots - 1) / slots;
      const double t = (double)waves * (per + 4.0 + (parts > 1 ? 2.0 : 0.0));     // in k-blocks
      const double eff = (double)tiles * p.num_kb / slots / t;
      if (eff > best + 0.02) { best = eff; p.ksplit = parts; }
    }
  }
  p.kb_per_split = (p.num_kb + p.ksplit - 1) / p.ksplit;
  if (tiles * p.ksplit >= lim) return p;
  // status block, packed filter, then kTailFlagBytes of flag words (hand-off between the CTAs that share
  // a tile of a short last round; cleared by the filter pack)
  p.flags_off = ((size_t)kStatusBytes + (size_t)g.Co * p.K * 2 + 255) / 256 * 256;
  // ... and, for layers of few rounds of tiles, the partial-sum area of a last round handed out by
  // reduction length
  p.partial_off = p.flags_off + kTailFlagBytes;
  p.partial_bytes = tiles < 8 * slots ? kPartialBytes : 0;
  p.scratch_bytes = p.partial_off + p.partial_bytes;
  p.eligible = true;
  return p;
}

cudaError_t launch_transform_nhwc(const uint16_t* x, int x_is_nhwc, uint16_t* window, const Geometry& g,
                                  cudaStream_t stream) {
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  if (x_is_nhwc) {
    const int c8n = plan.Cp / 8;
    bool by_strip = (int64_t)g.N * g.Ho < ((int64_t)1 << 31) && (int64_t)g.Wp * g.Kh * c8n < ((int64_t)1 << 30);
    if (const char* v = debug_getenv("IM2WIN_NHWC_TRANSFORM")) by_strip = by_strip && strcmp(v, "chunks") != 0;   // testing aid
    const unsigned strips = (unsigned)((int64_t)g.N * g.Ho);
    if (by_strip && g.C % 8 == 0) {
      uint4* w4 = reinterpret_cast<uint4*>(window);
      int sh = 0;
      while ((1 << sh) < c8n) ++sh;
      if ((c8n & (c8n - 1)) == 0)
        transform_nhwc_from_nhwc_strip_kernel<true><<<strips, 256, 0, stream>>>(x, w4, g.C, c8n, sh, g.H, g.W, g.Ho, g.Wp, g.Kh, g.s, g.p);
      else
        transform_nhwc_from_nhwc_strip_kernel<false><<<strips, 256, 0, stream>>>(x, w4, g.C, c8n, 0, g.H, g.W, g.Ho, g.Wp, g.Kh, g.s, g.p);
      return cudaGetLastError();
    }
    const size_t px_smem = (size_t)g.Kh * g.W * g.C * 2;
    if (by_strip && plan.Cp == 8 && px_smem <= 48 * 1024) {
      transform_nhwc_from_nhwc_small_c_kernel<<<strips, 256, px_smem, stream>>>(x, reinterpret_cast<uint4*>(window), g.C, g.H, g.W,
                                                                               g.Ho, g.Wp, g.Kh, g.s, g.p);
      return cudaGetLastError();
    }
    const int64_t chunks = plan.window_elems / 8;
    int64_t blocks = (chunks + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    transform_nhwc_from_nhwc_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, window, g.C, plan.Cp, g.H, g.W, g.Ho, g.Wp,
                                                                          g.Kh, g.s, g.p, chunks);
    return cudaGetLastError();
  }
  // at most 8 channels: one block per strip, built in shared memory and written as one run
  const int SP = (g.Kh * g.W + 16 + 7) & ~7;              // staged halves per channel: a run plus the phase padding
  const int64_t strip_smem = (((int64_t)g.Wp * (4 * g.Kh + 1) + 3) & ~(int64_t)3) * 4 + (int64_t)g.C * SP * 2;
  bool by_strip = plan.Cp == 8 && strip_smem <= 100 * 1024 && (int64_t)g.N * g.Ho < ((int64_t)1 << 31);
  if (const char* v = debug_getenv("IM2WIN_NHWC_TRANSFORM")) by_strip = by_strip && strcmp(v, "rows") != 0;
  if (by_strip) {
    static bool attr_done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (strip_smem > 48 * 1024 && !attr_done[dev]) {
      cudaError_t e = cudaFuncSetAttribute(transform_nhwc_strip_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e != cudaSuccess) return e;
      attr_done[dev] = true;
    }
    transform_nhwc_strip_kernel<<<(unsigned)((int64_t)g.N * g.Ho), 256, (size_t)strip_smem, stream>>>(
        x, window, g.C, g.H, g.W, g.Ho, g.Wp, g.Kh, g.s, g.p, SP);
    return cudaGetLastError();
  }
  // columns per block: the whole row when it fits 48 KB of shared memory as T[w][Cp + 2]
  const int octs = plan.Cp / 8;
  bool swz = (octs & (octs - 1)) == 0;                     // chunks found by shift and mask, swizzled rows without padding
  if (const char* v = debug_getenv("IM2WIN_NHWC_TRANSFORM_SWZ")) swz = swz && v[0] != '0';   // testing aid
  const int64_t per_col = (int64_t)(plan.Cp + (swz ? 0 : 2)) * 2;
  int kc = (int)((48 * 1024) / per_col);
  if (kc < 8) return cudaErrorInvalidValue;
  if (kc > g.W) kc = g.W;
  else kc &= ~7;                                           // chunk boundaries stay multiples of 8 for the vector loads
  if (kc < 1) return cudaErrorInvalidValue;
  // columns per load: rows must start on a multiple of it (W a multiple) and so must the chunks
  const int vec = g.W % 8 == 0 ? 8 : (g.W % 4 == 0 ? 4 : (g.W % 2 == 0 ? 2 : 1));
  const int kchunks = (g.W + kc - 1) / kc;
  // rows per block: two (a block's set-up then serves both) when there are many more row blocks than
  // the GPU holds at once and a row is written to few places; measured 4-10 % faster on 3x3 and 5x5
  // layers with 56x56 and 24x24 images, slower from three rows on and for tall kernels
  const int rows_total = g.H + 2 * g.p;
  int R = ((int64_t)g.N * rows_total * kchunks >= 148 * 16 && g.Kh <= 5) ? 2 : 1;
  if (const char* v = debug_getenv("IM2WIN_NHWC_TRANSFORM_ROWS")) { const int r = atoi(v); if (r >= 1 && r <= 64) R = r; }   // testing aid
  const int rgroups = (rows_total + R - 1) / R;
  const int64_t blocks = (int64_t)g.N * rgroups * kchunks;
  if (blocks >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  const size_t smem = (size_t)(per_col * kc);
#define IM2WIN_LAUNCH_T(V, S)                                                                                       \
  transform_nhwc_from_nchw_kernel<V, S><<<(unsigned)blocks, 256, smem, stream>>>(x, window, g.C, plan.Cp, g.H, g.W, g.Ho, \
                                                                               g.Wp, g.Kh, g.s, g.p, kc, kchunks, R, rgroups)
  if (swz) {
    if (vec == 8) IM2WIN_LAUNCH_T(8, true);
    else if (vec == 4) IM2WIN_LAUNCH_T(4, true);
    else if (vec == 2) IM2WIN_LAUNCH_T(2, true);
    else IM2WIN_LAUNCH_T(1, true);
  } else {
    if (vec == 8) IM2WIN_LAUNCH_T(8, false);
    else if (vec == 4) IM2WIN_LAUNCH_T(4, false);
    else if (vec == 2) IM2WIN_LAUNCH_T(2, false);
    else IM2WIN_LAUNCH_T(1, false);
  }
#undef IM2WIN_LAUNCH_T
  return cudaGetLastError();
}

cudaError_t launch_pack_f16_nhwc(const uint16_t* filter, void* scratch, const Geometry& g, cudaStream_t stream) {
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  // channels per block: as many as fit 32 KB of staging, a multiple of 8, at least 8
  int cb = (32 * 1024 / 2 / g.T) / 8 * 8;
  if (cb < 8) cb = 8;
  if (cb > plan.Cp) cb = plan.Cp;
  const size_t smem = (size_t)cb * g.T * 2 + 32;
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(pack_f16_nhwc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)((plan.Cp + cb - 1) / cb), (unsigned)(g.Co < 32768 ? g.Co : 32768));
  pack_f16_nhwc_kernel<<<grid, 256, smem, stream>>>(filter, reinterpret_cast<uint16_t*>(base + kStatusBytes),
                                                     reinterpret_cast<uint32_t*>(base),
                                                     reinterpret_cast<uint32_t*>(base + plan.flags_off), g.C, plan.Cp, g.Co,
                                                     g.Kh, g.Kw, cb);
  return cudaGetLastError();
}

namespace {

// Everything a convolution call decides before it launches: tile plan, which of the two kernels, and
// whether every tile's K is split over several CTAs (the output is then cleared first).
struct NhwcChoice {
  NhwcPlan plan;
  ShiftViewPlan sp;
  bool use_shift, split;
  bool runs;                 // overlapping-row kernel: the last round of tiles goes out as runs of its reduction
};

NhwcChoice choose_nhwc(const Geometry& g, const EpilogueArgs& epi) {
  NhwcChoice c{};
  NhwcPlan& plan = c.plan;
  plan = plan_nhwc(g);
  if (!plan.eligible) return c;
  // testing aids (read only when IM2WIN_DEBUG is set): tile width, pairing and K split
  if (const char* v = debug_getenv("IM2WIN_NHWC_BN")) {
    const int bn = atoi(v);
    if (bn == 64 || bn == 128 || bn == 256) { plan.bn = bn; plan.ntn = (g.Co + bn - 1) / bn; }
  }
  if (const char* v = debug_getenv("IM2WIN_NHWC_PAIR")) plan.pair = v[0] == '1';
  if (const char* v = debug_getenv("IM2WIN_NHWC_KSPLIT")) {
    const int ks = atoi(v);
    if (ks >= 1 && ks <= plan.num_kb) plan.ksplit = ks;
  }
  bool split = plan.ksplit > 1 && !epi.relu && !epi.out16;   // partial sums cannot pass a ReLU or a rounding
  if (!split) plan.ksplit = 1;
  // Which kernel.  The shifted-view kernel brings s/Kw of the activation bytes into the SM but computes
  // Wq rows per strip for Wo outputs, and it needs one filter stage per k2-block (all kernel columns)
  // to keep its MMA warp's barrier traffic low.  Measured: it wins where every column is reused by
  // three kernel columns or more (Kw >= 3s) and two such filter stages fit beside two activation
  // stages; elsewhere the overlapping-row kernel is as fast or faster.
  c.sp = plan_shift_view(g, plan);
  const ShiftViewPlan& sp = c.sp;
  const int64_t b_bytes = (int64_t)(plan.pair ? plan.bn / 2 : plan.bn) * KB * 2;
  // Kernels no wider than the stride read every column once in either kernel; there the shifted view
  // is taken when its full 128-position tiles need fewer rounds than the overlapping-row kernel's
  // tiles of whole strips.
  const bool reuse = g.Kw >= 3 * g.s, once = g.Kw <= g.s;
  bool use_shift = sp.eligible && (reuse || (once && plan.ksplit == 1)) &&
                   2 * (int64_t)sp.a_stage_bytes + 2 * (int64_t)g.Kw * b_bytes <= kSmemMax - 2048;
  if (use_shift && plan.ksplit == 1) {
    // Rounds of tiles on the CTAs (pairs): the overlapping-row kernel can hand the tiles of a last round
    // that is at most half full out as half tiles, the shifted-view kernel cannot; where that saves
    // more than the shifted view's lower traffic is worth (measured: about 15 % per round), take it.
    const int slots = plan.pair ? 74 : 148;
    const int64_t it_o = (plan.pair ? (plan.ntm + 1) / 2 : plan.ntm) * plan.ntn;
    const int64_t tiles_s = (sp.VQ + TILE_M - 1) / TILE_M;
    const int64_t it_s = (plan.pair ? (tiles_s + 1) / 2 : tiles_s) * plan.ntn;
    const int64_t tail = it_o % slots;
    const double r_o = (double)(it_o / slots) + (tail == 0 ? 0.0 : (plan.bn >= 128 && 2 * tail <= slots ? 0.55 : 1.0));
    // (the shifted-view kernel hands a short last round out as quarter or half tiles when its filter is streamed)
    const int64_t tail_s = it_s % slots;
    const double r_s = (double)(it_s / slots) + (tail_s == 0 ? 0.0 : (plan.bn >= 256 && 4 * tail_s <= slots ? 0.4 : (plan.bn >= 128 && 2 * tail_s <= slots ? 0.55 : 1.0)));
    if (reuse ? r_o < 0.85 * r_s : r_o <= r_s) use_shift = false;
  }
  if (const char* v = debug_getenv("IM2WIN_NHWC_KERNEL")) {
    if (strcmp(v, "shift") == 0) use_shift = sp.eligible;
    else if (strcmp(v, "overlap") == 0) use_shift = false;
  }
  if (use_shift && split) {
    // The shifted-view kernel can also split K for the tiles of a short last round only (parts meet
    // through a flag, no cleared output, atomics on those tiles only).  Rounds, in tile times: whole
    // rounds plus 1/P + 0.1 for a last round handed out as P parts, against the parts of a split of
    // every tile plus 0.1 for clearing the output and the atomics.  (Measured: cfg5k5 135 against 148 us.)
    const int slots = plan.pair ? 74 : 148;
    const int64_t tiles_s = (sp.VQ + TILE_M - 1) / TILE_M;
    const int64_t it_s = (plan.pair ? (tiles_s + 1) / 2 : tiles_s) * plan.ntn;
    const int64_t tail_s = it_s % slots;
    double frac = tail_s == 0 ? 0.0 : 1.0;
    for (int c = 3; c >= 1 && tail_s > 0 && sp.nkb2 * g.Kw >= 96; --c)
      if ((tail_s << c) <= slots && sp.nkb2 >= 2 * (1 << c)) { frac = 1.0 / (1 << c) + 0.1; break; }
    const double r_tail = (double)(it_s / slots) + frac;
    const double r_split = (double)((it_s * plan.ksplit + slots - 1) / slots) / plan.ksplit + 0.1;
    if (r_tail <= r_split) { split = false; plan.ksplit = 1; }
  }
  if (!use_shift && plan.partial_bytes > 0) {
    // Overlapping-row kernel: a short last round handed out as runs of its reduction (plan_runs), against
    // a K split of every tile (cleared output, atomics).  Measured: 7x7 on 256 channels 250 against 261 us,
    // 11x11 611-617 against 600.
    bool tail = true;
    if (const char* v = debug_getenv("IM2WIN_NHWC_TAIL")) tail = v[0] != '0';
    const int slots = plan.pair ? 74 : 148;
    const int64_t it_o = (plan.pair ? (plan.ntm + 1) / 2 : plan.ntm) * plan.ntn;
    const RunPlan rp = tail ? plan_runs(it_o, slots, plan.num_kb, 1, plan.bn) : RunPlan{};
    if (split && rp.tiles > 0) {
      // (the split's parts fill the CTAs almost evenly; its cost is the cleared output and the atomics, a
      // fixed time that weighs less the longer the tiles are: about 65 k-blocks' worth, measured)
      const double r_split = (double)it_o / slots + 65.0 / plan.num_kb;
      if (rp.rounds < r_split) { split = false; plan.ksplit = 1; }
    }
    c.runs = !split && rp.tiles > 0;
  }
  c.use_shift = use_shift;
  c.split = split;
  return c;
}

}  // namespace

const char* nhwc_kernel_name(const Geometry& g, const EpilogueArgs& epi) {
  const NhwcChoice c = choose_nhwc(g, epi);
  if (!c.plan.eligible) return "none";
  if (c.use_shift) return c.split ? "f16-nhwc-shift+ksplit" : "f16-nhwc-shift";
  return c.split ? "f16-nhwc-overlap+ksplit" : (c.runs ? "f16-nhwc-overlap+runs" : "f16-nhwc-overlap");
}

cudaError_t launch_conv_f16_nhwc(const uint16_t* window, void* y, void* scratch, const Geometry& g,
                                 const EpilogueArgs& epi, cudaStream_t stream) {
  const NhwcChoice c = choose_nhwc(g, epi);
  if (!c.plan.eligible) return cudaErrorInvalidValue;
  const NhwcPlan& plan = c.plan;
  const ShiftViewPlan& sp = c.sp;
  const bool use_shift = c.use_shift, split = c.split;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  uint16_t* fp = reinterpret_cast<uint16_t*>(base + kStatusBytes);
  if (split) {
    cudaError_t e = cudaMemsetAsync(y, 0, (size_t)g.out_elems * 4, stream);
    if (e != cudaSuccess) return e;
  }
  if (use_shift)
    return launch_shift_view(window, fp, y, reinterpret_cast<uint32_t*>(base), reinterpret_cast<uint32_t*>(base + plan.flags_off),
                             g, plan, sp, epi, split, encode, stream);

  // Activation operand: (k, wo, strip) with OVERLAPPING rows: the row of output column wo starts
  // s*Kh*Cp halves after that of wo-1.  k beyond K, columns beyond Wo and strips beyond N*Ho read
  // as zeros.
  CUtensorMap amap, bmap;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)plan.K, (cuuint64_t)g.Wo, (cuuint64_t)g.N * g.Ho};
    const cuuint64_t strides[2] = {(cuuint64_t)g.s * g.Kh * plan.Cp * 2, (cuuint64_t)plan.strip * 2};
    const cuuint32_t box[3] = {(cuuint32_t)KB, (cuuint32_t)plan.bw, (cuuint32_t)plan.G};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult cr = encode(&amap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<uint16_t*>(window), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  const int b_rows = plan.pair ? plan.bn / 2 : plan.bn;
  CUtensorMap bmap_h;                            // the same filter with boxes of half as many channels
  for (int half = 0; half < 2; ++half) {
    const cuuint64_t dims[2] = {(cuuint64_t)plan.K, (cuuint64_t)g.Co};
    const cuuint64_t strides[1] = {(cuuint64_t)plan.K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)KB, (cuuint32_t)(half ? b_rows / 2 : b_rows)};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = encode(half ? &bmap_h : &bmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, fp, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }

  NhwcParams q{};
  q.e.y = y;
  q.e.bias = epi.bias;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.e.relu = epi.relu; q.e.out16 = epi.out16; q.e.y_nhwc = epi.y_nhwc; q.e.atomic = split ? 1 : 0;
  q.e.Ho = g.Ho; q.e.Wo = g.Wo; q.e.Co = g.Co; q.e.HoWo = g.Ho * g.Wo;
  q.e.rows_total = g.N * g.Ho;
  q.bw = plan.bw; q.G = plan.G; q.tw = plan.tw;
  q.ksplit = plan.ksplit;
  q.ntn = plan.ntn;
  q.a_bytes = (uint32_t)(plan.G * plan.bw * KB * 2);
  int ksub = 1;
  if (const char* v = debug_getenv("IM2WIN_NHWC_KSUB")) ksub = atoi(v) == 1 ? 1 : 2;
  q.tail_halves = 1;
  if (const char* v = debug_getenv("IM2WIN_NHWC_TAIL")) q.tail_halves = v[0] != '0';
  q.flags = reinterpret_cast<uint32_t*>(base + plan.flags_off);
  q.partial = plan.partial_bytes > 0 ? reinterpret_cast<float*>(base + plan.partial_off) : nullptr;
  q.epoch = next_epoch();
  if (ksub == 1) return launch_ksub<1>(amap, bmap, bmap_h, q, plan, stream);
  return launch_ksub<2>(amap, bmap, bmap_h, q, plan, stream);
}

}  // namespace im2win
