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
#include <stdlib.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;
constexpr int KB = kF16KBlock;                 // 64 halves = one 128-byte swizzle row
constexpr int WARP_TMA = 0, WARP_MMA = 1, WARP_EPI0 = 2;
constexpr int NUM_WARPS = 6;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 8;
constexpr int A_SLOT_BYTES = TILE_M * KB * 2;  // 16 KB: room for 128 rows even when a tile holds fewer
constexpr int kSmemMax = 227 * 1024;

struct NhwcParams {
  void* y;
  const float* bias;
  uint32_t* status;
  int32_t relu, out16, y_nhwc, atomic;
  int32_t Ho, Wo, Co, HoWo;
  int32_t rows_total;        // N*Ho strips
  int32_t bw, G, tw;         // tile = G strips x bw output columns; tw tiles along a strip
  int32_t num_kb;            // 64-wide k-blocks
  int32_t nks_last;          // 16-wide MMA steps of the last k-block
  int32_t ksplit, kb_per_split;
  int32_t ntn, nwork;        // channel tiles; work items = position tiles (pairs) x channel tiles x k parts
  int32_t stages;
  uint32_t a_bytes;          // bytes one activation copy brings: G*bw*128
};

__device__ __forceinline__ void red_add_f32(float* p, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

// Epilogue of one accumulator row chunk: v[j] belongs to output channel c0 + j (j < cnt) of the
// row's position; `base` is the element index of channel c0 at that position and `cs` the element
// distance between channels (Ho*Wo for NCHW, 1 for NHWC).
__device__ __forceinline__ void store_chunk(const NhwcParams& q, int64_t base, int64_t cs, const uint32_t (&v)[32],
                                            int cnt, bool vec_ok) {
  if (q.atomic) {
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

template <int BN, bool PAIR>
__device__ __forceinline__ void conv_nhwc_body(const CUtensorMap& amap, const CUtensorMap& bmap, const NhwcParams& q) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;              // filter rows (output channels) this CTA stages
  constexpr uint32_t B_BYTES = (uint32_t)B_ROWS * KB * 2;
  constexpr uint32_t STAGE_BYTES = (uint32_t)A_SLOT_BYTES + B_BYTES;     // a multiple of 1024
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int w_first = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[2 * MAX_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(&bars[0]);
  const uint32_t empty0 = smem_u32(&bars[MAX_STAGES]);
  const uint32_t acc_full0 = smem_u32(&bars[2 * MAX_STAGES]);
  const uint32_t acc_empty0 = smem_u32(&bars[2 * MAX_STAGES + 2]);

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int i = 0; i < MAX_STAGES; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full0 + 8 * i, 1);
      mbar_init(acc_empty0 + 8 * i, PAIR ? 8 : 4);        // the four epilogue warps (of each CTA)
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WARP_MMA) {
    if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_slot), 2 * BN);
    else tmem_alloc(smem_u32(&tmem_base_slot), 2 * BN);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();               // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  const uint32_t full_dst = PAIR ? mapa_shared(full0, 0) : full0;          // the leader's barriers
  const uint32_t acc_empty_dst = PAIR ? mapa_shared(acc_empty0, 0) : acc_empty0;

  // work item w -> (position tile (pair) mt, channel tile nt, k part ks), nt and ks fastest so that
  // the CTAs that share an activation tile run at the same time
  const int per_mt = q.ntn * q.ksplit;

  if (warp == WARP_TMA) {
    // ---------------- copies of both operands ------------------------------------
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0;
    for (int w = w_first; w < q.nwork && ok; w += w_step) {
      const int mt = w / per_mt, rem = w - mt * per_mt;
      const int nt = rem / q.ksplit, ks = rem - nt * q.ksplit;
      const int mti = PAIR ? 2 * mt + (int)rank : mt;
      const int rg = mti / q.tw, wt = mti - rg * q.tw;
      const int z = rg * q.G, yc = wt * q.bw;
      const int brow = nt * BN + (int)rank * B_ROWS;
      const int kb0 = ks * q.kb_per_split;
      const int kb1 = kb0 + q.kb_per_split < q.num_kb ? kb0 + q.kb_per_split : q.num_kb;
      for (int kb = kb0; kb < kb1; ++kb) {
        ok = mbar_wait(empty0 + 8 * st, ph ^ 1u, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (leader) {
          const uint32_t a_dst = ring + (uint32_t)st * STAGE_BYTES;
          const uint32_t b_dst = a_dst + (uint32_t)A_SLOT_BYTES;
          if (PAIR) {
            // the leader CTA announces the bytes of both CTAs; every copy reports to its barrier
            if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * st, 2u * (q.a_bytes + B_BYTES));
            tma_load_3d_pair(a_dst, &amap, kb * KB, yc, z, full_dst + 8 * st);
            tma_load_2d_pair(b_dst, &bmap, kb * KB, brow, full_dst + 8 * st);
          } else {
            mbar_arrive_expect_tx(full0 + 8 * st, q.a_bytes + B_BYTES);
            tma_load_3d(a_dst, &amap, kb * KB, yc, z, full0 + 8 * st);
            tma_load_2d(b_dst, &bmap, kb * KB, brow, full0 + 8 * st);
          }
        }
        __syncwarp();
        if (++st == q.stages) { st = 0; ph ^= 1u; }
      }
    }
  } else if (warp == WARP_MMA && rank == 0) {
    // ---------------- MMA issuer (leader CTA of a pair) -----------------------------
    constexpr uint32_t idesc = instr_desc_f16(PAIR ? 2 * TILE_M : TILE_M, BN);
    const bool leader = elect_one();
    bool ok = true;
    int st = 0;
    uint32_t ph = 0, it = 0;
    for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
      const int rem = w % per_mt;
      const int ks = rem % q.ksplit;
      const int kb0 = ks * q.kb_per_split;
      const int kb1 = kb0 + q.kb_per_split < q.num_kb ? kb0 + q.kb_per_split : q.num_kb;
      const uint32_t buf = it & 1u;
      ok = PAIR ? mbar_wait_cluster(acc_empty0 + 8 * buf, ((it >> 1) & 1u) ^ 1u, &abort_flag, q.status)
                : mbar_wait(acc_empty0 + 8 * buf, ((it >> 1) & 1u) ^ 1u, &abort_flag, q.status);   // drained by the epilogue
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = tmem_acc + buf * (uint32_t)BN;
      uint32_t accumulate = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        ok = PAIR ? mbar_wait_cluster(full0 + 8 * st, ph, &abort_flag, q.status)
                  : mbar_wait(full0 + 8 * st, ph, &abort_flag, q.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (leader) {
          const uint32_t a_lo = smem_desc_lo(ring + (uint32_t)st * STAGE_BYTES);
          const uint32_t b_lo = smem_desc_lo(ring + (uint32_t)st * STAGE_BYTES + (uint32_t)A_SLOT_BYTES);
          const int nks = kb == q.num_kb - 1 ? q.nks_last : KB / 16;
#pragma unroll
          for (int j = 0; j < KB / 16; ++j) {
            if (j < nks) {
              if (PAIR)
                umma_f16_ab_pair(acc, a_lo + 2 * j, kSmemDescHiSw128, b_lo + 2 * j, kSmemDescHiSw128, idesc, accumulate);
              else
                umma_f16_lohi(acc, a_lo + 2 * j, b_lo + 2 * j, idesc, accumulate);
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
    }
  } else if (warp >= WARP_EPI0) {
    // ---------------- epilogue: tensor memory -> output -----------------------------
    const int lq = warp & 3;                     // tensor-memory lane quadrant this warp may read
    const bool vec_ok = q.out16 ? (q.Co % 8 == 0) : (q.Co % 4 == 0);
    bool ok = true;
    uint32_t it = 0;
    for (int w = w_first; w < q.nwork && ok; w += w_step, ++it) {
      const uint32_t buf = it & 1u;
      const int mt = w / per_mt, rem = w - mt * per_mt;
      const int nt = rem / q.ksplit, ks = rem - nt * q.ksplit;
      const int mti = PAIR ? 2 * mt + (int)rank : mt;
      const int rg = mti / q.tw, wt = mti - rg * q.tw;
      const int n0 = nt * BN;
      // accumulator row r = lane of tensor memory = (strip j of the tile, column i of the tile)
      const int r = lq * 32 + lane;
      const int j = r / q.bw, i = r - j * q.bw;
      const int strip = rg * q.G + j, wo = wt * q.bw + i;
      const bool valid = j < q.G && strip < q.rows_total && wo < q.Wo;
      int64_t base = 0, cs = 1;
      if (valid) {
        if (q.y_nhwc) {
          base = ((int64_t)strip * q.Wo + wo) * q.Co + n0;
        } else {
          const int n = strip / q.Ho, ho = strip - n * q.Ho;
          cs = q.HoWo;
          base = ((int64_t)n * q.Co + n0) * q.HoWo + ho * q.Wo + wo;
        }
      }
      if (lane == 0) ok = mbar_wait(acc_full0 + 8 * buf, (it >> 1) & 1u, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if (!ok) break;
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + buf * (uint32_t)BN + ((uint32_t)(lq * 32) << 16);
      const bool first_part = ks == 0;           // of a split K, only the first part adds the bias
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        const int cnt = q.Co - n0 - c0;          // channels left from c0 on
        if (cnt <= 0) break;
        uint32_t v[32];
        tmem_ld32(lane_base + (uint32_t)c0, v);
        if (q.bias != nullptr && first_part) {
          const float b = lane < cnt ? __ldg(q.bias + n0 + c0 + lane) : 0.0f;
#pragma unroll
          for (int t = 0; t < 32; ++t) v[t] = __float_as_uint(__uint_as_float(v[t]) + __shfl_sync(0xffffffffu, b, t));
        }
        if (q.relu) {
#pragma unroll
          for (int t = 0; t < 32; ++t) v[t] = __float_as_uint(fmaxf(__uint_as_float(v[t]), 0.0f));
        }
        if (valid) store_chunk(q, base + (int64_t)c0 * cs, cs, v, cnt < 32 ? cnt : 32, vec_ok);
      }
      // the buffer may be overwritten once all four warps (of both CTAs) have read it
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
    for (int i = 0; i < 64; ++i) __nanosleep(1000);     // copies in flight land before the CTA leaves
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
conv_f16_nhwc_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap, NhwcParams q) {
  conv_nhwc_body<BN, false>(amap, bmap, q);
}

template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
conv_f16_nhwc_pair_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap, NhwcParams q) {
  conv_nhwc_body<BN, true>(amap, bmap, q);
}

// Filter pack (paper Section "Im2win Convolution": height before width; here with the channel below
// both): fp[co][(v*Kh + u)*Cp + c] = f[co][c][u][v], zeros for c >= C.  Thread 0.. of block 0 also
// clears the status block.
__global__ void pack_f16_nhwc_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp, uint32_t* status,
                                     int C, int Cp, int Kh, int Kw, int64_t total) {
  if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int64_t K = (int64_t)Kw * Kh * Cp;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t co = idx / K;
    int64_t t = idx - co * K;
    const int c = (int)(t % Cp);
    t /= Cp;
    const int u = (int)(t % Kh), v = (int)(t / Kh);
    fp[idx] = c < C ? f[((co * C + c) * Kh + u) * Kw + v] : (uint16_t)0;
  }
}

// ---------------------------------------------------------------- transform ----
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

// x given NCHW: a transposition.  One block moves the 64 channels x 64 columns of one (n, ho, u):
// input row h = ho*s + u - p of 64 channels is read along w (coalesced), turned in shared memory and
// written along c (128 bytes per column k).
constexpr int TT = 64;
__global__ void __launch_bounds__(256)
transform_nhwc_from_nchw_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ win, int C, int Cp, int H, int W,
                                int Ho, int Wp, int Kh, int s, int p, int ctiles, int ktiles) {
  __shared__ uint16_t tile[TT][TT + 2];          // [k][c], 33-word pitch: conflict-free both ways
  int64_t b = blockIdx.x;
  const int kt = (int)(b % ktiles); b /= ktiles;
  const int ct = (int)(b % ctiles); b /= ctiles;
  const int u = (int)(b % Kh); b /= Kh;
  const int ho = (int)(b % Ho);
  const int64_t n = b / Ho;
  const int h = ho * s + u - p;
  const int k0 = kt * TT, c0 = ct * TT;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;      // 64 x 4
  const bool row_ok = h >= 0 && h < H;
  for (int cc = ty; cc < TT; cc += 4) {
    const int c = c0 + cc, w = k0 + tx - p;
    uint16_t v = 0;
    if (row_ok && c < C && w >= 0 && w < W && k0 + tx < Wp) v = __ldg(x + ((n * C + c) * H + h) * (int64_t)W + w);
    tile[tx][cc] = v;
  }
  __syncthreads();
  // write: thread -> (column k, channel pair): 32 lanes write 128 contiguous bytes of one column
  const int cw = (Cp - c0 < TT ? Cp - c0 : TT) / 2;            // channel pairs of this tile (Cp is even)
  const int lane2 = threadIdx.x & 31, kq = threadIdx.x >> 5;   // 32 x 8
  for (int kk = kq; kk < TT; kk += 8) {
    const int k = k0 + kk;
    if (k >= Wp || lane2 >= cw) continue;
    const uint32_t v = *reinterpret_cast<const uint32_t*>(&tile[kk][2 * lane2]);    // rows are 132 bytes: 4-byte aligned
    uint16_t* dst = win + ((((n * Ho + ho) * Wp + k) * Kh + u) * (int64_t)Cp) + c0 + 2 * lane2;
    *reinterpret_cast<uint32_t*>(dst) = v;
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

template <int BN, bool PAIR>
cudaError_t launch_variant(const CUtensorMap& amap, const CUtensorMap& bmap, NhwcParams q, int slots, cudaStream_t stream) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  constexpr int STAGE = A_SLOT_BYTES + B_ROWS * KB * 2;
  int stages = (kSmemMax - 2048) / STAGE;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return cudaErrorInvalidValue;
  q.stages = stages;
  const int smem_bytes = stages * STAGE + 1024;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  if (PAIR) {
    cudaError_t e = cudaFuncSetAttribute(conv_f16_nhwc_pair_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(148, 1, 1);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;                           // as many pairs as can be resident at once
    e = cudaOccupancyMaxActiveClusters(&clusters, conv_f16_nhwc_pair_kernel<BN>, &cfg);
    if (e != cudaSuccess) return e;
    if (clusters < 1) return cudaErrorInvalidValue;
    if (clusters > slots) clusters = slots;
    if (clusters > q.nwork) clusters = q.nwork;
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    return cudaLaunchKernelEx(&cfg, conv_f16_nhwc_pair_kernel<BN>, amap, bmap, q);
  }
  cudaError_t e = cudaFuncSetAttribute(conv_f16_nhwc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  cfg.gridDim = dim3((unsigned)(slots < q.nwork ? slots : q.nwork), 1, 1);
  return cudaLaunchKernelEx(&cfg, conv_f16_nhwc_kernel<BN>, amap, bmap, q);
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
  // position tiles: tw tiles along a strip of bw columns each (one when the strip fits 128 rows),
  // G whole strips per tile when a strip is short
  p.tw = (g.Wo + TILE_M - 1) / TILE_M;
  p.bw = (g.Wo + p.tw - 1) / p.tw;
  p.G = p.tw > 1 ? 1 : TILE_M / p.bw;
  if (p.G > 256) p.G = 256;
  const int64_t groups = ((int64_t)g.N * g.Ho + p.G - 1) / p.G;
  p.ntm = groups * p.tw;
  // channel tile: the narrowest MMA N that covers Co, at most 256; tiles of 256 run as CTA pairs
  // (each CTA stages half of the filter tile)
  p.bn = g.Co <= 64 ? 64 : (g.Co <= 128 ? 128 : 256);
  p.pair = p.bn == 256;
  p.ntn = (g.Co + p.bn - 1) / p.bn;
  p.ksplit = 1;
  const int64_t ntm_eff = p.pair ? (p.ntm + 1) / 2 : p.ntm;
  const int slots = p.pair ? 74 : 148;
  const int64_t tiles = ntm_eff * p.ntn;
  // K is split when the tiles alone leave most of a wave empty or the last wave nearly so: parts of
  // at least 8 k-blocks, as many as bring the number of work items to a whole number of waves
  if (tiles < 2 * slots && p.num_kb >= 16) {
    double best = 0.0;
    for (int ks = 1; ks <= 8; ++ks) {
      const int per = (p.num_kb + ks - 1) / ks;
      if (per < 8 && ks > 1) break;
      const int parts = (p.num_kb + per - 1) / per;
      const int64_t items = tiles * parts;
      const int64_t waves = (items + slots - 1) / slots;
      // time ~ waves * (k-blocks per part + fixed cost of an item in k-block units)
      const double t = (double)waves * (per + 3.0 + (parts > 1 ? 1.5 : 0.0));
      const double eff = (double)tiles * p.num_kb / slots / t;
      if (eff > best + 1e-9) { best = eff; p.ksplit = parts; }
    }
  }
  p.kb_per_split = (p.num_kb + p.ksplit - 1) / p.ksplit;
  p.ksplit = (p.num_kb + p.kb_per_split - 1) / p.kb_per_split;
  if (tiles * p.ksplit >= lim) return p;
  p.scratch_bytes = (size_t)kStatusBytes + (size_t)g.Co * p.K * 2;
  p.scratch_bytes = (p.scratch_bytes + 255) / 256 * 256;
  p.eligible = true;
  return p;
}

cudaError_t launch_transform_nhwc(const uint16_t* x, int x_is_nhwc, uint16_t* window, const Geometry& g,
                                  cudaStream_t stream) {
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  if (x_is_nhwc) {
    const int64_t chunks = plan.window_elems / 8;
    int64_t blocks = (chunks + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    transform_nhwc_from_nhwc_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, window, g.C, plan.Cp, g.H, g.W, g.Ho, g.Wp,
                                                                          g.Kh, g.s, g.p, chunks);
    return cudaGetLastError();
  }
  const int ctiles = (plan.Cp + TT - 1) / TT, ktiles = (g.Wp + TT - 1) / TT;
  const int64_t blocks = (int64_t)g.N * g.Ho * g.Kh * ctiles * ktiles;
  if (blocks >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  transform_nhwc_from_nchw_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, window, g.C, plan.Cp, g.H, g.W, g.Ho, g.Wp,
                                                                        g.Kh, g.s, g.p, ctiles, ktiles);
  return cudaGetLastError();
}

cudaError_t launch_pack_f16_nhwc(const uint16_t* filter, void* scratch, const Geometry& g, cudaStream_t stream) {
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  const int64_t total = (int64_t)g.Co * plan.K;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  pack_f16_nhwc_kernel<<<(unsigned)blocks, 256, 0, stream>>>(filter, reinterpret_cast<uint16_t*>(base + kStatusBytes),
                                                             reinterpret_cast<uint32_t*>(base), g.C, plan.Cp, g.Kh, g.Kw, total);
  return cudaGetLastError();
}

cudaError_t launch_conv_f16_nhwc(const uint16_t* window, void* y, void* scratch, const Geometry& g,
                                 const EpilogueArgs& epi, cudaStream_t stream) {
  NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return cudaErrorInvalidValue;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  uint16_t* fp = reinterpret_cast<uint16_t*>(base + kStatusBytes);
  // testing aids (read only when IM2WIN_DEBUG is set): tile width, pairing and K split
  if (const char* v = debug_getenv("IM2WIN_NHWC_BN")) {
    const int bn = atoi(v);
    if (bn == 64 || bn == 128 || bn == 256) { plan.bn = bn; plan.ntn = (g.Co + bn - 1) / bn; plan.pair = bn == 256; }
  }
  if (const char* v = debug_getenv("IM2WIN_NHWC_PAIR")) plan.pair = v[0] == '1' && plan.bn >= 128;
  if (const char* v = debug_getenv("IM2WIN_NHWC_KSPLIT")) {
    int ks = atoi(v);
    if (ks >= 1 && ks <= plan.num_kb) {
      plan.kb_per_split = (plan.num_kb + ks - 1) / ks;
      plan.ksplit = (plan.num_kb + plan.kb_per_split - 1) / plan.kb_per_split;
    }
  }
  const bool split = plan.ksplit > 1 && !epi.relu && !epi.out16;   // partial sums cannot pass a ReLU or a rounding
  if (!split) { plan.ksplit = 1; plan.kb_per_split = plan.num_kb; }

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
  {
    const cuuint64_t dims[2] = {(cuuint64_t)plan.K, (cuuint64_t)g.Co};
    const cuuint64_t strides[1] = {(cuuint64_t)plan.K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)KB, (cuuint32_t)b_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = encode(&bmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, fp, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }

  NhwcParams q{};
  q.y = y;
  q.bias = epi.bias;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.relu = epi.relu; q.out16 = epi.out16; q.y_nhwc = epi.y_nhwc; q.atomic = split ? 1 : 0;
  q.Ho = g.Ho; q.Wo = g.Wo; q.Co = g.Co; q.HoWo = g.Ho * g.Wo;
  q.rows_total = g.N * g.Ho;
  q.bw = plan.bw; q.G = plan.G; q.tw = plan.tw;
  q.num_kb = plan.num_kb;
  q.nks_last = (int32_t)((plan.K - (int64_t)(plan.num_kb - 1) * KB + 15) / 16);
  q.ksplit = plan.ksplit; q.kb_per_split = plan.kb_per_split;
  q.ntn = plan.ntn;
  const int64_t ntm_eff = plan.pair ? (plan.ntm + 1) / 2 : plan.ntm;
  const int64_t nwork = ntm_eff * plan.ntn * plan.ksplit;
  if (nwork >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  q.nwork = (int32_t)nwork;
  q.a_bytes = (uint32_t)(plan.G * plan.bw * KB * 2);
  if (split) {
    cudaError_t e = cudaMemsetAsync(y, 0, (size_t)g.out_elems * 4, stream);
    if (e != cudaSuccess) return e;
  }
  if (plan.pair) {
    if (plan.bn == 256) return launch_variant<256, true>(amap, bmap, q, 74, stream);
    return launch_variant<128, true>(amap, bmap, q, 74, stream);
  }
  if (plan.bn == 64) return launch_variant<64, false>(amap, bmap, q, 148, stream);
  if (plan.bn == 128) return launch_variant<128, false>(amap, bmap, q, 148, stream);
  return launch_variant<256, false>(amap, bmap, q, 148, stream);
}

}  // namespace im2win
