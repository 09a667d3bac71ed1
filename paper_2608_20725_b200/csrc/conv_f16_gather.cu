// fp16-input / fp32-accumulate im2win convolution on the sm_100a tensor cores
// (paper Algorithm 1, "TC" variant; GEMM view with positions as rows):
//
//     y[p][co] = sum_k A[p][k] * Fp[co][k],   p = (n, ho, wo),  k = c*T + v*Kh + u,
//     A[p][k]  = window[n][c][ho][(wo*s)*Kh + v*Kh + u].
//
// One CTA owns a 128-position x BN-channel tile whose fp32 accumulator lives in
// tensor memory.  The reduction runs in k-blocks of 64 through a ring of
// shared-memory stages:
//   * the filter tile (BN x 64 halves, k contiguous) arrives by TMA with the
//     128-byte swizzle, signalled on the stage's "full" mbarrier;
//   * the window tile (128 x 64 halves) cannot be described to TMA -- rows of
//     A overlap and start s*Kh elements (6 bytes for 3x3, stride 1) apart -- so
//     four producer warps gather it from the window tensor, one position per
//     thread, and store it in the same swizzled, k-major layout;
//   * one thread issues four tcgen05.mma (K = 16 each) per stage and commits
//     them to the stage's "empty" mbarrier, which frees the stage.
// After the last k-block the producer warps turn into the epilogue: they read
// the accumulator with tcgen05.ld (lane = position, column = channel) and write
// the NCHW output, contiguous along positions.
//
// Every mbarrier wait is bounded: on giving up a thread raises the status word
// at the start of the scratch buffer and the CTA drains and exits normally.
#include <cuda.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
namespace {

using namespace ptx;

constexpr int TILE_M = 128;               // positions per CTA (= MMA M)
constexpr int KB = kF16KBlock;            // halves per k-block (one 128-byte row)
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = TILE_M * KB * 2;
constexpr int NUM_THREADS = 192;          // warps 0-3 producers/epilogue, 4 TMA, 5 MMA

struct ConvF16Params {
  const uint16_t* __restrict__ win;
  float* __restrict__ y;
  uint32_t* status;
  int64_t P, img_stride, strip, chan_stride, K;
  int32_t HoWo, Wo, sKh, Co, T, num_kb;
};

// ---------------------------------------------------------------------- kernel
template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_f16_gather_kernel(const __grid_constant__ CUtensorMap fmap, ConvF16Params q) {
  constexpr int B_STAGE_BYTES = BN * KB * 2;
  constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;

  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment keeps the swizzle pattern of every stage anchored.
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bars[2 * STAGES + 1];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t full_bar0 = smem_u32(&bars[0]);
  const uint32_t empty_bar0 = smem_u32(&bars[STAGES]);
  const uint32_t acc_bar = smem_u32(&bars[2 * STAGES]);

  const int64_t m0 = (int64_t)blockIdx.x * TILE_M;
  const int n0 = blockIdx.y * BN;

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar0 + 8 * s, 4 + 1);   // 4 producer warps + the TMA thread's expect_tx arrive
      mbar_init(empty_bar0 + 8 * s, 1);      // one tcgen05.commit
    }
    mbar_init(acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(&tmem_base_slot), BN);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp < 4) {
    // ---------------- producers of the window operand, then epilogue ----------
    const int m = threadIdx.x;                     // row of the tile = position
    const int64_t p = m0 + m;
    const bool valid = p < q.P;
    int64_t n = 0;
    int r = 0;
    const uint16_t* ptr = q.win;
    if (valid) {
      n = p / q.HoWo;
      r = (int)(p - n * q.HoWo);
      const int ho = r / q.Wo;
      const int wo = r - ho * q.Wo;
      ptr += n * q.img_stride + ho * q.strip + (int64_t)wo * q.sKh;
    }
    int t = 0;                                     // offset inside the current channel's window
    int64_t k = 0;
    const int64_t wrap = q.chan_stride - q.T;      // pointer step from the end of one window to the next channel
    const uint32_t row_off = (uint32_t)m * 128u;
    const uint32_t sw = (uint32_t)(m & 7);
    bool ok = true;

    for (int kb = 0; kb < q.num_kb && ok; ++kb) {
      const int s = kb % STAGES;
      const uint32_t it = (uint32_t)(kb / STAGES);
      // Lane 0 polls; the result is shared so that the whole warp takes the same path.
      if (lane == 0) ok = mbar_wait(empty_bar0 + 8 * s, (it & 1u) ^ 1u, &abort_flag, q.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
      if (!ok) break;
      const uint32_t a_stage = smem_base + s * STAGE_BYTES;
#pragma unroll 1
      for (int ch = 0; ch < 8; ++ch) {
        uint32_t h[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          uint32_t v = 0;
          if (valid && k < q.K) v = (uint32_t)__ldg(ptr);
          h[e] = v;
          ++k;
          ++ptr;
          if (++t == q.T) {
            t = 0;
            ptr += wrap;
          }
        }
        const uint32_t w0 = h[0] | (h[1] << 16), w1 = h[2] | (h[3] << 16);
        const uint32_t w2 = h[4] | (h[5] << 16), w3 = h[6] | (h[7] << 16);
        const uint32_t dst = a_stage + row_off + (((uint32_t)ch ^ sw) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3)
                     : "memory");
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar0 + 8 * s);
    }

    // ---------------- epilogue ------------------------------------------------
    // tcgen05.ld is warp-collective: the decision must be uniform in the warp.
    if (ok && lane == 0) ok = mbar_wait(acc_bar, 0u, &abort_flag, q.status);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    __syncwarp();   // lane 0 observed the barrier: orders the other lanes' accesses after it
    if (ok) {
      tc_fence_after();
      const uint32_t lane_base = tmem_acc + ((uint32_t)(warp * 32) << 16);
      float* yrow = q.y + (n * q.Co) * q.HoWo + r;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (n0 + c0 >= q.Co) break;                // uniform across the CTA
        uint32_t v[32];
        tmem_ld32(lane_base + (uint32_t)c0, v);
        if (valid) store_strided32(yrow + (int64_t)(n0 + c0) * q.HoWo, q.HoWo, v, q.Co - n0 - c0);
      }
    }
  } else if (warp == 4) {
    // ---------------- TMA producer of the filter operand ----------------------
    if (lane == 0) {
      for (int kb = 0; kb < q.num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t it = (uint32_t)(kb / STAGES);
        if (!mbar_wait(empty_bar0 + 8 * s, (it & 1u) ^ 1u, &abort_flag, q.status)) break;
        const uint32_t bar = full_bar0 + 8 * s;
        mbar_arrive_expect_tx(bar, B_STAGE_BYTES);
        tma_load_2d(smem_base + s * STAGE_BYTES + A_STAGE_BYTES, &fmap, kb * KB, n0, bar);
      }
    }
  } else {
    // ---------------- MMA issuer ----------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_f16(TILE_M, BN);
      bool ok = true;
      for (int kb = 0; kb < q.num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t it = (uint32_t)(kb / STAGES);
        ok = mbar_wait(full_bar0 + 8 * s, it & 1u, &abort_flag, q.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_base + s * STAGE_BYTES;
        const uint32_t b_addr = a_addr + A_STAGE_BYTES;
#pragma unroll
        for (int j = 0; j < KB / 16; ++j) {
          const uint64_t ad = smem_desc_k_major_sw128(a_addr + j * 32);
          const uint64_t bd = smem_desc_k_major_sw128(b_addr + j * 32);
          umma_f16(tmem_acc, ad, bd, idesc, (kb > 0 || j > 0) ? 1u : 0u);
        }
        umma_commit(empty_bar0 + 8 * s);
      }
      if (ok) umma_commit(acc_bar);
    }
  }

  // ---------------- teardown ---------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // Give copies that may still be in flight time to land before the CTA's
    // shared memory is released.
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) {
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

template <int BN>
cudaError_t launch_bn(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                      const ScratchLayout& l, cudaStream_t stream) {
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return cudaErrorNotSupported;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  CUtensorMap fmap;
  const cuuint64_t dims[2] = {(cuuint64_t)l.Kp, (cuuint64_t)g.Co};
  const cuuint64_t strides[1] = {(cuuint64_t)l.Kp * 2};
  const cuuint32_t box[2] = {(cuuint32_t)KB, (cuuint32_t)BN};
  const cuuint32_t estr[2] = {1, 1};
  CUresult cr = encode(&fmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base + l.filter_off, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;

  ConvF16Params q;
  q.win = window;
  q.y = y;
  q.status = reinterpret_cast<uint32_t*>(base);
  q.P = g.P; q.img_stride = g.img_stride; q.strip = g.strip; q.chan_stride = g.chan_stride; q.K = g.K;
  q.HoWo = g.Ho * g.Wo; q.Wo = g.Wo; q.sKh = g.s * g.Kh; q.Co = g.Co; q.T = g.T;
  q.num_kb = (int32_t)(l.Kp / KB);

  constexpr int smem_bytes = STAGES * (A_STAGE_BYTES + BN * KB * 2) + 1024;
  cudaError_t e = cudaFuncSetAttribute(conv_f16_gather_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  dim3 grid((unsigned)((g.P + TILE_M - 1) / TILE_M), (unsigned)((g.Co + BN - 1) / BN));
  conv_f16_gather_kernel<BN><<<grid, NUM_THREADS, smem_bytes, stream>>>(fmap, q);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_conv_f16_gather(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream) {
  if (g.Co <= 64) return launch_bn<64>(window, y, scratch, g, l, stream);
  if (g.Co <= 128) return launch_bn<128>(window, y, scratch, g, l, stream);
  return launch_bn<256>(window, y, scratch, g, l, stream);
}

}  // namespace im2win
