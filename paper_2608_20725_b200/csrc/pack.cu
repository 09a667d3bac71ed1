// Filter repacking for the im2win convolution kernels (sm_100a).
//
// The im2win window of one channel is stored height-fastest (offset v*Kh + u),
// so the filter is repacked to the same order (paper, Section "Im2win
// Convolution": the filter layout puts height before width):
//     k = c*T + v*Kh + u,   T = Kh*Kw,   Fp[co][k] = F[co][c][u][v].
// The same pass writes the table k -> element offset of window element k
// relative to the window of channel 0 (c*chan_stride + v*Kh + u); entries of
// the zero-padded tail k >= K hold -1.  It also clears the status block at the
// start of the scratch buffer.
//   fp32 kernel layout: Fk[k][Co_pad]  (co contiguous), zero padded in k and co
//   fp16 gather kernel: Fp[co][Kp]     (k contiguous),  zero padded in k
//   fp16 shifted-view kernel: Fp2[v][co][K2p] with k2 = c*Kh + u (see pack_f16_shift_kernel)
#include "common.cuh"

namespace im2win {
namespace {

struct PackParams {
  int32_t C, Co, Kh, Kw, T;
  int64_t K, Kp, Co_pad, chan_stride;
};

__device__ __forceinline__ void split_k(const PackParams& q, int64_t k, int& c, int& u, int& v) {
  c = (int)(k / q.T);
  const int t = (int)(k - (int64_t)c * q.T);
  v = t / q.Kh;
  u = t - v * q.Kh;
}

__global__ void pack_f32_kernel(const float* __restrict__ f, float* __restrict__ fk,
                                int32_t* __restrict__ koff, uint32_t* __restrict__ status,
                                PackParams q) {
  if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int64_t total = q.Kp * q.Co_pad;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t k = i / q.Co_pad;
    const int co = (int)(i - k * q.Co_pad);
    float val = 0.f;
    if (k < q.K && co < q.Co) {
      int c, u, v;
      split_k(q, k, c, u, v);
      val = f[(((int64_t)co * q.C + c) * q.Kh + u) * q.Kw + v];
    }
    fk[i] = val;
    if (co == 0) {
      int32_t off = -1;
      if (k < q.K) {
        int c, u, v;
        split_k(q, k, c, u, v);
        off = (int32_t)(c * q.chan_stride + v * q.Kh + u);
      }
      koff[k] = off;
    }
  }
}

__global__ void pack_f16_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp,
                                int32_t* __restrict__ koff, uint32_t* __restrict__ status,
                                PackParams q) {
  if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int64_t total = q.Kp * q.Co;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t co = i / q.Kp;
    const int64_t k = i - co * q.Kp;
    uint16_t val = 0;
    int32_t off = -1;
    if (k < q.K) {
      int c, u, v;
      split_k(q, k, c, u, v);
      val = f[((co * q.C + c) * q.Kh + u) * q.Kw + v];
      off = (int32_t)(c * q.chan_stride + v * q.Kh + u);
    }
    fp[i] = val;
    if (co == 0) koff[k] = off;
  }
}

// Layout of the shifted-view fp16 kernels: Fp2[v][co][k2], k2 = c*Kh + u (zero padded to K2p),
// and one of two tables: k2 -> c*chan_stride + u (gathering kernel, raw_pitch = 0; -1 for padded
// k2), or k2 -> byte offset of element (c, u) inside a raw box, slot (c - first channel of the
// k-block) * raw_pitch + u*2, padded k2 pointing at the all-zero slot `nslot` (TMA-staged kernel).
// One block handles one output channel and `chunk` (even, <= 512) consecutive k2: its Kw*chunk source halves
// are one contiguous run of the OIHW filter ((co*K2 + k2)*Kw + v), which is read coalesced into
// shared memory and written back out as Kw coalesced rows of the packed layout.
__global__ void pack_f16_shift_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp,
                                      uint32_t* __restrict__ table, uint32_t* __restrict__ status,
                                      PackParams q, int raw_pitch, int nslot, int chunk) {
  extern __shared__ __align__(16) uint16_t pack_s[];
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int K2 = q.C * q.Kh;
  const int K2p = (int)q.Kp;
  const int k2a = blockIdx.x * chunk;
  const int k2b = k2a + chunk < K2p ? k2a + chunk : K2p;
  const int nreal = (k2b < K2 ? k2b : K2) - k2a;          // k2 of this chunk that exist in the filter (may be <= 0)
  const size_t f_total = (size_t)q.Co * K2 * q.Kw;
  for (int co = blockIdx.y; co < q.Co; co += gridDim.y) {
    // The run is read with 16-byte loads from the 16-byte boundary at or before its start; run
    // element i then sits at pack_s[i + mis].
    const size_t start = ((size_t)co * K2 + k2a) * q.Kw;
    const int mis = (int)(start & 7);
    const int n = nreal > 0 ? nreal * q.Kw : 0;
    __syncthreads();
    for (int vec = threadIdx.x; vec * 8 < mis + n; vec += blockDim.x) {
      const size_t i0 = start - mis + (size_t)vec * 8;
      if (i0 + 8 <= f_total) {
        reinterpret_cast<uint4*>(pack_s)[vec] = __ldg(reinterpret_cast<const uint4*>(f + i0));
      } else {
        for (int h = 0; h < 8; ++h) pack_s[vec * 8 + h] = i0 + h < f_total ? f[i0 + h] : (uint16_t)0;
      }
    }
    __syncthreads();
    const uint16_t* run = pack_s + mis;
    for (int v = 0; v < q.Kw; ++v) {
      uint16_t* dst = fp + ((size_t)v * q.Co + co) * K2p + k2a;
      // eight k2 per thread: one 16-byte store (k2a and K2p are multiples of 8)
      for (int j = 8 * threadIdx.x; j < k2b - k2a; j += 8 * blockDim.x) {
        uint32_t w[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const uint32_t lo = j + 2 * h < nreal ? run[(j + 2 * h) * q.Kw + v] : 0u;
          const uint32_t hi = j + 2 * h + 1 < nreal ? run[(j + 2 * h + 1) * q.Kw + v] : 0u;
          w[h] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  if (blockIdx.y == 0) {
    for (int k2 = k2a + threadIdx.x; k2 < k2b; k2 += blockDim.x) {
      uint32_t entry = raw_pitch > 0 ? (uint32_t)(nslot * raw_pitch) : 0xffffffffu;
      if (k2 < K2) {
        const int c = k2 / q.Kh;
        const int u = k2 - c * q.Kh;
        if (raw_pitch > 0) {
          const int c_lo = (k2 / kF16KBlock) * kF16KBlock / q.Kh;
          entry = (uint32_t)((c - c_lo) * raw_pitch + u * 2);
        } else {
          entry = (uint32_t)(c * q.chan_stride + u);
        }
      }
      table[k2] = entry;
    }
  }
}

PackParams make_params(const Geometry& g, const ScratchLayout& l) {
  PackParams q;
  q.C = g.C; q.Co = g.Co; q.Kh = g.Kh; q.Kw = g.Kw; q.T = g.T;
  q.K = g.K; q.Kp = l.Kp; q.Co_pad = l.Co_pad; q.chan_stride = g.chan_stride;
  return q;
}

int grid_for(int64_t total) {
  int64_t b = (total + 255) / 256;
  if (b > 148 * 8) b = 148 * 8;
  if (b < 1) b = 1;
  return (int)b;
}

}  // namespace

cudaError_t launch_pack_f32(const float* filter, void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream) {
  unsigned char* base = static_cast<unsigned char*>(scratch);
  PackParams q = make_params(g, l);
  pack_f32_kernel<<<grid_for(q.Kp * q.Co_pad), 256, 0, stream>>>(
      filter, reinterpret_cast<float*>(base + l.filter_off),
      reinterpret_cast<int32_t*>(base + l.koff_off), reinterpret_cast<uint32_t*>(base), q);
  return cudaGetLastError();
}

cudaError_t launch_pack_f16(const uint16_t* filter, void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream) {
  unsigned char* base = static_cast<unsigned char*>(scratch);
  PackParams q = make_params(g, l);
  pack_f16_kernel<<<grid_for(q.Kp * q.Co), 256, 0, stream>>>(
      filter, reinterpret_cast<uint16_t*>(base + l.filter_off),
      reinterpret_cast<int32_t*>(base + l.koff_off), reinterpret_cast<uint32_t*>(base), q);
  return cudaGetLastError();
}

static cudaError_t pack_shift_common(const uint16_t* filter, void* scratch, const Geometry& g,
                                     const ScratchLayout& l, int raw_pitch, int nslot, cudaStream_t stream) {
  unsigned char* base = static_cast<unsigned char*>(scratch);
  PackParams q = make_params(g, l);
  int chunk = 512;                                          // k2 per block: staging of chunk*Kw halves within 40 KB
  while (chunk > 8 && (size_t)chunk * g.Kw * sizeof(uint16_t) > 40 * 1024) chunk /= 2;
  const size_t smem = ((size_t)chunk * g.Kw + 16) * sizeof(uint16_t);
  if (smem > 48 * 1024) return cudaErrorInvalidValue;
  dim3 grid((unsigned)((q.Kp + chunk - 1) / chunk), (unsigned)(g.Co < 32768 ? g.Co : 32768));
  pack_f16_shift_kernel<<<grid, 256, smem, stream>>>(filter, reinterpret_cast<uint16_t*>(base + l.filter_off),
                                                     reinterpret_cast<uint32_t*>(base + l.koff_off),
                                                     reinterpret_cast<uint32_t*>(base), q, raw_pitch, nslot, chunk);
  return cudaGetLastError();
}

cudaError_t launch_pack_f16_shift(const uint16_t* filter, void* scratch, const Geometry& g,
                                  const ScratchLayout& l, cudaStream_t stream) {
  return pack_shift_common(filter, scratch, g, l, 0, 0, stream);
}

cudaError_t launch_pack_f16_raw(const uint16_t* filter, void* scratch, const Geometry& g,
                                const ScratchLayout& l, const RawPlan& plan, cudaStream_t stream) {
  return pack_shift_common(filter, scratch, g, l, plan.pitch, plan.nslot, stream);
}

}  // namespace im2win
