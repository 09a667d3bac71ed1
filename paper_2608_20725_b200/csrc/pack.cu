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

// Layout of the shifted-view fp16 kernel: Fp2[v][co][k2], k2 = c*Kh + u (zero padded to K2p),
// and the table k2 -> c*chan_stride + u.
__global__ void pack_f16_shift_kernel(const uint16_t* __restrict__ f, uint16_t* __restrict__ fp,
                                      int32_t* __restrict__ koff, uint32_t* __restrict__ status,
                                      PackParams q) {
  if (blockIdx.x == 0 && threadIdx.x < kStatusBytes / 4) status[threadIdx.x] = 0u;
  const int64_t K2 = (int64_t)q.C * q.Kh;
  const int64_t per_v = q.Kp * q.Co;
  const int64_t total = per_v * q.Kw;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t v = i / per_v;
    const int64_t r = i - v * per_v;
    const int64_t co = r / q.Kp;
    const int64_t k2 = r - co * q.Kp;
    uint16_t val = 0;
    int32_t off = -1;
    if (k2 < K2) {
      const int64_t c = k2 / q.Kh;
      const int64_t u = k2 - c * q.Kh;
      val = f[((co * q.C + c) * q.Kh + u) * q.Kw + v];
      off = (int32_t)(c * q.chan_stride + u);
    }
    fp[i] = val;
    if (v == 0 && co == 0) koff[k2] = off;
  }
}

// Table of the TMA-staged fp16 kernel: k2 -> byte offset of element (c, u) inside a raw box,
// slot (c - first channel of the k-block) * pitch + u*2; padded k2 point at the all-zero slot
// `nslot`.
__global__ void rawtab_kernel(uint32_t* __restrict__ tab, int64_t K2, int64_t K2p, int Kh, int pitch, int nslot,
                              int cs16) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t k2 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k2 < K2p; k2 += stride) {
    uint32_t e = (uint32_t)(nslot * pitch);
    if (k2 < K2) {
      const int64_t c = k2 / Kh;
      const int u = (int)(k2 - c * Kh);
      const int64_t c_lo = (k2 / kF16KBlock) * kF16KBlock / Kh;
      e = (uint32_t)((c - c_lo) * pitch + u * 2);
    }
    tab[k2] = e;
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

cudaError_t launch_pack_f16_shift(const uint16_t* filter, void* scratch, const Geometry& g,
                                  const ScratchLayout& l, cudaStream_t stream) {
  unsigned char* base = static_cast<unsigned char*>(scratch);
  PackParams q = make_params(g, l);
  pack_f16_shift_kernel<<<grid_for(q.Kp * q.Co * q.Kw), 256, 0, stream>>>(
      filter, reinterpret_cast<uint16_t*>(base + l.filter_off),
      reinterpret_cast<int32_t*>(base + l.koff_off), reinterpret_cast<uint32_t*>(base), q);
  return cudaGetLastError();
}

cudaError_t launch_pack_f16_raw(const uint16_t* filter, void* scratch, const Geometry& g,
                                const ScratchLayout& l, const RawPlan& plan, cudaStream_t stream) {
  // same filter layout as the shifted-view kernel; its offset table is then replaced by the raw table
  cudaError_t e = launch_pack_f16_shift(filter, scratch, g, l, stream);
  if (e != cudaSuccess) return e;
  unsigned char* base = static_cast<unsigned char*>(scratch);
  rawtab_kernel<<<grid_for(plan.K2p), 256, 0, stream>>>(reinterpret_cast<uint32_t*>(base + l.koff_off), plan.K2,
                                                        plan.K2p, g.Kh, plan.pitch, plan.nslot,
                                                        (int)((g.chan_stride * 2) & 15));
  return cudaGetLastError();
}

}  // namespace im2win
