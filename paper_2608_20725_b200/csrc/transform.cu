// im2win data transformation (paper Eq. 2) for sm_100a.
//
//   window[n][c][ho][k*Kh + u] = Xpad[n][c][ho*s + u][k]
//
// The window tensor is one flat array of "columns": column g = (strip, k) with
// strip = (n*C + c)*Ho + ho holds the Kh elements {u = 0..Kh-1} at flat offset
// g*Kh.  A CTA owns a contiguous range of columns, hence a contiguous range of
// the output.  Its threads gather the Kh inputs of one column at a time
// (lanes walk k, so every input row is read as coalesced runs), place them in
// shared memory in output order, and the CTA then streams the staged range to
// HBM with 16-byte stores.  The kernel is HBM-bound: the input is read once
// from DRAM (re-reads by overlapping strips hit L1/L2) and the window tensor
// is written once.
#include "common.cuh"

namespace im2win {
namespace {

struct TransformParams {
  int32_t H, W, Wp, Kh, s, p, Ho;
  int32_t cols_per_cta;   // multiple of 8, so every CTA's output range starts 16-byte aligned
  int64_t total_cols;     // N*C*Ho*Wp
};

constexpr int kTransformThreads = 256;

template <typename E, int KH>
__global__ void __launch_bounds__(kTransformThreads)
transform_kernel(const E* __restrict__ x, E* __restrict__ win, TransformParams q) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  E* stage = reinterpret_cast<E*>(smem_raw);

  const int Kh = KH > 0 ? KH : q.Kh;
  const int64_t g0 = (int64_t)blockIdx.x * q.cols_per_cta;
  const int64_t left = q.total_cols - g0;
  const int ncols = left < q.cols_per_cta ? (int)left : q.cols_per_cta;

  // Mixed-radix position (plane, ho, k) of this thread's first column and the
  // digits of the per-iteration step (blockDim.x columns).
  const int64_t g = g0 + threadIdx.x;
  int64_t strip = g / q.Wp;
  int k = (int)(g - strip * q.Wp);
  int64_t plane = strip / q.Ho;
  int ho = (int)(strip - plane * q.Ho);
  const int step = kTransformThreads;
  const int dk = step % q.Wp;
  const int dstrip = step / q.Wp;
  const int dho = dstrip % q.Ho;
  const int dplane = dstrip / q.Ho;

  for (int i = threadIdx.x; i < ncols; i += step) {
    const int w = k - q.p;
    const bool w_ok = (unsigned)w < (unsigned)q.W;
    const int h0 = ho * q.s - q.p;
    const E* src = x + ((size_t)plane * q.H) * q.W + w;
    E* dst = stage + (size_t)i * Kh;
    if constexpr (KH > 0) {
      E v[KH];
#pragma unroll
      for (int u = 0; u < KH; ++u) {
        const int h = h0 + u;
        v[u] = 0;
        if (w_ok && (unsigned)h < (unsigned)q.H) v[u] = __ldg(src + (size_t)h * q.W);
      }
#pragma unroll
      for (int u = 0; u < KH; ++u) dst[u] = v[u];
    } else {
      for (int u = 0; u < Kh; ++u) {
        const int h = h0 + u;
        E v = 0;
        if (w_ok && (unsigned)h < (unsigned)q.H) v = __ldg(src + (size_t)h * q.W);
        dst[u] = v;
      }
    }
    k += dk;
    int carry = k >= q.Wp;
    k -= carry ? q.Wp : 0;
    ho += dho + carry;
    carry = ho >= q.Ho;
    ho -= carry ? q.Ho : 0;
    plane += dplane + carry;
  }
  __syncthreads();

  // Stream the staged, contiguous output range.
  const size_t bytes = (size_t)ncols * Kh * sizeof(E);
  unsigned char* out = reinterpret_cast<unsigned char*>(win) + (size_t)g0 * Kh * sizeof(E);
  const int nvec = (int)(bytes / 16);
  const uint4* s4 = reinterpret_cast<const uint4*>(smem_raw);
  uint4* o4 = reinterpret_cast<uint4*>(out);
  for (int v = threadIdx.x; v < nvec; v += step) __stcs(o4 + v, s4[v]);
  const int tail0 = nvec * (16 / (int)sizeof(E));
  const int nelem = ncols * Kh;
  E* oe = reinterpret_cast<E*>(out);
  for (int e = tail0 + threadIdx.x; e < nelem; e += step) oe[e] = stage[e];
}

template <typename E>
cudaError_t launch_typed(const void* x, void* window, const Geometry& g, cudaStream_t stream) {
  TransformParams q;
  q.H = g.H; q.W = g.W; q.Wp = g.Wp; q.Kh = g.Kh; q.s = g.s; q.p = g.p; q.Ho = g.Ho;
  q.total_cols = (int64_t)g.N * g.C * g.Ho * g.Wp;
  // about 16 KB of staged output per CTA, in whole columns, a multiple of 8 columns
  int cols = (int)(16384 / (g.Kh * sizeof(E)));
  cols = cols / 8 * 8;
  if (cols < 8) cols = 8;
  q.cols_per_cta = cols;
  const size_t smem = (size_t)cols * g.Kh * sizeof(E);
  const int64_t blocks = (q.total_cols + cols - 1) / cols;
  const E* xi = static_cast<const E*>(x);
  E* wo = static_cast<E*>(window);
  auto run = [&](auto kernel) -> cudaError_t {
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    kernel<<<(unsigned)blocks, kTransformThreads, smem, stream>>>(xi, wo, q);
    return cudaGetLastError();
  };
  switch (g.Kh) {
    case 1: return run(transform_kernel<E, 1>);
    case 3: return run(transform_kernel<E, 3>);
    case 5: return run(transform_kernel<E, 5>);
    case 7: return run(transform_kernel<E, 7>);
    case 11: return run(transform_kernel<E, 11>);
    default: return run(transform_kernel<E, 0>);
  }
}

}  // namespace

cudaError_t launch_transform(const void* x, void* window, const Geometry& g, int elem_bytes,
                             cudaStream_t stream) {
  if (elem_bytes == 4) return launch_typed<uint32_t>(x, window, g, stream);
  return launch_typed<uint16_t>(x, window, g, stream);
}

}  // namespace im2win
