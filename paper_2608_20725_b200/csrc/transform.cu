// im2win data transformation (paper Eq. 2) for sm_100a.
//
//   window[n][c][ho][k*Kh + u] = Xpad[n][c][ho*s + u][k]
//
// Two kernels.  The strip kernel (default) gives every CTA a run of whole strips
// (n, c, ho): sub-warps walk the columns of a strip (lanes = consecutive k, so
// each input row is read as coalesced runs; the Kh rows of a column come from
// L1/L2 when neighbouring strips re-read them; four items per thread are loaded
// before the first is stored), pack the Kh (fp32) or 2*Kh (fp16, two columns)
// elements of an item into 32-bit words and store them into a
// shared-memory staging buffer laid out exactly like the output range -- same
// 16-byte phase as the global address.  The 16-byte-aligned body of the range
// then leaves with ONE bulk asynchronous copy (cp.async.bulk shared -> global)
// issued by one thread; only the ragged head and tail (< 16 bytes each) are
// stored by hand.  The column kernel below serves kernel heights other than
// 1, 3, 5 and strips too long to stage.
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
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace im2win {
namespace {

// Predicated read-only load: the element if `ok`, else 0.  One predicated instruction instead
// of a branch around the load, and no memory request at all when the predicate is off.
__device__ __forceinline__ uint32_t ld_if(const uint32_t* p, bool ok) {
  uint32_t v = 0;
  asm("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p ld.global.nc.b32 %0, [%1];\n\t}"
      : "+r"(v)
      : "l"(p), "r"((int)ok));
  return v;
}
__device__ __forceinline__ uint16_t ld_if(const uint16_t* p, bool ok) {
  uint16_t v = 0;
  asm("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p ld.global.nc.u16 %0, [%1];\n\t}"
      : "+h"(v)
      : "l"(p), "r"((int)ok));
  return v;
}

__device__ __forceinline__ uint4 ld_if128(const void* p, bool ok) {
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  asm("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t@p ld.global.nc.v4.b32 {%0, %1, %2, %3}, [%4];\n\t}"
      : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w)
      : "l"(p), "r"((int)ok));
  return v;
}

__device__ __forceinline__ uint2 ld_if64(const void* p, bool ok) {
  uint2 v = make_uint2(0u, 0u);
  asm("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %3, 0;\n\t@p ld.global.nc.v2.b32 {%0, %1}, [%2];\n\t}"
      : "+r"(v.x), "+r"(v.y)
      : "l"(p), "r"((int)ok));
  return v;
}

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
        v[u] = ld_if(src + (size_t)h * q.W, w_ok && (unsigned)h < (unsigned)q.H);
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


// ------------------------------------------------------------------ strip kernel
struct StripParams {
  int32_t H, W, Wp, Kh, s, p, Ho;
  int32_t L;                 // Kh*Wp elements per strip
  int32_t strips_per_cta;
  int32_t group;             // threads that walk one strip together: a power of two <= 256
  int64_t total_strips;      // N*C*Ho
};

constexpr int kStripThreads = 256;
// items per thread whose loads are issued before the first store: fewer for tall kernels (registers)
__host__ __device__ constexpr int strip_unroll(int kh, int es) { return (4 / es) * kh > 10 ? 2 : 4; }

// Output order of a run of columns whose KH rows were loaded as one vector of NW 32-bit words
// each (r[row][word]): element n of the run is row n % KH, column n / KH.
template <int KH, int NW>
__device__ __forceinline__ uint32_t run_word32(const uint32_t (&r)[KH][NW], int n) {
  return r[n % KH][n / KH];
}
// 32-bit word made of halves n0 (low) and n1 (high) of a run of 2-byte elements.
template <int KH, int NW>
__device__ __forceinline__ uint32_t run_pair16(const uint32_t (&r)[KH][NW], int n0, int n1) {
  const uint32_t a = r[n0 % KH][(n0 / KH) >> 1], b = r[n1 % KH][(n1 / KH) >> 1];
  const uint32_t sel = (((n0 / KH) & 1) ? 0x32u : 0x10u) | (((n1 / KH) & 1) ? 0x7600u : 0x5400u);
  return __byte_perm(a, b, sel);
}

// VB > 0: the input rows are read as aligned VB-byte vectors (16 or 8; the row length must be a
// multiple of VB bytes so that every row starts aligned): one load per kernel row brings VB/ES
// columns, which leave as a contiguous run of KH*VB/ES output elements.  Per element that is
// well under half the instructions of the element-wise form (VB = 0), which is what bounds
// this kernel.
template <typename E, int KH, int VB>
__global__ void __launch_bounds__(kStripThreads, KH >= 7 ? 4 : 0)   // (tall kernels: four CTAs per SM; they would otherwise take 76-128 registers and run three)
transform_strips_kernel(const E* __restrict__ x, E* __restrict__ win, StripParams q) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int ES = (int)sizeof(E);
  constexpr int CPL = 4 / ES;                     // columns per item: one 32-bit word per kernel row
  constexpr int U = strip_unroll(KH, ES);

  const int64_t s0 = (int64_t)blockIdx.x * q.strips_per_cta;
  const int64_t left = q.total_strips - s0;
  const int ns = left < q.strips_per_cta ? (int)left : q.strips_per_cta;
  const int64_t out_byte0 = s0 * q.L * ES;        // first output byte of this CTA
  const int mis = (int)(out_byte0 & 15);          // staging mirrors the 16-byte phase of the output
  unsigned char* stage = smem_raw + mis;

  // A group of G threads walks one strip, U items per thread and pass; 256/G strips are in
  // flight per pass.  Strip index -> (plane, ho) by one 32-bit division relative to the CTA's first strip.
  const int G = q.group;
  const int grp = threadIdx.x / G, gl = threadIdx.x - grp * G;
  const int ngrp = kStripThreads / G;
  const int64_t plane0 = s0 / q.Ho;
  const int ho0 = (int)(s0 - plane0 * q.Ho);
  const int64_t plane_elems = (int64_t)q.H * q.W;

  for (int ls = grp; ls < ns; ls += ngrp) {
    const int t = ho0 + ls;
    const int dpl = t / q.Ho;
    const int ho = t - dpl * q.Ho;
    const int h0 = ho * q.s - q.p;
    const E* __restrict__ src = x + (plane0 + dpl) * plane_elems;
    const int sbyte = ls * q.L * ES;              // byte offset of the strip inside the staging
    unsigned char* dst_strip = stage + sbyte;
    const bool word_ok = ((mis + sbyte) & 3) == 0;
    if constexpr (VB > 0) {
      constexpr int VL = VB / ES;                 // columns per vector
      constexpr int NW = VB / 4;                  // 32-bit words per vector
      constexpr int VU = KH <= 3 ? 32 / VB : 1;   // vectors per thread whose loads precede the first store
      constexpr int RUN = VL * KH;                // output elements per vector
      const int nvec = q.W / VL;
      // padded columns on both sides of the strip: p*KH zeros each
      const int padel = q.p * KH;
      for (int e = gl; e < padel; e += G) {
        reinterpret_cast<E*>(dst_strip)[e] = (E)0;
        reinterpret_cast<E*>(dst_strip)[q.L - padel + e] = (E)0;
      }
      const bool aligned4 = ES == 4 || ((mis + sbyte + padel * ES) & 3) == 0;
      for (int vb = gl; vb < nvec; vb += G * VU) {
        uint32_t r[VU][KH][NW];
#pragma unroll
        for (int j = 0; j < VU; ++j) {
          const int vi = vb + j * G;
#pragma unroll
          for (int u = 0; u < KH; ++u) {
            const int h = h0 + u;
            const bool ok = vi < nvec && (unsigned)h < (unsigned)q.H;
            if constexpr (VB == 16) {
              const uint4 t = ld_if128(src + (int64_t)h * q.W + vi * VL, ok);
              r[j][u][0] = t.x; r[j][u][1] = t.y; r[j][u][2] = t.z; r[j][u][3] = t.w;
            } else {
              const uint2 t = ld_if64(src + (int64_t)h * q.W + vi * VL, ok);
              r[j][u][0] = t.x; r[j][u][1] = t.y;
            }
          }
        }
#pragma unroll
        for (int j = 0; j < VU; ++j) {
          const int vi = vb + j * G;
          if (vi >= nvec) break;
          unsigned char* d = dst_strip + (size_t)(vi * VL + q.p) * KH * ES;
          if constexpr (ES == 4) {
#pragma unroll
            for (int n = 0; n < RUN; ++n) reinterpret_cast<uint32_t*>(d)[n] = run_word32<KH, NW>(r[j], n);
          } else {
            if (aligned4) {
#pragma unroll
              for (int w = 0; w < RUN / 2; ++w)
                reinterpret_cast<uint32_t*>(d)[w] = run_pair16<KH, NW>(r[j], 2 * w, 2 * w + 1);
            } else {
              // the run starts on an odd half: one half, RUN/2 - 1 words, one half
              reinterpret_cast<uint16_t*>(d)[0] = (uint16_t)(run_pair16<KH, NW>(r[j], 0, 0) & 0xffffu);
#pragma unroll
              for (int w = 0; w < RUN / 2 - 1; ++w)
                reinterpret_cast<uint32_t*>(d + 2)[w] = run_pair16<KH, NW>(r[j], 2 * w + 1, 2 * w + 2);
              reinterpret_cast<uint16_t*>(d)[RUN - 1] = (uint16_t)(run_pair16<KH, NW>(r[j], RUN - 1, RUN - 1) & 0xffffu);
            }
          }
        }
      }
    } else {
    for (int kbase = gl * CPL; kbase < q.Wp; kbase += G * CPL * U) {
      E v[U][CPL][KH];
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int k = kbase + j * G * CPL;
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
          const int w = k + c - q.p;
          const bool w_ok = (unsigned)w < (unsigned)q.W;     // also false beyond the strip
#pragma unroll
          for (int u = 0; u < KH; ++u) {
            const int h = h0 + u;
            v[j][c][u] = ld_if(src + h * q.W + w, w_ok && (unsigned)h < (unsigned)q.H);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < U; ++j) {
        const int k = kbase + j * G * CPL;
        if (k >= q.Wp) break;
        unsigned char* d = dst_strip + (size_t)k * KH * ES;
        if constexpr (ES == 4) {
#pragma unroll
          for (int u = 0; u < KH; ++u) reinterpret_cast<uint32_t*>(d)[u] = (uint32_t)v[j][0][u];
        } else {
          if (word_ok && k + 1 < q.Wp) {
#pragma unroll
            for (int jj = 0; jj < KH; ++jj) {        // word jj holds elements 2jj, 2jj+1 of the 2*KH run
              const int e0 = 2 * jj, e1 = 2 * jj + 1;
              const uint32_t lo = (uint32_t)(e0 < KH ? v[j][0][e0] : v[j][1][e0 - KH]);
              const uint32_t hi = (uint32_t)(e1 < KH ? v[j][0][e1] : v[j][1][e1 - KH]);
              reinterpret_cast<uint32_t*>(d)[jj] = lo | (hi << 16);
            }
          } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c)
              if (k + c < q.Wp) {
#pragma unroll
                for (int u = 0; u < KH; ++u) reinterpret_cast<E*>(d)[c * KH + u] = v[j][c][u];
              }
          }
        }
      }
    }
    }
  }
  // Make the generic-proxy writes visible to the bulk-copy engine, then meet.
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  // The 16-byte-aligned body leaves with one bulk copy.
  const int total = ns * q.L * ES;
  int head = (16 - mis) & 15;
  if (head > total) head = total;
  const int body = (total - head) & ~15;
  const int tail = total - head - body;
  unsigned char* gout = reinterpret_cast<unsigned char*>(win) + out_byte0;
  if (threadIdx.x == 0 && body > 0) {
    const uint32_t saddr = (uint32_t)__cvta_generic_to_shared(stage + head);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gout + head), "r"(saddr),
                 "r"(body)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
  // ragged ends, element by element (never more than 15 bytes each)
  if ((int)threadIdx.x * ES < head)
    reinterpret_cast<E*>(gout)[threadIdx.x] = reinterpret_cast<const E*>(stage)[threadIdx.x];
  if ((int)threadIdx.x * ES < tail) {
    const int o = head + body;
    reinterpret_cast<E*>(gout + o)[threadIdx.x] = reinterpret_cast<const E*>(stage + o)[threadIdx.x];
  }
  // the staging buffer must outlive the bulk copy's reads
  if (threadIdx.x == 0 && body > 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// The strip kernel is used for the kernel heights it is instantiated for, when a strip can be
// staged; measured faster than the column kernel for Kh <= 5 and slower beyond (register
// pressure of the unrolled gathers), so taller kernels keep the column kernel.
template <typename E>
bool plan_strips(const Geometry& g, StripParams* q, size_t* smem_bytes, int* vec) {
  constexpr int ES = (int)sizeof(E);
  if (!(g.Kh == 1 || g.Kh == 3 || g.Kh == 5 || g.Kh == 7 || g.Kh == 11)) return false;
  const int64_t strip_bytes = g.strip * ES;
  const int64_t total_strips = (int64_t)g.N * g.C * g.Ho;
  if (strip_bytes > 64 * 1024 || total_strips >= ((int64_t)1 << 31)) return false;
  // Staged output per CTA.  A CTA's life is one round of loads, a barrier and one bulk store, so with 16 KB
  // per CTA the kernel was bound by CTA turnaround, most visibly on short strips of tall kernels (11x11 on
  // 28x28 images in fp16: 836-byte strips, 24 k CTAs, 123 us; 93 us with 48 KB).  Measured per config: 32 KB
  // is 1-4 % faster than 16 KB nearly everywhere, 48 KB (just under the default shared-memory limit) wins in
  // fp16 for kernels 7 and 11 high (cfg3 54 -> 44 us, cfg5k7 79 -> 61) and for large images (3x3 at 112x112:
  // 339 -> 291 us) and loses 5-7 % on 28x28 images with 5x5 kernels and on 7x7 images.
  int64_t stage_bytes = (ES == 2 && (g.Kh >= 7 || (int64_t)g.H * g.W >= 2048)) ? 48 * 1024 - 64 : 32 * 1024;
  if (const char* v = debug_getenv("IM2WIN_TRANSFORM_STAGE")) { const int64_t b = atoll(v); if (b >= 4096 && b <= 160 * 1024) stage_bytes = b; }   // testing aid
  int r = (int)(stage_bytes / strip_bytes);
  if (r < 1) r = 1;
  q->H = g.H; q->W = g.W; q->Wp = g.Wp; q->Kh = g.Kh; q->s = g.s; q->p = g.p; q->Ho = g.Ho;
  q->L = (int32_t)g.strip;
  q->total_strips = total_strips;
  q->strips_per_cta = r;
  // vector loads: rows must start 16- (or 8-) byte aligned; IM2WIN_TRANSFORM_SCALAR forces the
  // element-wise form (a testing aid)
  *vec = 0;
  if (debug_getenv("IM2WIN_TRANSFORM_SCALAR") == nullptr && (ES == 2 || g.Kh <= 3)) {   // fp32, Kh > 3: measured slower
    if ((g.W * ES) % 16 == 0) *vec = 16;
    else if (ES == 2 && (g.W * ES) % 8 == 0) *vec = 8;      // 8-byte vectors of 4-byte elements measured slower
  }
  const int items = *vec ? g.W * ES / *vec : (g.Wp + (4 / ES) - 1) / (4 / ES);
  const int unroll = *vec ? (g.Kh <= 3 ? 32 / *vec : 1) : strip_unroll(g.Kh, ES);
  if (!*vec && g.Kh > 5) return false;          // element-wise strips are slower than columns for tall kernels
  const int per_group = (items + unroll - 1) / unroll;
  int grp = 1;
  while (grp < kStripThreads && grp < per_group) grp *= 2;
  q->group = grp;
  *smem_bytes = (size_t)(r * strip_bytes + 16);
  return true;
}

template <typename E>
cudaError_t launch_strips(const void* x, void* window, const StripParams& q, size_t smem, int Kh, int vec,
                          cudaStream_t stream) {
  const int64_t blocks = (q.total_strips + q.strips_per_cta - 1) / q.strips_per_cta;
  const E* xi = static_cast<const E*>(x);
  E* wo = static_cast<E*>(window);
  auto run = [&](auto kernel) -> cudaError_t {
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    kernel<<<(unsigned)blocks, kStripThreads, smem, stream>>>(xi, wo, q);
    return cudaGetLastError();
  };
  if (vec == 16) {
    switch (Kh) {
      case 1: return run(transform_strips_kernel<E, 1, 16>);
      case 3: return run(transform_strips_kernel<E, 3, 16>);
      case 5: return run(transform_strips_kernel<E, 5, 16>);
      case 7: return run(transform_strips_kernel<E, 7, 16>);
      default: return run(transform_strips_kernel<E, 11, 16>);
    }
  }
  if (vec == 8) {
    switch (Kh) {
      case 1: return run(transform_strips_kernel<E, 1, 8>);
      case 3: return run(transform_strips_kernel<E, 3, 8>);
      case 5: return run(transform_strips_kernel<E, 5, 8>);
      case 7: return run(transform_strips_kernel<E, 7, 8>);
      default: return run(transform_strips_kernel<E, 11, 8>);
    }
  }
  switch (Kh) {
    case 1: return run(transform_strips_kernel<E, 1, 0>);
    case 3: return run(transform_strips_kernel<E, 3, 0>);
    default: return run(transform_strips_kernel<E, 5, 0>);
  }
}

template <typename E>
cudaError_t launch_typed(const void* x, void* window, const Geometry& g, cudaStream_t stream) {
  TransformParams q;
  q.H = g.H; q.W = g.W; q.Wp = g.Wp; q.Kh = g.Kh; q.s = g.s; q.p = g.p; q.Ho = g.Ho;
  q.total_cols = (int64_t)g.N * g.C * g.Ho * g.Wp;
  // about 32 KB of staged output per CTA (16 KB: 2-9 % slower, CTA turnaround; 48 KB: slower again), in whole
  // columns, a multiple of 8 columns
  int64_t stage_bytes = 32768;
  if (const char* v = debug_getenv("IM2WIN_TRANSFORM_STAGE")) { const int64_t b = atoll(v); if (b >= 4096 && b <= 160 * 1024) stage_bytes = b; }   // testing aid
  int cols = (int)(stage_bytes / (g.Kh * sizeof(E)));
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
  // Strips that fit a staging buffer go to the strip kernel; IM2WIN_TRANSFORM_KERNEL=columns
  // forces the fallback (a testing aid).
  const char* force = debug_getenv("IM2WIN_TRANSFORM_KERNEL");
  const bool columns = force && strcmp(force, "columns") == 0;
  StripParams q;
  size_t smem = 0;
  int vec = 0;
  if (elem_bytes == 4) {
    if (!columns && plan_strips<uint32_t>(g, &q, &smem, &vec))
      return launch_strips<uint32_t>(x, window, q, smem, g.Kh, vec, stream);
    return launch_typed<uint32_t>(x, window, g, stream);
  }
  if (!columns && plan_strips<uint16_t>(g, &q, &smem, &vec))
    return launch_strips<uint16_t>(x, window, q, smem, g.Kh, vec, stream);
  return launch_typed<uint16_t>(x, window, g, stream);
}

}  // namespace im2win
