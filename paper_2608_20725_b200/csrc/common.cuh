// Shared host-side definitions of the im2win library: derived geometry,
// scratch layout and launch prototypes.  Device code lives in the .cu files.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/im2win.h"

namespace im2win {

// Quantities derived from an im2win_shape (notation of the paper's Section
// "Notation" and Eq. 2/3): Wp = W + 2p, strip = Kh*Wp elements per (n,c,ho),
// T = Kh*Kw window elements per channel, K = C*T reduction length,
// P = N*Ho*Wo output positions.
struct Geometry {
  int32_t N, C, H, W, Co, Kh, Kw, s, p;
  int32_t Ho, Wo, Wp, T;
  int64_t strip;         // Kh*Wp
  int64_t chan_stride;   // Ho*strip: distance between channels of one image in the window tensor
  int64_t img_stride;    // C*chan_stride
  int64_t K;             // C*T
  int64_t P;             // N*Ho*Wo
  int64_t window_elems;  // N*img_stride
  int64_t out_elems;     // N*Co*Ho*Wo
};

// Scratch layout shared by both precisions (offsets in bytes from `scratch`):
//   [0, 256)            status block (uint32 words; word 0 = timeout flag)
//   [256, 256 + 4*Kp)   k -> element offset table (int32), -1 for padded k
//   [filter_off, ...)   repacked filter
struct ScratchLayout {
  int64_t Kp;            // reduction length rounded up to the k-block of the kernel
  int64_t Co_pad;        // Co rounded up to the filter tile of the kernel
  size_t koff_off, filter_off, total;
  bool f16_shift;        // fp16 only: a shifted-view kernel (and its filter layout) is used
  bool f16_raw;          // fp16 only: the bulk-copy variant of the shifted-view kernel is used
  bool f16_mat;          // fp16 only: the matrix-transpose variant is used (own scratch layout)
  bool f16_stem;         // fp16 only: the one-k-block kernel for C*Kh <= 64 is used (filter layout of f16_shift)
};

// Tile geometry of the fp16 shifted-view kernel for one layer (see conv_f16_shift.cu).
struct ShiftPlan {
  bool eligible;
  int32_t Wq;            // virtual positions per strip = ceil(Wp / s)
  int32_t rows;          // rows of one shared-memory sub-tile: 128 + halo, multiple of 8
  int32_t total_rows;    // s * rows
  int32_t items;         // 16-byte chunks each producer thread fills per stage
  int32_t chunks;        // 16-byte chunks staged per row (8, fewer when one short k-block is all)
  int32_t nks_last;      // 16-wide MMA steps of the last k-block
  int64_t K2, K2p;       // C*Kh and its round-up to 64
  int64_t VQ;            // N*Ho*Wq virtual positions
};
ShiftPlan plan_f16_shift(const Geometry& g);

// Tile geometry of the bulk-copy shifted-view kernel (see conv_f16_raw.cu).
struct RawPlan {
  bool eligible;
  int32_t Wq, rows;
  int32_t nslot, pitch, raw_stage_bytes, a_stage_bytes;
  int64_t K2, K2p, VQ;
};
RawPlan plan_f16_raw(const Geometry& g);

// Tile geometry of the matrix-transpose shifted-view kernel (see conv_f16_mat.cu).
struct MatPlan {
  bool eligible;
  int32_t Wq, rows, R, Cp8, nch_last, nplanes, box_bytes, raw_stage_bytes, a_stage_bytes, num_kb;
  int64_t K2p, VQ;
  size_t scratch_bytes;  // status block + packed filter
};
MatPlan plan_f16_mat(const Geometry& g);

// Tile geometry of the one-k-block kernel for layers with C*Kh <= 64 (see conv_f16_stem.cu).
struct StemPlan {
  bool eligible;
  int32_t Wq, ragged, rows, R, nks, chan_region, raw_stage_bytes, a_stage_bytes, b_stage_bytes, bn;
  int32_t sa, rs, sb, resident, smem_bytes, epi_bufs;
  int64_t VQ;
};
StemPlan plan_f16_stem(const Geometry& g);

// Tile geometry of the channel-innermost (NHWC) path (see nhwc.cu).
struct NhwcPlan {
  bool eligible;
  bool pair;               // CTA pairs (cta_group::2)
  int32_t Cp;              // stored channels: C rounded up to 8
  int32_t num_kb;          // 64-wide k-blocks of K
  int32_t tw, bw, G;       // tw tiles of bw output columns along a strip; G strips per tile
  int32_t bn, ntn;         // channel tile and their number
  int32_t ksplit, kb_per_split;
  int64_t K;               // Kw*Kh*Cp
  int64_t strip;           // Wp*Kh*Cp halves per (n, ho)
  int64_t window_elems;    // N*Ho*strip
  int64_t ntm;             // position tiles
  size_t flags_off;        // byte offset of the tail-tile flag words inside the scratch
  size_t partial_off;      // byte offset and size of the partial-sum area (0 bytes: layer of many rounds of tiles)
  size_t partial_bytes;
  size_t scratch_bytes;    // status block + packed filter + flag words + partial sums
};
NhwcPlan plan_nhwc(const Geometry& g);

// What the convolution does with a finished accumulator (last step of the paper's Algorithm 1).
struct EpilogueArgs {
  const float* bias;       // device, Co floats, or nullptr
  int32_t relu;            // 1: max(y, 0) after the bias
  int32_t out16;           // 1: store binary16 (round to nearest even), 0: binary32
  int32_t y_nhwc;          // 1: y is [N][Ho][Wo][Co], 0: [N][Co][Ho][Wo]
};

// Tile shape of the fp32 kernel for a layer (see conv_f32.cu); the packed filter's K is padded to bk.
struct F32Plan {
  int32_t bm, bn, bk;
  bool klanes;             // the window operand is gathered with k along the lanes of a warp
  bool tall;               // 16 positions x 8 channels per thread (position pairs packed)
};
F32Plan plan_f32(const Geometry& g);

// Environment switches are testing aids: they are looked at only when IM2WIN_DEBUG is set in the
// environment (checked once per process), so the default call path reads no environment.
const char* debug_getenv(const char* name);

constexpr int kStatusBytes = 256;
constexpr int kF32KBlock = 16;     // smallest k-block of the fp32 kernel (see plan_f32)
constexpr int kF16KBlock = 64;     // k-block of the fp16 kernel (64 halves = one 128-byte swizzle row)

im2win_status derive_geometry(const im2win_shape* s, Geometry* g);
im2win_status scratch_layout(const Geometry& g, im2win_dtype dtype, ScratchLayout* l);

// Kernel launchers (each queues work on `stream` and returns the launch status).
cudaError_t launch_transform(const void* x, void* window, const Geometry& g, int elem_bytes,
                             cudaStream_t stream);
cudaError_t launch_pack_f32(const float* filter, void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_pack_f16(const uint16_t* filter, void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_conv_f32(const float* window, float* y, const void* scratch, const Geometry& g,
                            const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_pack_f16_shift(const uint16_t* filter, void* scratch, const Geometry& g,
                                  const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_pack_f16_raw(const uint16_t* filter, void* scratch, const Geometry& g,
                                const ScratchLayout& l, const RawPlan& plan, cudaStream_t stream);
cudaError_t launch_conv_f16_raw(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                const ScratchLayout& l, cudaStream_t stream);
// Matrix-transpose kernel: filter pack into `scratch` (own layout) and the convolution on it.
cudaError_t launch_pack_f16_mat(const uint16_t* filter, void* scratch, const Geometry& g, cudaStream_t stream);
cudaError_t launch_conv_f16_mat(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                cudaStream_t stream);
cudaError_t launch_conv_f16_stem(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                 const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_conv_f16_gather(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                   const ScratchLayout& l, cudaStream_t stream);
cudaError_t launch_conv_f16_shift(const uint16_t* window, float* y, void* scratch, const Geometry& g,
                                  const ScratchLayout& l, cudaStream_t stream);

cudaError_t launch_transform_nhwc(const uint16_t* x, int x_is_nhwc, uint16_t* window, const Geometry& g,
                                  cudaStream_t stream);
const char* nhwc_kernel_name(const Geometry& g, const EpilogueArgs& epi);
cudaError_t launch_pack_f16_nhwc(const uint16_t* filter, void* scratch, const Geometry& g, cudaStream_t stream);
cudaError_t launch_conv_f16_nhwc(const uint16_t* window, void* y, void* scratch, const Geometry& g,
                                 const EpilogueArgs& epi, cudaStream_t stream);

}  // namespace im2win
