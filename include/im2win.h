/*
 * im2win.h -- C ABI of the B200 (sm_100a) im2win convolution library.
 *
 * The library implements the hot path of the im2win convolution: the im2win
 * data transformation (paper Eq. 2) and the forward convolution over the
 * im2win tensor (paper Eq. 3, GEMM view of Algorithm 1) in two precisions:
 * fp32 on CUDA cores and fp16-input / fp32-accumulate on tensor cores.
 *
 * Problem statement (paper, Section "Notation"): input I[N][C][H][W], filter
 * F[Co][C][Kh][Kw] (OIHW), output O[N][Co][Ho][Wo], all row-major with the
 * last index fastest; one stride s for both axes; a symmetric zero padding p
 * (the paper's layers have p = 0).  Ho = floor((H + 2p - Kh) / s) + 1 and
 * likewise Wo.  The operation is a cross-correlation (Eq. 1, no kernel flip).
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer unless its name ends in _host.
 *     The caller owns all memory; the library allocates no device memory and
 *     keeps no per-call state (per device it keeps two auxiliary streams, see
 *     im2win_layer_forward_host, and the array of im2win_conv_f32_static).
 *     Buffers must stay valid until the work queued on `cuda_stream` has
 *     completed.
 *   - All calls are asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL is the default stream), except where stated.
 *   - Inputs are never written.  Output, window, scratch and input buffers
 *     must not overlap one another.
 *   - Device pointers must be 16-byte aligned, else IM2WIN_ERR_MISALIGNED.
 *   - Arguments are validated before anything is launched; on any error no
 *     device work has been queued by that call.
 *   - There is no CPU fallback: without a CUDA device the compute entry points
 *     return IM2WIN_ERR_CUDA.
 */
#ifndef IM2WIN_H_
#define IM2WIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t N, C, H, W;   /* input  [N][C][H][W]                          */
  int32_t Co, Kh, Kw;   /* filter [Co][C][Kh][Kw]                       */
  int32_t stride;       /* >= 1, same for both axes                     */
  int32_t pad;          /* >= 0, zero rows/columns added on every side  */
} im2win_shape;

typedef enum {
  IM2WIN_F32 = 0,       /* 4-byte elements, IEEE binary32 */
  IM2WIN_F16 = 1        /* 2-byte elements, IEEE binary16 */
} im2win_dtype;

typedef enum {
  IM2WIN_OK = 0,
  IM2WIN_ERR_INVALID_ARG = 1,         /* non-positive size, negative pad, Ho or Wo < 1, bad dtype */
  IM2WIN_ERR_NULL_POINTER = 2,
  IM2WIN_ERR_MISALIGNED = 3,          /* a device pointer is not 16-byte aligned */
  IM2WIN_ERR_WORKSPACE_TOO_SMALL = 4,
  IM2WIN_ERR_UNSUPPORTED = 5,         /* sizes beyond the kernels' index ranges */
  IM2WIN_ERR_CUDA = 6,                /* a CUDA call failed (no device, launch error) */
  IM2WIN_ERR_TIMEOUT = 7              /* a bounded device-side wait gave up (see im2win_check_status) */
} im2win_status;

/* Static, NUL-terminated description of a status code. */
const char* im2win_status_string(im2win_status status);

/*
 * Name of the convolution kernel the library selects for a layer (host-only,
 * launches nothing; static storage): "f32-ffma" for IM2WIN_F32; for IM2WIN_F16
 * one of the tensor-core kernels of Algorithm 1's GEMM view, "f16-stem",
 * "f16-mat", "f16-raw", "f16-shift" or "f16-gather"; "none" for an
 * invalid shape.  For reports and tests; the choice is an implementation detail.
 */
const char* im2win_conv_kernel_name(const im2win_shape* shape, im2win_dtype dtype);

/*
 * Sizes, in bytes, of the buffers a layer needs (host-only, launches nothing).
 *   window_bytes  = N*C*Ho*Kh*(W+2p) * sizeof(element): the closed-form size
 *                   of the im2win tensor (paper Eq. 2; Section "Im2win Data
 *                   Transformation"), with no hidden padding.
 *   scratch_bytes = what im2win_conv_f32 / im2win_conv_f16 need in `scratch`
 *                   (a status block, the repacked filter and an offset table).
 *   Ho, Wo        = output height and width.
 * Any of the four output pointers may be NULL.
 */
im2win_status im2win_workspace_size(const im2win_shape* shape, im2win_dtype dtype,
                                    size_t* window_bytes, size_t* scratch_bytes,
                                    int32_t* Ho, int32_t* Wo);

/*
 * im2win data transformation (paper Eq. 2, 0-based):
 *     window[n][c][ho][k*Kh + u] = Xpad[n][c][ho*s + u][k],
 *     k in [0, W+2p), u in [0, Kh),
 * where Xpad is x with p zero rows/columns on every side.  The result is
 * [N][C][Ho][Kh*(W+2p)]; every Kh x Kw sliding window of output row ho is the
 * contiguous run of Kh*Kw elements starting at (wo*s)*Kh.  Elements are moved
 * as bit patterns (NaN payloads and -0 are preserved); padding positions are
 * written as +0.  `x_nchw` holds N*C*H*W elements and `window` window_bytes
 * bytes, both of `dtype`.
 */
im2win_status im2win_transform(const void* x_nchw, void* window, const im2win_shape* shape,
                               im2win_dtype dtype, void* cuda_stream);

/*
 * Forward convolution over the im2win tensor, fp32 on CUDA cores
 * (paper Eq. 3; Section "im2win convolutions", the "CC" variant):
 *     y[n][co][ho][wo] = sum_c sum_{t < Kh*Kw} window[n][c][ho][(wo*s)*Kh + t] * Fp[co][c][t],
 *     Fp[co][c][v*Kh + u] = filter_oihw[co][c][u][v]   (height before width).
 * The filter is repacked into `scratch` on every call (part of the timed
 * operation).  `y_nchw` is [N][Co][Ho][Wo] fp32.  `scratch` must hold at least
 * the scratch_bytes reported by im2win_workspace_size(shape, IM2WIN_F32, ...).
 * Products and sums are fp32; the summation order is unspecified.
 */
im2win_status im2win_conv_f32(const float* window, const float* filter_oihw, float* y_nchw,
                              void* scratch, size_t scratch_bytes, const im2win_shape* shape,
                              void* cuda_stream);

/*
 * Forward convolution over the im2win tensor, fp16 inputs on tensor cores with
 * fp32 accumulation and fp32 output (paper Algorithm 1; Section "Im2win
 * Convolution on Tensor Cores", the "TC" variant; GEMM view M x N x K =
 * positions x Co x C*Kh*Kw).  `window` and `filter_oihw` hold IEEE binary16
 * bit patterns; `y_nchw` is [N][Co][Ho][Wo] fp32.  `scratch` as above with
 * IM2WIN_F16.  Device-side waits in this kernel are bounded; if one gives up
 * the kernel records it in the status block at the start of `scratch` and
 * returns early (see im2win_check_status).
 */
im2win_status im2win_conv_f16(const uint16_t* window, const uint16_t* filter_oihw, float* y_nchw,
                              void* scratch, size_t scratch_bytes, const im2win_shape* shape,
                              void* cuda_stream);

/*
 * The two halves of im2win_conv_f32 / im2win_conv_f16 for static weights (the
 * paper repacks the filter "height before width" once, Section "Im2win
 * Convolution"): im2win_pack_filter writes the packed filter (and clears the
 * status block) into `scratch`; im2win_conv_packed runs the convolution of
 * `dtype` on a filter packed earlier into the same `scratch` for the same
 * shape and dtype, any number of times.  `filter_oihw` and `window` hold
 * elements of `dtype` (binary16 bit patterns for IM2WIN_F16); arguments,
 * scratch size and errors as for the one-call forms.  The packed layout depends
 * on the kernel the library selects for the shape; both calls must come from
 * the same process with an unchanged environment.
 */
im2win_status im2win_pack_filter(const void* filter_oihw, void* scratch, size_t scratch_bytes,
                                 const im2win_shape* shape, im2win_dtype dtype, void* cuda_stream);
im2win_status im2win_conv_packed(const void* window, float* y_nchw, void* scratch, size_t scratch_bytes,
                                 const im2win_shape* shape, im2win_dtype dtype, void* cuda_stream);

/*
 * Synchronises `cuda_stream`, reads the status block at the start of `scratch`
 * (written by the last convolution call that used it) and returns
 * IM2WIN_ERR_TIMEOUT if a bounded device wait gave up, IM2WIN_ERR_CUDA if the
 * stream reports an error, else IM2WIN_OK.  Blocking.
 *
 * Layout of the status block (the first 256 bytes of `scratch`, 32-bit words,
 * all cleared by every filter pack): word 0 is raised by a wait that gave up.
 * Words 1 and 2 are testing aids read by the fp16 kernels: a non-zero word 1
 * replaces the number of polls after which a wait gives up (2^24, and never
 * more than about four seconds); the marker 0x0d0a11fe in word 2 makes the
 * one-k-block kernel leave out one barrier arrival, the marker 0x0d0a11ff makes
 * the NHWC shifted-view kernel keep down the flags its split tiles hand their
 * partial sums over with, so that a test can watch a wait run out and the
 * kernel return.  Nothing in the library writes them.
 */
im2win_status im2win_check_status(const void* scratch, void* cuda_stream);

/*
 * Size in bytes of the device workspace im2win_layer_forward_host needs for
 * one layer: input copy + window tensor + scratch + output, each rounded up
 * to 256 bytes (host-only, launches nothing).
 */
im2win_status im2win_layer_workspace_size(const im2win_shape* shape, im2win_dtype dtype,
                                          size_t* device_bytes);

/*
 * Whole layer from HOST buffers: copies x and the filter to the device
 * workspace, runs im2win_transform and the convolution of `dtype`, and copies
 * y back, all queued on `cuda_stream` (paper Sections "Im2win Data
 * Transformation" and "Im2win Convolution" back to back).  x_host and
 * filter_host hold elements of `dtype` (binary16 bit patterns for F16);
 * y_host receives N*Co*Ho*Wo floats.  Host buffers should be page-locked for
 * the copies to overlap nothing else; they must stay valid until the stream
 * has been synchronised by the caller.  `device_workspace` is a 256-byte
 * aligned device buffer of at least im2win_layer_workspace_size bytes.
 * Layers that move more than 8 MB are processed in four batch chunks: the
 * upload of a chunk, the kernels of the previous one and the download of the
 * one before overlap.  The copies of such a call run on two auxiliary streams
 * that the library creates once per device and keeps; they are ordered after
 * everything queued on `cuda_stream` before the call, and `cuda_stream` waits
 * for the last of them, so synchronising `cuda_stream` still completes the
 * call.  The result does not depend on the chunking.  Arguments and every
 * chunk's geometry are validated before anything is queued; should a CUDA call
 * fail after the first chunk was queued, the call still makes `cuda_stream`
 * wait for the auxiliary streams before it returns the error.
 */
im2win_status im2win_layer_forward_host(const void* x_host, const void* filter_host, float* y_host,
                                        void* device_workspace, size_t device_workspace_bytes,
                                        const im2win_shape* shape, im2win_dtype dtype,
                                        void* cuda_stream);

/* ------------------------------------------------------------------------
 * Channel-innermost (NHWC) form of the path, fp16 on tensor cores.
 *
 * The paper's tensor-core kernel works on NHWC data (Section "Im2win
 * Convolution on Tensor Cores"); the index map it prints (Eq. 2) is the NCHW
 * one.  The reading taken here is Eq. 2 with the channel moved to the fastest
 * position:
 *     window[n][ho][k][u][c] = Xpad[n][c][ho*s + u][k],
 *     k in [0, W+2p), u in [0, Kh), c in [0, Cp),  Cp = C rounded up to 8,
 * channels C..Cp-1 holding +0.  The Kh x Kw x C window of output (ho, wo) is
 * then the contiguous run of Kw*Kh*Cp elements that starts (wo*s)*Kh*Cp
 * elements into strip (n, ho), ordered (v, u, c): height before width as in
 * Eq. 3, the channel below both.  The tensor has N*Ho*(W+2p)*Kh*Cp elements:
 * the closed-form im2win size when C is a multiple of 8.
 */
typedef enum {
  IM2WIN_LAYOUT_NCHW = 0,   /* [N][C][H][W] */
  IM2WIN_LAYOUT_NHWC = 1    /* [N][H][W][C] */
} im2win_layout;

/*
 * What a convolution does with its finished fp32 accumulator (the last step
 * of the paper's Algorithm 1, "write C", whose output type the paper leaves
 * open): y = acc + bias[co] (if bias is not NULL), then max(y, 0) (if relu),
 * then the store, as binary32 or rounded once to binary16 (nearest, ties to
 * even), in NCHW or NHWC order.  A NULL epilogue means no bias, no ReLU,
 * binary32, NCHW.
 */
typedef struct {
  const float* bias;        /* DEVICE pointer to Co floats (16-byte aligned), or NULL */
  int32_t relu;             /* 0 or 1                                           */
  int32_t out_dtype;        /* IM2WIN_F32 or IM2WIN_F16: element type of y      */
  int32_t out_layout;       /* im2win_layout of y                               */
} im2win_epilogue;

/*
 * Buffer sizes of the NHWC form (host-only): window_bytes = N*Ho*(W+2p)*Kh*Cp*2,
 * scratch_bytes for im2win_conv_f16_nhwc (status block + repacked filter + flag
 * words + for layers of few rounds of tiles 19 MB for partial sums that CTAs
 * hand to one another), the output size and the stored channel count Cp.  Any
 * output pointer may be NULL.
 */
im2win_status im2win_nhwc_workspace_size(const im2win_shape* shape, size_t* window_bytes, size_t* scratch_bytes,
                                         int32_t* Ho, int32_t* Wo, int32_t* Cp);

/*
 * im2win transformation into the NHWC window tensor defined above, from an
 * input of binary16 bit patterns given as [N][C][H][W] or [N][H][W][C]
 * (`x_layout`).  Bit patterns are copied verbatim; padding positions and the
 * channels C..Cp-1 are written as +0.
 */
im2win_status im2win_transform_nhwc(const uint16_t* x, im2win_layout x_layout, uint16_t* window,
                                    const im2win_shape* shape, void* cuda_stream);

/*
 * Forward convolution over the NHWC window tensor on tensor cores (paper
 * Algorithm 1 in its GEMM view, M x N x K = positions x Co x Kw*Kh*Cp):
 *     acc[n][ho][wo][co] = sum_{t < Kw*Kh*Cp} window[n][ho][(wo*s)*Kh*Cp + t] * Fp[co][t],
 *     Fp[co][(v*Kh + u)*Cp + c] = filter_oihw[co][c][u][v]  (0 for c >= C),
 * fp16 products, fp32 accumulation, then `epilogue` (may be NULL).  `y` holds
 * N*Co*Ho*Wo elements of epilogue->out_dtype in epilogue->out_layout.  The
 * filter is repacked into `scratch` on every call.  Layers with few position
 * tiles split the reduction over several CTAs, which add their partial sums
 * into a `y` the call clears first (only without ReLU and with binary32
 * output; the summation order then varies from run to run).  A short last
 * round of tiles may instead be shared between CTAs by runs of the reduction:
 * the CTA that starts a tile adds the other CTAs' partial sums from `scratch`
 * in a fixed order and applies the epilogue (any epilogue; deterministic).
 * Waits are bounded as in im2win_conv_f16 (see im2win_check_status).
 * im2win_pack_filter_nhwc / im2win_conv_packed_nhwc are the two halves for
 * static weights.
 */
im2win_status im2win_conv_f16_nhwc(const uint16_t* window, const uint16_t* filter_oihw, void* y,
                                   const im2win_epilogue* epilogue, void* scratch, size_t scratch_bytes,
                                   const im2win_shape* shape, void* cuda_stream);
im2win_status im2win_pack_filter_nhwc(const uint16_t* filter_oihw, void* scratch, size_t scratch_bytes,
                                      const im2win_shape* shape, void* cuda_stream);
im2win_status im2win_conv_packed_nhwc(const uint16_t* window, void* y, const im2win_epilogue* epilogue,
                                      void* scratch, size_t scratch_bytes, const im2win_shape* shape,
                                      void* cuda_stream);

/*
 * Name of the kernel im2win_conv_f16_nhwc selects for a layer and an epilogue
 * (NULL: the plain one); host-only, launches nothing, static storage:
 * "f16-nhwc-shift" (row-shifted MMA views of columns staged once) or
 * "f16-nhwc-overlap" (a tensor map with overlapping rows), with "+ksplit" when
 * every tile's reduction is split over several CTAs or "+runs" when the tiles
 * of a short last round are shared by runs of the reduction (decided for the
 * nominal 148 SMs; the launch decides for the device); "none" for a shape the
 * NHWC form does not take.  For reports and tests; the choice is an
 * implementation detail.
 */
const char* im2win_nhwc_kernel_name(const im2win_shape* shape, const im2win_epilogue* epilogue);

/*
 * fp32 convolution without a scratch argument, for callers that cannot allocate
 * device memory (the paper has no counterpart; this is a convenience of this
 * library).  Think of code running where cudaMalloc is off limits: a real-time
 * loop with a frozen memory map, a plug-in that receives input and output
 * buffers but no allocator, a process whose device memory is managed by another
 * runtime.  Such a caller cannot produce the `scratch` buffer im2win_conv_f32
 * wants, so the library keeps one itself: a fixed array of
 * IM2WIN_STATIC_SCRATCH_BYTES that every GPU which loads the library holds until
 * the process exits.
 *
 * Same operation, arguments and results as im2win_conv_f32 (window, filter and
 * y are the caller's device buffers).  Differences:
 *   - A layer whose scratch_bytes (im2win_workspace_size, IM2WIN_F32) exceed
 *     IM2WIN_STATIC_SCRATCH_BYTES is rejected with IM2WIN_ERR_WORKSPACE_TOO_SMALL
 *     before anything is launched (roughly: Co*C*Kh*Kw above one million filter
 *     elements does not fit).
 *   - The call allocates nothing: no cudaMalloc, no cudaFree, no allocating
 *     library routine.
 *   - The first call on each device looks up the device address of the array
 *     (with that device current) and caches it; make that first call outside any
 *     stream capture.  The cached address belongs to the device's current
 *     context: it does not survive a cudaDeviceReset, after which this entry
 *     point must not be used again in the process.
 *   - All calls on a device share the one array, which keeps whatever the last
 *     call left in it.  Each call rewrites every byte it later reads, so
 *     back-to-back calls on one stream are safe; two calls whose kernels may
 *     overlap on the GPU (different streams, no ordering between them) race on
 *     the array and must be serialised by the caller.
 */
#define IM2WIN_STATIC_SCRATCH_BYTES (4u << 20)
im2win_status im2win_conv_f32_static(const float* window, const float* filter_oihw, float* y_nchw,
                                     const im2win_shape* shape, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* IM2WIN_H_ */
