// C ABI of the im2win library: argument validation, buffer-size queries and
// dispatch to the kernels.  Declarations and the contract of every entry
// point are in include/im2win.h.
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "common.cuh"

namespace im2win {

static inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

const char* debug_getenv(const char* name) {
  static const bool enabled = getenv("IM2WIN_DEBUG") != nullptr;   // looked up once per process
  return enabled ? getenv(name) : nullptr;
}

im2win_status derive_geometry(const im2win_shape* s, Geometry* g) {
  if (!s) return IM2WIN_ERR_NULL_POINTER;
  if (s->N < 1 || s->C < 1 || s->H < 1 || s->W < 1 || s->Co < 1 || s->Kh < 1 || s->Kw < 1 ||
      s->stride < 1 || s->pad < 0)
    return IM2WIN_ERR_INVALID_ARG;
  const int64_t hspan = (int64_t)s->H + 2 * (int64_t)s->pad - s->Kh;
  const int64_t wspan = (int64_t)s->W + 2 * (int64_t)s->pad - s->Kw;
  if (hspan < 0 || wspan < 0) return IM2WIN_ERR_INVALID_ARG;
  g->N = s->N; g->C = s->C; g->H = s->H; g->W = s->W; g->Co = s->Co;
  g->Kh = s->Kh; g->Kw = s->Kw; g->s = s->stride; g->p = s->pad;
  g->Ho = (int32_t)(hspan / s->stride) + 1;
  g->Wo = (int32_t)(wspan / s->stride) + 1;
  const int64_t Wp = (int64_t)s->W + 2 * (int64_t)s->pad;
  const int64_t T = (int64_t)s->Kh * s->Kw;
  // Index ranges of the kernels: 32-bit per-image offsets and counts, 64-bit bases.
  const int64_t lim = (int64_t)1 << 31;
  if (Wp >= lim || T >= lim) return IM2WIN_ERR_UNSUPPORTED;
  g->Wp = (int32_t)Wp;
  g->T = (int32_t)T;
  g->strip = (int64_t)s->Kh * Wp;
  if (g->strip >= lim) return IM2WIN_ERR_UNSUPPORTED;
  g->chan_stride = (int64_t)g->Ho * g->strip;
  if (g->chan_stride >= lim) return IM2WIN_ERR_UNSUPPORTED;
  g->img_stride = (int64_t)s->C * g->chan_stride;
  if (g->img_stride >= lim) return IM2WIN_ERR_UNSUPPORTED;    // k -> offset table is int32
  g->K = (int64_t)s->C * T;
  if (g->K >= lim - 64) return IM2WIN_ERR_UNSUPPORTED;
  if ((int64_t)g->Ho * g->Wo >= lim) return IM2WIN_ERR_UNSUPPORTED;
  g->P = (int64_t)s->N * g->Ho * g->Wo;
  if (g->P >= lim * 64) return IM2WIN_ERR_UNSUPPORTED;        // grid.x of 128-row tiles
  if ((int64_t)s->N * s->C * g->Ho * Wp >= lim * 4) return IM2WIN_ERR_UNSUPPORTED;      // transform grid
  if ((int64_t)s->H * s->W >= lim) return IM2WIN_ERR_UNSUPPORTED;
  if ((int64_t)s->Kh * 8 * 4 > 200 * 1024) return IM2WIN_ERR_UNSUPPORTED;  // transform staging
  if ((int64_t)s->Co * g->K >= lim * 16) return IM2WIN_ERR_UNSUPPORTED;
  g->window_elems = (int64_t)s->N * g->img_stride;
  g->out_elems = (int64_t)s->N * s->Co * g->Ho * g->Wo;
  return IM2WIN_OK;
}

im2win_status scratch_layout(const Geometry& g, im2win_dtype dtype, ScratchLayout* l) {
  if (dtype == IM2WIN_F32) {
    l->Kp = round_up(g.K, plan_f32(g).bk);
    l->Co_pad = round_up(g.Co, plan_f32(g).bn);
  } else if (dtype == IM2WIN_F16) {
    l->Kp = round_up(g.K, kF16KBlock);
    l->Co_pad = g.Co;
  } else {
    return IM2WIN_ERR_INVALID_ARG;
  }
  l->f16_shift = false;
  l->f16_raw = false;
  l->f16_mat = false;
  l->f16_stem = false;
  l->koff_off = kStatusBytes;
  l->filter_off = (size_t)round_up((int64_t)l->koff_off + 4 * l->Kp, 256);
  int64_t fbytes = l->Kp * l->Co_pad * (dtype == IM2WIN_F32 ? 4 : 2);
  l->total = (size_t)round_up((int64_t)l->filter_off + fbytes, 256);
  if (dtype == IM2WIN_F16) {
    // The shifted-view kernel is used whenever the layer is eligible; IM2WIN_F16_KERNEL=gather
    // forces the general gather kernel (a testing aid).  The scratch size covers both layouts.
    const ShiftPlan plan = plan_f16_shift(g);
    const bool stem_ok = plan_f16_stem(g).eligible;       // shares the filter layout of the shifted-view kernel
    if (plan.eligible || stem_ok) {
      const int64_t K2p = round_up((int64_t)g.C * g.Kh, kF16KBlock);
      const size_t shift_filter_off = (size_t)round_up((int64_t)kStatusBytes + 4 * K2p, 256);
      const size_t shift_total = (size_t)round_up((int64_t)shift_filter_off + K2p * g.Co * g.Kw * 2, 256);
      const char* force = debug_getenv("IM2WIN_F16_KERNEL");
      const bool use_shift = !(force && strcmp(force, "gather") == 0);
      if (use_shift) {
        l->f16_shift = plan.eligible;
        l->Kp = K2p;
        l->filter_off = shift_filter_off;
        // the bulk-copy variant shares the filter layout; IM2WIN_F16_KERNEL=shift keeps the gathering one
        l->f16_raw = plan.eligible && plan_f16_raw(g).eligible && !(force && strcmp(force, "shift") == 0);
        // layers with one k-block: their own kernel unless another one is forced
        l->f16_stem = stem_ok && (!force || strcmp(force, "stem") == 0);
      }
      if (shift_total > l->total) l->total = shift_total;
    }
    const MatPlan mat = plan_f16_mat(g);
    const char* force = debug_getenv("IM2WIN_F16_KERNEL");
    // measured: the matrix-transpose kernel wins for strided layers (the others stage such layers
    // with 2-byte gathers) and for kernels up to 5 wide with 128 output channels or more (CTA pairs
    // above 128); IM2WIN_F16_KERNEL=mat forces it wherever it can run (a testing aid)
    const bool want = force ? strcmp(force, "mat") == 0 : (g.s > 1 || (g.Co >= 128 && g.Kw <= 5));
    // (the scratch size covers every layout, whichever kernel is picked or forced)
    if (mat.eligible) {
      l->f16_mat = want && !l->f16_stem;
      const size_t mat_total = (size_t)round_up((int64_t)mat.scratch_bytes, 256);
      if (mat_total > l->total) l->total = mat_total;
    }
  }
  return IM2WIN_OK;
}

static inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// mode bit 0: pack the filter into scratch; bit 1: run the convolution on the packed filter.
enum { kDoPack = 1, kDoConv = 2 };
static im2win_status conv_common(const void* window, const void* filter, float* y, void* scratch,
                                 size_t scratch_bytes, const im2win_shape* shape, im2win_dtype dtype,
                                 void* cuda_stream, int mode = kDoPack | kDoConv) {
  if (!scratch || !shape) return IM2WIN_ERR_NULL_POINTER;
  if ((mode & kDoPack) && !filter) return IM2WIN_ERR_NULL_POINTER;
  if ((mode & kDoConv) && (!window || !y)) return IM2WIN_ERR_NULL_POINTER;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  ScratchLayout l;
  st = scratch_layout(g, dtype, &l);
  if (st != IM2WIN_OK) return st;
  if (misaligned(scratch) || ((mode & kDoPack) && misaligned(filter)) ||
      ((mode & kDoConv) && (misaligned(window) || misaligned(y))))
    return IM2WIN_ERR_MISALIGNED;
  if (scratch_bytes < l.total) return IM2WIN_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaSuccess;
  if (mode & kDoPack) {
    if (dtype == IM2WIN_F32) e = launch_pack_f32(static_cast<const float*>(filter), scratch, g, l, stream);
    else if (l.f16_stem) e = launch_pack_f16_shift(static_cast<const uint16_t*>(filter), scratch, g, l, stream);
    else if (l.f16_mat) e = launch_pack_f16_mat(static_cast<const uint16_t*>(filter), scratch, g, stream);
    else if (l.f16_raw)
      e = launch_pack_f16_raw(static_cast<const uint16_t*>(filter), scratch, g, l, plan_f16_raw(g), stream);
    else if (l.f16_shift) e = launch_pack_f16_shift(static_cast<const uint16_t*>(filter), scratch, g, l, stream);
    else e = launch_pack_f16(static_cast<const uint16_t*>(filter), scratch, g, l, stream);
    if (e != cudaSuccess) return IM2WIN_ERR_CUDA;
  }
  if (mode & kDoConv) {
    if (dtype == IM2WIN_F32) e = launch_conv_f32(static_cast<const float*>(window), y, scratch, g, l, stream);
    else if (l.f16_stem) e = launch_conv_f16_stem(static_cast<const uint16_t*>(window), y, scratch, g, l, stream);
    else if (l.f16_mat) e = launch_conv_f16_mat(static_cast<const uint16_t*>(window), y, scratch, g, stream);
    else if (l.f16_raw) e = launch_conv_f16_raw(static_cast<const uint16_t*>(window), y, scratch, g, l, stream);
    else if (l.f16_shift) e = launch_conv_f16_shift(static_cast<const uint16_t*>(window), y, scratch, g, l, stream);
    else e = launch_conv_f16_gather(static_cast<const uint16_t*>(window), y, scratch, g, l, stream);
  }
  return e == cudaSuccess ? IM2WIN_OK : IM2WIN_ERR_CUDA;
}

}  // namespace im2win

using namespace im2win;

extern "C" {

const char* im2win_status_string(im2win_status status) {
  switch (status) {
    case IM2WIN_OK: return "ok";
    case IM2WIN_ERR_INVALID_ARG: return "invalid argument";
    case IM2WIN_ERR_NULL_POINTER: return "null pointer";
    case IM2WIN_ERR_MISALIGNED: return "device pointer not 16-byte aligned";
    case IM2WIN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case IM2WIN_ERR_UNSUPPORTED: return "shape beyond the kernels' index ranges";
    case IM2WIN_ERR_CUDA: return "CUDA error";
    case IM2WIN_ERR_TIMEOUT: return "bounded device wait gave up";
  }
  return "unknown status";
}

const char* im2win_conv_kernel_name(const im2win_shape* shape, im2win_dtype dtype) {
  Geometry g;
  ScratchLayout l;
  if (derive_geometry(shape, &g) != IM2WIN_OK || scratch_layout(g, dtype, &l) != IM2WIN_OK) return "none";
  if (dtype == IM2WIN_F32) return "f32-ffma";
  if (l.f16_stem) return "f16-stem";
  if (l.f16_mat) return "f16-mat";
  if (l.f16_raw) return "f16-raw";
  if (l.f16_shift) return "f16-shift";
  return "f16-gather";
}

im2win_status im2win_workspace_size(const im2win_shape* shape, im2win_dtype dtype, size_t* window_bytes,
                                    size_t* scratch_bytes, int32_t* Ho, int32_t* Wo) {
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  ScratchLayout l;
  st = scratch_layout(g, dtype, &l);
  if (st != IM2WIN_OK) return st;
  if (window_bytes) *window_bytes = (size_t)g.window_elems * (dtype == IM2WIN_F32 ? 4 : 2);
  if (scratch_bytes) *scratch_bytes = l.total;
  if (Ho) *Ho = g.Ho;
  if (Wo) *Wo = g.Wo;
  return IM2WIN_OK;
}

im2win_status im2win_transform(const void* x_nchw, void* window, const im2win_shape* shape,
                               im2win_dtype dtype, void* cuda_stream) {
  if (!x_nchw || !window || !shape) return IM2WIN_ERR_NULL_POINTER;
  if (dtype != IM2WIN_F32 && dtype != IM2WIN_F16) return IM2WIN_ERR_INVALID_ARG;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  if (misaligned(x_nchw) || misaligned(window)) return IM2WIN_ERR_MISALIGNED;
  cudaError_t e = launch_transform(x_nchw, window, g, dtype == IM2WIN_F32 ? 4 : 2,
                                   static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? IM2WIN_OK : IM2WIN_ERR_CUDA;
}

im2win_status im2win_conv_f32(const float* window, const float* filter_oihw, float* y_nchw, void* scratch,
                              size_t scratch_bytes, const im2win_shape* shape, void* cuda_stream) {
  return conv_common(window, filter_oihw, y_nchw, scratch, scratch_bytes, shape, IM2WIN_F32, cuda_stream);
}

im2win_status im2win_conv_f16(const uint16_t* window, const uint16_t* filter_oihw, float* y_nchw,
                              void* scratch, size_t scratch_bytes, const im2win_shape* shape,
                              void* cuda_stream) {
  return conv_common(window, filter_oihw, y_nchw, scratch, scratch_bytes, shape, IM2WIN_F16, cuda_stream);
}

im2win_status im2win_pack_filter(const void* filter_oihw, void* scratch, size_t scratch_bytes,
                                 const im2win_shape* shape, im2win_dtype dtype, void* cuda_stream) {
  return conv_common(nullptr, filter_oihw, nullptr, scratch, scratch_bytes, shape, dtype, cuda_stream, kDoPack);
}

im2win_status im2win_conv_packed(const void* window, float* y_nchw, void* scratch, size_t scratch_bytes,
                                 const im2win_shape* shape, im2win_dtype dtype, void* cuda_stream) {
  return conv_common(window, nullptr, y_nchw, scratch, scratch_bytes, shape, dtype, cuda_stream, kDoConv);
}

// ---- channel-innermost (NHWC) form ------------------------------------------------------------
static im2win_status epilogue_args(const im2win_epilogue* e, bool nhwc_allowed, EpilogueArgs* out) {
  out->bias = nullptr; out->relu = 0; out->out16 = 0; out->y_nhwc = 0;
  if (!e) return IM2WIN_OK;
  if ((e->relu != 0 && e->relu != 1) || (e->out_dtype != IM2WIN_F32 && e->out_dtype != IM2WIN_F16) ||
      (e->out_layout != IM2WIN_LAYOUT_NCHW && e->out_layout != IM2WIN_LAYOUT_NHWC))
    return IM2WIN_ERR_INVALID_ARG;
  if (e->out_layout == IM2WIN_LAYOUT_NHWC && !nhwc_allowed) return IM2WIN_ERR_UNSUPPORTED;
  if (e->bias && (reinterpret_cast<uintptr_t>(e->bias) & 15u)) return IM2WIN_ERR_MISALIGNED;
  out->bias = e->bias; out->relu = e->relu; out->out16 = e->out_dtype == IM2WIN_F16;
  out->y_nhwc = e->out_layout == IM2WIN_LAYOUT_NHWC;
  return IM2WIN_OK;
}

static im2win_status nhwc_common(const uint16_t* window, const uint16_t* filter, void* y, const im2win_epilogue* epilogue,
                                 void* scratch, size_t scratch_bytes, const im2win_shape* shape, void* cuda_stream,
                                 int mode) {
  if (!scratch || !shape) return IM2WIN_ERR_NULL_POINTER;
  if ((mode & kDoPack) && !filter) return IM2WIN_ERR_NULL_POINTER;
  if ((mode & kDoConv) && (!window || !y)) return IM2WIN_ERR_NULL_POINTER;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return IM2WIN_ERR_UNSUPPORTED;
  EpilogueArgs epi;
  st = epilogue_args(epilogue, true, &epi);
  if (st != IM2WIN_OK) return st;
  if (misaligned(scratch) || ((mode & kDoPack) && misaligned(filter)) ||
      ((mode & kDoConv) && (misaligned(window) || misaligned(y))))
    return IM2WIN_ERR_MISALIGNED;
  if (scratch_bytes < plan.scratch_bytes) return IM2WIN_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if ((mode & kDoPack) && launch_pack_f16_nhwc(filter, scratch, g, stream) != cudaSuccess) return IM2WIN_ERR_CUDA;
  if ((mode & kDoConv) && launch_conv_f16_nhwc(window, y, scratch, g, epi, stream) != cudaSuccess) return IM2WIN_ERR_CUDA;
  return IM2WIN_OK;
}

const char* im2win_nhwc_kernel_name(const im2win_shape* shape, const im2win_epilogue* epilogue) {
  Geometry g;
  EpilogueArgs epi;
  if (!shape || derive_geometry(shape, &g) != IM2WIN_OK || epilogue_args(epilogue, true, &epi) != IM2WIN_OK) return "none";
  return nhwc_kernel_name(g, epi);
}

im2win_status im2win_nhwc_workspace_size(const im2win_shape* shape, size_t* window_bytes, size_t* scratch_bytes,
                                         int32_t* Ho, int32_t* Wo, int32_t* Cp) {
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  const NhwcPlan plan = plan_nhwc(g);
  if (!plan.eligible) return IM2WIN_ERR_UNSUPPORTED;
  if (window_bytes) *window_bytes = (size_t)plan.window_elems * 2;
  if (scratch_bytes) *scratch_bytes = plan.scratch_bytes;
  if (Ho) *Ho = g.Ho;
  if (Wo) *Wo = g.Wo;
  if (Cp) *Cp = plan.Cp;
  return IM2WIN_OK;
}

im2win_status im2win_transform_nhwc(const uint16_t* x, im2win_layout x_layout, uint16_t* window,
                                    const im2win_shape* shape, void* cuda_stream) {
  if (!x || !window || !shape) return IM2WIN_ERR_NULL_POINTER;
  if (x_layout != IM2WIN_LAYOUT_NCHW && x_layout != IM2WIN_LAYOUT_NHWC) return IM2WIN_ERR_INVALID_ARG;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  if (!plan_nhwc(g).eligible) return IM2WIN_ERR_UNSUPPORTED;
  if (misaligned(x) || misaligned(window)) return IM2WIN_ERR_MISALIGNED;
  cudaError_t e = launch_transform_nhwc(x, x_layout == IM2WIN_LAYOUT_NHWC, window, g, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? IM2WIN_OK : IM2WIN_ERR_CUDA;
}

im2win_status im2win_conv_f16_nhwc(const uint16_t* window, const uint16_t* filter_oihw, void* y,
                                   const im2win_epilogue* epilogue, void* scratch, size_t scratch_bytes,
                                   const im2win_shape* shape, void* cuda_stream) {
  return nhwc_common(window, filter_oihw, y, epilogue, scratch, scratch_bytes, shape, cuda_stream, kDoPack | kDoConv);
}

im2win_status im2win_pack_filter_nhwc(const uint16_t* filter_oihw, void* scratch, size_t scratch_bytes,
                                      const im2win_shape* shape, void* cuda_stream) {
  return nhwc_common(nullptr, filter_oihw, nullptr, nullptr, scratch, scratch_bytes, shape, cuda_stream, kDoPack);
}

im2win_status im2win_conv_packed_nhwc(const uint16_t* window, void* y, const im2win_epilogue* epilogue,
                                      void* scratch, size_t scratch_bytes, const im2win_shape* shape,
                                      void* cuda_stream) {
  return nhwc_common(window, nullptr, y, epilogue, scratch, scratch_bytes, shape, cuda_stream, kDoConv);
}

im2win_status im2win_check_status(const void* scratch, void* cuda_stream) {
  if (!scratch) return IM2WIN_ERR_NULL_POINTER;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return IM2WIN_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return IM2WIN_ERR_CUDA;
  return word ? IM2WIN_ERR_TIMEOUT : IM2WIN_OK;
}

namespace {
// Two auxiliary streams per device for the chunked host-to-host path (created on first use and kept
// for the life of the process; the only state the library keeps besides the static scratch array).
struct AuxStreams {
  cudaStream_t in, out;
};
bool get_aux_streams(AuxStreams* a) {
  static std::mutex mu;
  static AuxStreams cache[64];
  static bool have[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (!have[dev]) {
    if (cudaStreamCreateWithFlags(&cache[dev].in, cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaStreamCreateWithFlags(&cache[dev].out, cudaStreamNonBlocking) != cudaSuccess) {
      cudaStreamDestroy(cache[dev].in);
      return false;
    }
    have[dev] = true;
  }
  *a = cache[dev];
  return true;
}

struct LayerLayout {
  size_t x_off, f_off, win_off, scratch_off, y_off, total;
  size_t x_bytes, f_bytes, win_bytes, scratch_bytes, y_bytes;
};
im2win_status layer_layout(const Geometry& g, im2win_dtype dtype, LayerLayout* L) {
  ScratchLayout l;
  im2win_status st = scratch_layout(g, dtype, &l);
  if (st != IM2WIN_OK) return st;
  const size_t es = dtype == IM2WIN_F32 ? 4 : 2;
  L->x_bytes = (size_t)g.N * g.C * g.H * g.W * es;
  L->f_bytes = (size_t)g.Co * g.K * es;
  L->win_bytes = (size_t)g.window_elems * es;
  L->scratch_bytes = l.total;
  L->y_bytes = (size_t)g.out_elems * 4;
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  L->x_off = 0;
  L->f_off = L->x_off + up(L->x_bytes);
  L->win_off = L->f_off + up(L->f_bytes);
  L->scratch_off = L->win_off + up(L->win_bytes);
  L->y_off = L->scratch_off + up(L->scratch_bytes);
  L->total = L->y_off + up(L->y_bytes);
  return IM2WIN_OK;
}
}  // namespace

im2win_status im2win_layer_workspace_size(const im2win_shape* shape, im2win_dtype dtype, size_t* device_bytes) {
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  LayerLayout L;
  st = layer_layout(g, dtype, &L);
  if (st != IM2WIN_OK) return st;
  if (device_bytes) *device_bytes = L.total;
  return IM2WIN_OK;
}

im2win_status im2win_layer_forward_host(const void* x_host, const void* filter_host, float* y_host,
                                        void* device_workspace, size_t device_workspace_bytes,
                                        const im2win_shape* shape, im2win_dtype dtype, void* cuda_stream) {
  if (!x_host || !filter_host || !y_host || !device_workspace || !shape) return IM2WIN_ERR_NULL_POINTER;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  LayerLayout L;
  st = layer_layout(g, dtype, &L);
  if (st != IM2WIN_OK) return st;
  if ((reinterpret_cast<uintptr_t>(device_workspace) & 255u) != 0) return IM2WIN_ERR_MISALIGNED;
  if (device_workspace_bytes < L.total) return IM2WIN_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(device_workspace);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t es = dtype == IM2WIN_F32 ? 4 : 2;

  // Large layers are cut into batch chunks so that the upload of chunk i+1, the kernels of chunk
  // i and the download of chunk i-1 overlap (the two copy directions run concurrently on the
  // link).  Chunks start at images whose slices of x, window and y are 16-byte aligned.
  const size_t x_img = (size_t)g.C * g.H * g.W * es, w_img = (size_t)g.img_stride * es,
               y_img = (size_t)g.Co * g.Ho * g.Wo * 4;
  int unit = 1;                                   // images per alignment unit
  while (unit <= 8 && ((unit * x_img) % 16 || (unit * w_img) % 16 || (unit * y_img) % 16)) unit *= 2;
  int nchunk = 1;
  AuxStreams aux{};
  if (unit <= 8 && g.N >= 4 * unit && L.x_bytes + L.y_bytes >= ((size_t)8 << 20) && get_aux_streams(&aux)) nchunk = 4;
  if (nchunk == 1) {
    if (cudaMemcpyAsync(ws + L.x_off, x_host, L.x_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return IM2WIN_ERR_CUDA;
    if (cudaMemcpyAsync(ws + L.f_off, filter_host, L.f_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return IM2WIN_ERR_CUDA;
    st = im2win_transform(ws + L.x_off, ws + L.win_off, shape, dtype, cuda_stream);
    if (st != IM2WIN_OK) return st;
    st = conv_common(ws + L.win_off, ws + L.f_off, reinterpret_cast<float*>(ws + L.y_off), ws + L.scratch_off,
                     L.scratch_bytes, shape, dtype, cuda_stream);
    if (st != IM2WIN_OK) return st;
    if (cudaMemcpyAsync(y_host, ws + L.y_off, L.y_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
      return IM2WIN_ERR_CUDA;
    return IM2WIN_OK;
  }

  // Everything the auxiliary streams do is ordered after the work already queued on `stream`, and
  // `stream` ends up waiting for the last download, so the caller still only synchronises `stream`.
  cudaEvent_t ev;
  auto fence = [&](cudaStream_t from, cudaStream_t to) -> bool {      // `to` waits for what `from` has queued
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return false;
    const bool ok = cudaEventRecord(ev, from) == cudaSuccess && cudaStreamWaitEvent(to, ev, 0) == cudaSuccess;
    cudaEventDestroy(ev);                                              // released once it has completed
    return ok;
  };
  const int per = ((g.N + nchunk - 1) / nchunk + unit - 1) / unit * unit;
  // Every distinct chunk size is validated before anything is queued: its geometry must derive and
  // the scratch its kernels want (the kernel choice can depend on N) must fit the scratch that was
  // sized for the whole batch.
  for (int n0 = 0; n0 < g.N; n0 += per) {
    im2win_shape part = *shape;
    part.N = n0 + per < g.N ? per : g.N - n0;
    Geometry gp;
    ScratchLayout lp;
    st = derive_geometry(&part, &gp);
    if (st == IM2WIN_OK) st = scratch_layout(gp, dtype, &lp);
    if (st != IM2WIN_OK) return st;
    if (lp.total > L.scratch_bytes) return IM2WIN_ERR_WORKSPACE_TOO_SMALL;
  }
  if (!fence(stream, aux.in) || !fence(stream, aux.out)) return IM2WIN_ERR_CUDA;
  // From here on work is queued on the auxiliary streams: on any failure `stream` is still made to
  // wait for both of them, so that synchronising `stream` completes whatever was queued.
  im2win_status result = IM2WIN_OK;
  if (cudaMemcpyAsync(ws + L.f_off, filter_host, L.f_bytes, cudaMemcpyHostToDevice, aux.in) != cudaSuccess)
    result = IM2WIN_ERR_CUDA;
  for (int n0 = 0; n0 < g.N && result == IM2WIN_OK; n0 += per) {
    const int n1 = n0 + per < g.N ? n0 + per : g.N;
    im2win_shape part = *shape;
    part.N = n1 - n0;
    unsigned char* xd = ws + L.x_off + (size_t)n0 * x_img;
    unsigned char* wd = ws + L.win_off + (size_t)n0 * w_img;
    unsigned char* yd = ws + L.y_off + (size_t)n0 * y_img;
    if (cudaMemcpyAsync(xd, static_cast<const unsigned char*>(x_host) + (size_t)n0 * x_img, (size_t)part.N * x_img,
                        cudaMemcpyHostToDevice, aux.in) != cudaSuccess || !fence(aux.in, stream)) {
      result = IM2WIN_ERR_CUDA;
      break;
    }
    result = im2win_transform(xd, wd, &part, dtype, cuda_stream);
    if (result != IM2WIN_OK) break;
    result = conv_common(wd, ws + L.f_off, reinterpret_cast<float*>(yd), ws + L.scratch_off, L.scratch_bytes, &part,
                         dtype, cuda_stream);
    if (result != IM2WIN_OK) break;
    if (!fence(stream, aux.out) ||
        cudaMemcpyAsync(reinterpret_cast<unsigned char*>(y_host) + (size_t)n0 * y_img, yd, (size_t)part.N * y_img,
                        cudaMemcpyDeviceToHost, aux.out) != cudaSuccess)
      result = IM2WIN_ERR_CUDA;
  }
  const bool joined = fence(aux.out, stream) & fence(aux.in, stream);
  if (result == IM2WIN_OK && !joined) result = IM2WIN_ERR_CUDA;
  return result;
}

}  // extern "C"
