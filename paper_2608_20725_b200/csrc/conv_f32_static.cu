// im2win_conv_f32_static: the fp32 convolution for callers that cannot allocate.
//
// Some callers may not call cudaMalloc at all: code that runs where device
// allocation is forbidden or must not happen (a real-time loop that has frozen
// its memory map, a plug-in that is handed input and output buffers but no
// allocator, a process whose memory pool belongs to another runtime).  The
// normal entry point asks such a caller for a scratch buffer it has no way to
// create.  This variant keeps the scratch (status block, offset table, repacked
// filter) in a fixed array inside the library instead.
//
// The array is a file-scope __device__ object: every GPU that loads the library
// holds IM2WIN_STATIC_SCRATCH_BYTES of it until the process exits.  In host code
// the array's name is only a stand-in, not a device address; the address the
// kernels need is fetched once per device with cudaGetSymbolAddress, with that
// device current, and cached.
#include <mutex>

#include "common.cuh"

namespace im2win {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[IM2WIN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the static scratch on the current device (set-up on first use).
cudaError_t static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace im2win

using namespace im2win;

extern "C" im2win_status im2win_conv_f32_static(const float* window, const float* filter_oihw, float* y_nchw,
                                                const im2win_shape* shape, void* cuda_stream) {
  if (!window || !filter_oihw || !y_nchw || !shape) return IM2WIN_ERR_NULL_POINTER;
  Geometry g;
  im2win_status st = derive_geometry(shape, &g);
  if (st != IM2WIN_OK) return st;
  ScratchLayout l;
  st = scratch_layout(g, IM2WIN_F32, &l);
  if (st != IM2WIN_OK) return st;
  if ((reinterpret_cast<uintptr_t>(window) | reinterpret_cast<uintptr_t>(filter_oihw) |
       reinterpret_cast<uintptr_t>(y_nchw)) & 15u)
    return IM2WIN_ERR_MISALIGNED;
  // The layer's scratch must fit the fixed array; nothing has touched CUDA yet.
  if (l.total > (size_t)IM2WIN_STATIC_SCRATCH_BYTES) return IM2WIN_ERR_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) return IM2WIN_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The pack kernel rewrites the status block, the whole offset table and the whole padded
  // filter, so nothing of the previous call's contents is read.
  if (launch_pack_f32(filter_oihw, scratch, g, l, stream) != cudaSuccess) return IM2WIN_ERR_CUDA;
  if (launch_conv_f32(window, y_nchw, scratch, g, l, stream) != cudaSuccess) return IM2WIN_ERR_CUDA;
  return IM2WIN_OK;
}
