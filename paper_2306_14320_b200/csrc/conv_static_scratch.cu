// im2win_conv_static: transform + convolution with the im2win tensor held in a buffer that is part
// of the library image, so that the call allocates nothing.
//
// Some callers cannot obtain device memory at the time they need a convolution: a process whose GPU
// memory has been handed over whole to another allocator (an inference server's arena, a framework
// pool sized to the device), or a loop that runs under a "no allocation after start-up" rule, as
// hard-real-time and safety-reviewed code does.  For them the scratch that im2win_conv takes from
// the caller (the im2win tensor) lives here, in a file-scope device array of fixed size.
#include <atomic>

#include "common.cuh"

namespace im2win {

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = IM2WIN_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address.  The
// address a kernel may use is asked for once per device (with that device current) and kept.
constexpr int kMaxDevices = 64;
std::atomic<float*> g_scratch_addr[kMaxDevices];  // (two first calls racing on a device both store the same address)

int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  float* addr = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!addr) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      return IM2WIN_ECUDA;
    }
    addr = static_cast<float*>(p);
    g_scratch_addr[dev].store(addr, std::memory_order_release);
  }
  *out = addr;
  return IM2WIN_OK;
}

}  // namespace

}  // namespace im2win

using namespace im2win;

extern "C" {

int im2win_conv_static(const float* in_nchw, const float* filter_kcfhfw, const im2win_shape* shape,
                       int mode, float* out_nchw, void* cuda_stream) {
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!in_nchw || !filter_kcfhfw || !out_nchw) return IM2WIN_EINVAL;
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16 && mode != IM2WIN_MODE_FP32) return IM2WIN_EINVAL;
  // the im2win tensor of this problem must fit the built-in buffer
  if ((uint64_t)g.n_win * sizeof(float) > (uint64_t)kStaticScratchBytes) return IM2WIN_ESCRATCH;
  const uintptr_t mask = reinterpret_cast<uintptr_t>(in_nchw) | reinterpret_cast<uintptr_t>(filter_kcfhfw) |
                         reinterpret_cast<uintptr_t>(out_nchw);
  if (mask & 15u) return IM2WIN_EALIGN;
  const uintptr_t o0 = reinterpret_cast<uintptr_t>(out_nchw), o1 = o0 + (uintptr_t)g.n_out * 4;
  const uintptr_t i0 = reinterpret_cast<uintptr_t>(in_nchw), i1 = i0 + (uintptr_t)g.n_in * 4;
  const uintptr_t f0 = reinterpret_cast<uintptr_t>(filter_kcfhfw), f1 = f0 + (uintptr_t)g.n_flt * 4;
  if ((o0 < i1 && i0 < o1) || (o0 < f1 && f0 < o1)) return IM2WIN_EOVERLAP;

  float* scratch = nullptr;
  rc = scratch_for_current_device(&scratch);  // first call on a device: looks the address up
  if (rc != IM2WIN_OK) return rc;
  // Nothing in the scratch has to start at zero: the transform writes every element of the im2win
  // tensor the convolution reads, and what lies behind that tensor is only ever used for a copy of
  // the filter that the same call writes first.  Whatever the previous call left behind is overwritten.
  return conv_impl(in_nchw, IM2WIN_SRC_NCHW, filter_kcfhfw, shape, mode, out_nchw, /*out16=*/false, scratch,
                   kStaticScratchBytes, cuda_stream);
}

}  // extern "C"
