// im2win_conv_static: transform + convolution with the im2win tensor held in a buffer that is part
// of the library image, so that the call allocates nothing.
//
// Some callers cannot obtain device memory at the time they need a convolution: a process whose GPU
// memory has been handed over whole to another allocator (an inference server's arena, a framework
// pool sized to the device), or a loop that runs under a "no allocation after start-up" rule, as
// hard-real-time and safety-reviewed code does.  For them the scratch that im2win_conv takes from
// the caller (the im2win tensor) lives here, in a file-scope device array of fixed size.
#include "common.cuh"

namespace im2win {

namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = IM2WIN_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address.  The
// address a kernel may use is asked for once per device (with that device current) and kept.
constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices] = {};

int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      return IM2WIN_ECUDA;
    }
    g_scratch_addr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_addr[dev];
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
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // Nothing in the scratch has to start at zero: the transform writes every element the
  // convolution reads, so whatever the previous call left behind is overwritten first.
  rc = launch_transform(in_nchw, scratch, g, st);
  if (rc != IM2WIN_OK) return rc;
  if (mode == IM2WIN_MODE_FP32) return launch_conv_fp32(scratch, filter_kcfhfw, out_nchw, g, st);
  return launch_conv_tc(scratch, filter_kcfhfw, out_nchw, g, mode, st, /*may_alloc=*/false);
}

}  // extern "C"
