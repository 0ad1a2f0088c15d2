// Algorithm 2 on the CUDA cores in plain fp32 (IM2WIN_MODE_FP32).
//
// One thread per output element, the r,u,v loops of Algorithm 2 inside it, fp32 FMA accumulation.
// This is the exact-arithmetic check mode of the library (it localises indexing mistakes without
// any tensor-core rounding in the way); it is not tuned and is not the path that is benchmarked.
#include "common.cuh"

namespace im2win {

namespace {

__global__ void __launch_bounds__(256) conv_fp32_kernel(const float* __restrict__ xhat,
                                                        const float* __restrict__ f,
                                                        float* __restrict__ out, Geometry g) {
  const int64_t total = g.n_out;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (int64_t)gridDim.x * blockDim.x) {
    // e = ((i*K + j)*Ho + m)*Wo + n
    const int32_t n = (int32_t)(e % g.Wo);
    int64_t t = e / g.Wo;
    const int32_t m = (int32_t)(t % g.Ho);
    t /= g.Ho;
    const int32_t j = (int32_t)(t % g.K);
    const int64_t i = t / g.K;
    const float* strip0 = xhat + ((i * g.C) * g.Ho + m) * (int64_t)g.L + (int64_t)n * g.sFh;
    const float* fj = f + (int64_t)j * g.Kg;
    float acc = 0.f;
    for (int32_t r = 0; r < g.C; ++r) {
      const float* win = strip0 + (int64_t)r * g.HoL;  // the window's Fh*Fw contiguous floats
      const float* fr = fj + (int64_t)r * g.FF;
      for (int32_t u = 0; u < g.Fh; ++u)
        for (int32_t v = 0; v < g.Fw; ++v)
          acc = fmaf(__ldg(win + v * g.Fh + u), __ldg(fr + u * g.Fw + v), acc);
    }
    if (g.out_nhwc) out[((i * g.Ho + m) * g.Wo + n) * (int64_t)g.K + j] = acc;
    else out[e] = acc;
  }
}

}  // namespace

int launch_conv_fp32(const float* xhat, const float* f, float* out, const Geometry& g, cudaStream_t st) {
  const int64_t blocks = (g.n_out + 255) / 256;
  const int grid = (int)(blocks < 148 * 32 ? blocks : 148 * 32);
  conv_fp32_kernel<<<grid, 256, 0, st>>>(xhat, f, out, g);
  note_kernel(KERNEL_FP32);
  return cuda_status(cudaGetLastError());
}

}  // namespace im2win
