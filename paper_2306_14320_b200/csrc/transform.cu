// im2win transformation (Algorithm 1):  Ihat[i][r][m][k*Fh+u] = I[i][r][m*s+u][k].
//
// Pure data movement, bound by HBM bandwidth.  Per (image, channel) plane the input rows needed by
// a block of output rows form ONE contiguous range of the input, and the strips they produce form
// ONE contiguous range of the output.  A CTA therefore
//   1. copies its input range into shared memory with 128-bit loads (the range keeps its 16-byte
//      phase in shared memory, so aligned global chunks land on aligned shared chunks),
//   2. walks its output range in 16-byte chunks, gathering each chunk's four elements from shared
//      memory (an Fh x W -> W x Fh transposition per strip) and writing one 128-bit store.
// Every needed input row is read from HBM once per row block (the Fh-s halo rows between
// neighbouring blocks come from L2), every output element is written exactly once.
#include "common.cuh"

namespace im2win {

namespace {

constexpr int kThreads = 256;

struct TransformParams {
  const float* in;
  float* out;
  int32_t H, W, Fh, s, Ho, L;
  int32_t MB;          // output rows per CTA
  int32_t nblk;        // row blocks per plane
  int64_t HW;          // input plane (floats)
  int64_t HoL;         // output plane (floats)
  uint64_t magic_L;    // ceil(2^32 / L)
  uint64_t magic_Fh;   // ceil(2^32 / Fh)
};

__device__ __forceinline__ float4 ldg_stream(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// One CTA: plane p = blockIdx.x / nblk, row block b = blockIdx.x % nblk.
__global__ void __launch_bounds__(kThreads) transform_smem_kernel(TransformParams P) {
  extern __shared__ __align__(16) float smem[];
  const int64_t job = blockIdx.x;
  const int64_t plane = job / P.nblk;
  const int32_t b = (int32_t)(job - plane * P.nblk);
  const int32_t m0 = b * P.MB;
  const int32_t mb = min(P.MB, P.Ho - m0);
  const int32_t rows_in = (mb - 1) * P.s + P.Fh;
  const int32_t n_in = rows_in * P.W;

  // ---- stage the input range, keeping its 16-byte phase
  const float* src = P.in + plane * P.HW + (int64_t)m0 * P.s * P.W;
  const int32_t skew = (int32_t)((reinterpret_cast<uintptr_t>(src) >> 2) & 3);
  float* tile = smem + skew;  // tile[e] <-> src[e]
  {
    const int32_t head = min((4 - skew) & 3, n_in);
    const int32_t nvec = (n_in - head) >> 2;
    const int32_t tail0 = head + (nvec << 2);
    if ((int32_t)threadIdx.x < head) tile[threadIdx.x] = __ldg(src + threadIdx.x);
    const float4* src4 = reinterpret_cast<const float4*>(src + head);
    float4* dst4 = reinterpret_cast<float4*>(tile + head);
    for (int32_t i = threadIdx.x; i < nvec; i += kThreads) dst4[i] = ldg_stream(src4 + i);
    if ((int32_t)threadIdx.x < n_in - tail0) tile[tail0 + threadIdx.x] = __ldg(src + tail0 + threadIdx.x);
  }
  __syncthreads();

  // ---- emit the output range
  float* dst = P.out + plane * P.HoL + (int64_t)m0 * P.L;
  const int32_t n_out = mb * P.L;
  const int32_t dskew = (int32_t)((reinterpret_cast<uintptr_t>(dst) >> 2) & 3);
  const int32_t head = min((4 - dskew) & 3, n_out);
  const int32_t nvec = (n_out - head) >> 2;
  const int32_t tail0 = head + (nvec << 2);

  // element e of the output range -> shared-memory index of its source
  auto locate = [&](int32_t e, int32_t& mm, int32_t& k, int32_t& u) {
    mm = (int32_t)(((uint64_t)(uint32_t)e * P.magic_L) >> 32);
    const int32_t rem = e - mm * P.L;
    k = (int32_t)(((uint64_t)(uint32_t)rem * P.magic_Fh) >> 32);
    u = rem - k * P.Fh;
  };
  auto fetch = [&](int32_t mm, int32_t k, int32_t u) { return tile[(mm * P.s + u) * P.W + k]; };
  auto advance = [&](int32_t& mm, int32_t& k, int32_t& u) {
    if (++u == P.Fh) { u = 0; if (++k == P.W) { k = 0; ++mm; } }
  };

  if ((int32_t)threadIdx.x < head) {
    int32_t mm, k, u;
    locate(threadIdx.x, mm, k, u);
    dst[threadIdx.x] = fetch(mm, k, u);
  }
  float4* dst4 = reinterpret_cast<float4*>(dst + head);
  for (int32_t i = threadIdx.x; i < nvec; i += kThreads) {
    int32_t mm, k, u;
    locate(head + (i << 2), mm, k, u);
    float4 v;
    v.x = fetch(mm, k, u); advance(mm, k, u);
    v.y = fetch(mm, k, u); advance(mm, k, u);
    v.z = fetch(mm, k, u); advance(mm, k, u);
    v.w = fetch(mm, k, u);
    dst4[i] = v;
  }
  if ((int32_t)threadIdx.x < n_out - tail0) {
    int32_t mm, k, u;
    locate(tail0 + threadIdx.x, mm, k, u);
    dst[tail0 + threadIdx.x] = fetch(mm, k, u);
  }
}

// Fallback for rows too long to stage (Fh*W floats beyond the shared-memory budget): one thread
// per output element, reads through L1/L2.  Correct for every shape, not tuned.
__global__ void __launch_bounds__(kThreads) transform_gather_kernel(const float* __restrict__ in,
                                                                     float* __restrict__ out,
                                                                     int32_t H, int32_t W, int32_t Fh,
                                                                     int32_t s, int32_t Ho, int64_t total) {
  const int64_t L = (int64_t)W * Fh;
  for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < total;
       e += (int64_t)gridDim.x * kThreads) {
    const int64_t strip = e / L;
    const int32_t rem = (int32_t)(e - strip * L);
    const int32_t k = rem / Fh, u = rem - k * Fh;
    const int64_t plane = strip / Ho;
    const int32_t m = (int32_t)(strip - plane * Ho);
    out[e] = __ldg(in + (plane * H + (int64_t)m * s + u) * W + k);
  }
}

uint64_t magic_for(uint32_t d) { return ((uint64_t)1 << 32) / d + ((((uint64_t)1 << 32) % d) ? 1 : 0); }

}  // namespace

int launch_transform(const float* in, float* out, const Geometry& g, cudaStream_t st) {
  // Shared-memory budget for the staged input rows.  Small enough for several CTAs per SM so that
  // one CTA's loads overlap another's stores.
  constexpr int32_t kTileFloats = 8192 - 4;      // 32 KB including the phase skew
  constexpr int32_t kTileFloatsMax = 49152 - 4;  // opt-in ceiling for very wide rows
  const int64_t planes = (int64_t)g.N * g.C;
  const int64_t row_floats = (int64_t)g.Fh * g.W;

  if (row_floats > kTileFloatsMax) {
    const int64_t blocks = (g.n_win + kThreads - 1) / kThreads;
    const int grid = (int)(blocks < 148 * 64 ? blocks : 148 * 64);
    transform_gather_kernel<<<grid, kThreads, 0, st>>>(in, out, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
    return cuda_status(cudaGetLastError());
  }
  const int32_t budget = row_floats > kTileFloats ? kTileFloatsMax : kTileFloats;
  int32_t rows_fit = budget / g.W;                       // input rows that fit
  int32_t MB = (rows_fit - g.Fh) / g.s + 1;              // output rows those feed
  if (MB < 1) MB = 1;
  if (MB > g.Ho) MB = g.Ho;
  const int32_t nblk = (g.Ho + MB - 1) / MB;
  MB = (g.Ho + nblk - 1) / nblk;                         // balance the blocks
  const int32_t rows_in = (MB - 1) * g.s + g.Fh;
  const size_t smem = ((size_t)rows_in * g.W + 4) * sizeof(float);
  // magic-number division is exact while (range length) * divisor < 2^32
  if ((int64_t)MB * g.L * g.L >= ((int64_t)1 << 32) || planes * nblk > INT32_MAX) {
    const int64_t blocks = (g.n_win + kThreads - 1) / kThreads;
    const int grid = (int)(blocks < 148 * 64 ? blocks : 148 * 64);
    transform_gather_kernel<<<grid, kThreads, 0, st>>>(in, out, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
    return cuda_status(cudaGetLastError());
  }
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(transform_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return IM2WIN_ECUDA;
  }
  TransformParams P;
  P.in = in; P.out = out;
  P.H = g.H; P.W = g.W; P.Fh = g.Fh; P.s = g.s; P.Ho = g.Ho; P.L = g.L;
  P.MB = MB; P.nblk = nblk;
  P.HW = (int64_t)g.H * g.W; P.HoL = g.HoL;
  P.magic_L = magic_for((uint32_t)g.L);
  P.magic_Fh = magic_for((uint32_t)g.Fh);
  transform_smem_kernel<<<(unsigned)(planes * nblk), kThreads, smem, st>>>(P);
  return cuda_status(cudaGetLastError());
}

}  // namespace im2win
