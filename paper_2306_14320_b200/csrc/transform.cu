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
  int32_t MB;          // output rows per CTA (row-block mode)
  int32_t nblk;        // row blocks per plane (1: whole planes per CTA)
  int32_t PB;          // planes per CTA (> 1 only with nblk == 1)
  int64_t planes;      // N*C
  int64_t HW;          // input plane (floats)
  int64_t HoL;         // output plane (floats)
  uint64_t magic_L;    // ceil(2^32 / L)
  uint64_t magic_Fh;   // ceil(2^32 / Fh)
  uint64_t magic_HoL;  // ceil(2^32 / HoL)
};

__device__ __forceinline__ float4 ldg_stream(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

struct Cursor {  // position of an output element inside the CTA's range
  int32_t base;  // shared-memory index of (plane, row m, column 0, u = 0): plane*stride + m*s*W
  int32_t mm, k, u;
};

// One CTA: either PB whole consecutive planes (small planes), or one block of MB output rows of one
// plane.  In both cases the input it needs and the output it writes are one contiguous range each.
__global__ void __launch_bounds__(kThreads) transform_smem_kernel(const TransformParams P) {
  extern __shared__ __align__(16) float smem[];
  const int64_t job = blockIdx.x;
  const int64_t pg = job / P.nblk;
  const int32_t b = (int32_t)(job - pg * P.nblk);
  const bool whole = P.nblk == 1;
  const int64_t plane0 = pg * P.PB;
  const int32_t npl = whole ? (int32_t)min((int64_t)P.PB, P.planes - plane0) : 1;
  const int32_t m0 = b * P.MB;
  const int32_t mb = whole ? P.Ho : min(P.MB, P.Ho - m0);
  const int32_t rows_in = whole ? P.H : (mb - 1) * P.s + P.Fh;
  const int32_t plane_floats = rows_in * P.W;  // staged floats per plane
  const int32_t n_in = npl * plane_floats;

  // ---- stage the input range, keeping its 16-byte phase
  const float* src = P.in + plane0 * P.HW + (int64_t)m0 * P.s * P.W;
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
  float* dst = P.out + plane0 * P.HoL + (int64_t)m0 * P.L;
  const int32_t out_plane = mb * P.L;  // output floats per plane in this CTA
  const int32_t n_out = npl * out_plane;
  const int32_t dskew = (int32_t)((reinterpret_cast<uintptr_t>(dst) >> 2) & 3);
  const int32_t head = min((4 - dskew) & 3, n_out);
  const int32_t nvec = (n_out - head) >> 2;
  const int32_t tail0 = head + (nvec << 2);
  const int32_t sW = P.s * P.W;

  // element e of the output range -> cursor
  auto locate = [&](int32_t e) -> Cursor {
    int32_t pl = 0, rem = e;
    if (npl > 1) {
      pl = (int32_t)(((uint64_t)(uint32_t)e * P.magic_HoL) >> 32);
      rem = e - pl * out_plane;
    }
    const int32_t mm = (int32_t)(((uint64_t)(uint32_t)rem * P.magic_L) >> 32);
    const int32_t r2 = rem - mm * P.L;
    Cursor c;
    c.mm = mm;
    c.k = (int32_t)(((uint64_t)(uint32_t)r2 * P.magic_Fh) >> 32);
    c.u = r2 - c.k * P.Fh;
    c.base = pl * plane_floats + mm * sW;
    return c;
  };
  auto fetch = [&](const Cursor& c) { return tile[c.base + c.u * P.W + c.k]; };
  auto advance = [&](Cursor c) -> Cursor {
    if (++c.u == P.Fh) {
      c.u = 0;
      if (++c.k == P.W) {  // next strip: next output row, or the first row of the next plane
        c.k = 0;
        c.base += sW;
        if (++c.mm == mb) {  // first row of the next plane
          c.mm = 0;
          c.base += plane_floats - mb * sW;
        }
      }
    }
    return c;
  };

  if ((int32_t)threadIdx.x < head) dst[threadIdx.x] = fetch(locate(threadIdx.x));
  float4* dst4 = reinterpret_cast<float4*>(dst + head);
  for (int32_t i = threadIdx.x; i < nvec; i += kThreads) {
    Cursor c = locate(head + (i << 2));
    float4 v;
    v.x = fetch(c); c = advance(c);
    v.y = fetch(c); c = advance(c);
    v.z = fetch(c); c = advance(c);
    v.w = fetch(c);
    dst4[i] = v;
  }
  if ((int32_t)threadIdx.x < n_out - tail0) dst[tail0 + threadIdx.x] = fetch(locate(tail0 + threadIdx.x));
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
  int32_t nblk = (g.Ho + MB - 1) / MB;
  MB = (g.Ho + nblk - 1) / nblk;                         // balance the blocks
  // Small planes: several whole consecutive planes per CTA, so that a CTA still moves tens of KB.
  int32_t PB = 1;
  const int64_t hw = (int64_t)g.H * g.W;
  if (hw <= budget) {
    nblk = 1;
    MB = g.Ho;
    PB = (int32_t)(budget / hw);
    const int64_t want_ctas = 148 * 8;                   // keep enough CTAs to fill the machine
    if (planes / PB < want_ctas) PB = (int32_t)(planes / want_ctas > 0 ? planes / want_ctas : 1);
    if (PB < 1) PB = 1;
  }
  const int32_t rows_in = nblk == 1 ? g.H : (MB - 1) * g.s + g.Fh;
  const size_t smem = ((size_t)PB * rows_in * g.W + 4) * sizeof(float);
  const int64_t ctas = nblk == 1 ? (planes + PB - 1) / PB : planes * nblk;
  // magic-number division is exact while (range length) * divisor < 2^32
  const int64_t range = (int64_t)PB * (nblk == 1 ? g.HoL : (int64_t)MB * g.L);
  if (range * g.HoL >= ((int64_t)1 << 32) || ctas > INT32_MAX || smem > 200 * 1024) {
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
  P.MB = MB; P.nblk = nblk; P.PB = PB; P.planes = planes;
  P.HW = hw; P.HoL = g.HoL;
  P.magic_L = magic_for((uint32_t)g.L);
  P.magic_Fh = magic_for((uint32_t)g.Fh);
  P.magic_HoL = magic_for((uint32_t)g.HoL);
  transform_smem_kernel<<<(unsigned)ctas, kThreads, smem, st>>>(P);
  return cuda_status(cudaGetLastError());
}

}  // namespace im2win
