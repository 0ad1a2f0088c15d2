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
#include <cstdlib>
#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"

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
// FHT: the filter height as a compile-time constant (division by it is then a multiplication), or 0.
template <int FHT>
__global__ void __launch_bounds__(kThreads) transform_smem_kernel(const TransformParams P) {
  // a convolution launched next as a programmatic dependent may set up (barriers, tensor memory, resident
  // filter) while this grid drains; it waits for this grid's completion before it reads the im2win tensor
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ __align__(16) float smem[];
  const int32_t Fh = FHT ? FHT : P.Fh;
  const int64_t job = blockIdx.x;
  const int64_t pg = job / P.nblk;
  const int32_t b = (int32_t)(job - pg * P.nblk);
  const bool whole = P.nblk == 1;
  const int64_t plane0 = pg * P.PB;
  const int32_t npl = whole ? (int32_t)min((int64_t)P.PB, P.planes - plane0) : 1;
  const int32_t m0 = b * P.MB;
  const int32_t mb = whole ? P.Ho : min(P.MB, P.Ho - m0);
  const int32_t rows_in = whole ? P.H : (mb - 1) * P.s + Fh;
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
    c.u = r2 - c.k * Fh;
    c.base = pl * plane_floats + mm * sW;
    return c;
  };
  auto fetch = [&](const Cursor& c) { return tile[c.base + c.u * P.W + c.k]; };
  auto advance = [&](Cursor c) -> Cursor {
    if (++c.u == Fh) {
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
  static_assert(FHT == 0 || FHT >= 4, "a 16-byte chunk must not wrap the filter height twice");
  if (FHT != 0 && P.L >= 4 * kThreads) {
    // Long strips (the stems): the thread's position (strip, offset in the strip) is stepped from one
    // 16-byte chunk to its next, 4*kThreads elements on, instead of being located anew, and the four
    // gathers of a chunk that lies inside one strip walk (u, k) with compile-time Fh.  The kernel is
    // bound by its instruction count: this path issues about a third of the general one's.
    constexpr int FD = FHT ? FHT : 1;
    const int32_t L = P.L, W = P.W;
    Cursor c0 = locate(head + ((int32_t)threadIdx.x << 2));
    int32_t r2 = c0.k * FD + c0.u, mm = c0.mm, base = c0.base;
    for (int32_t i = threadIdx.x; i < nvec; i += kThreads) {
      float4 v;
      if (r2 + 3 < L) {
        int32_t k = r2 / FD, u = r2 - k * FD;
        const float* t = tile + base + k;
        int32_t idx = u * W;
        v.x = t[idx]; if (++u == FD) { u = 0; idx = idx - (FD - 1) * W + 1; } else idx += W;
        v.y = t[idx]; if (++u == FD) { u = 0; idx = idx - (FD - 1) * W + 1; } else idx += W;
        v.z = t[idx]; if (++u == FD) { u = 0; idx = idx - (FD - 1) * W + 1; } else idx += W;
        v.w = t[idx];
      } else {  // the chunk straddles two strips
        Cursor c;
        c.base = base; c.mm = mm; c.k = r2 / FD; c.u = r2 - c.k * FD;
        v.x = fetch(c); c = advance(c);
        v.y = fetch(c); c = advance(c);
        v.z = fetch(c); c = advance(c);
        v.w = fetch(c);
      }
      dst4[i] = v;
      r2 += 4 * kThreads;
      while (r2 >= L) {  // (at most once per step: L >= 4*kThreads)
        r2 -= L;
        base += sW;
        if (++mm == mb) { mm = 0; base += plane_floats - mb * sW; }
      }
    }
  } else {
    for (int32_t i = threadIdx.x; i < nvec; i += kThreads) {
      Cursor c = locate(head + (i << 2));
      float4 v;
      v.x = fetch(c); c = advance(c);
      v.y = fetch(c); c = advance(c);
      v.z = fetch(c); c = advance(c);
      v.w = fetch(c);
      dst4[i] = v;
    }
  }
  if ((int32_t)threadIdx.x < n_out - tail0) dst[tail0 + threadIdx.x] = fetch(locate(tail0 + threadIdx.x));
}

// bf16 storage variant of the staged-gather kernel: same jobs and staging, the output range walked
// in 16-byte chunks of eight bf16 (round to nearest even), one 128-bit store each.
__device__ __forceinline__ uint32_t bf16x2_rn(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint16_t bf16_rn(float x) { return (uint16_t)(bf16x2_rn(x, 0.f) & 0xffffu); }

__global__ void __launch_bounds__(kThreads) transform_smem_bf16_kernel(const TransformParams P, uint16_t* out16) {
  // a convolution launched next as a programmatic dependent may set up (barriers, tensor memory, resident
  // filter) while this grid drains; it waits for this grid's completion before it reads the im2win tensor
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
  const int32_t plane_floats = rows_in * P.W;
  const int32_t n_in = npl * plane_floats;

  const float* src = P.in + plane0 * P.HW + (int64_t)m0 * P.s * P.W;
  const int32_t skew = (int32_t)((reinterpret_cast<uintptr_t>(src) >> 2) & 3);
  float* tile = smem + skew;
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

  uint16_t* dst = out16 + plane0 * P.HoL + (int64_t)m0 * P.L;
  const int32_t out_plane = mb * P.L;
  const int32_t n_out = npl * out_plane;
  const int32_t dskew = (int32_t)((reinterpret_cast<uintptr_t>(dst) >> 1) & 7);  // 16-byte phase in elements
  const int32_t head = min((8 - dskew) & 7, n_out);
  const int32_t nvec = (n_out - head) >> 3;
  const int32_t tail0 = head + (nvec << 3);
  const int32_t sW = P.s * P.W;
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
      if (++c.k == P.W) {
        c.k = 0;
        c.base += sW;
        if (++c.mm == mb) {
          c.mm = 0;
          c.base += plane_floats - mb * sW;
        }
      }
    }
    return c;
  };
  if ((int32_t)threadIdx.x < head) dst[threadIdx.x] = bf16_rn(fetch(locate(threadIdx.x)));
  uint4* dst4 = reinterpret_cast<uint4*>(dst + head);
  for (int32_t i = threadIdx.x; i < nvec; i += kThreads) {
    Cursor c = locate(head + (i << 3));
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      x[j] = fetch(c);
      if (j < 7) c = advance(c);
    }
    uint4 v;
    v.x = bf16x2_rn(x[0], x[1]); v.y = bf16x2_rn(x[2], x[3]);
    v.z = bf16x2_rn(x[4], x[5]); v.w = bf16x2_rn(x[6], x[7]);
    dst4[i] = v;
  }
  if ((int32_t)threadIdx.x < n_out - tail0) dst[tail0 + threadIdx.x] = bf16_rn(fetch(locate(tail0 + threadIdx.x)));
}

// one thread per element; any shape
__global__ void __launch_bounds__(kThreads) transform_gather_bf16_kernel(const float* __restrict__ in,
                                                                          uint16_t* __restrict__ out,
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
    out[e] = bf16_rn(__ldg(in + (plane * H + (int64_t)m * s + u) * W + k));
  }
}

// ------------------------------------------------------------------------------------------------
// Tile kernel: the same jobs (whole planes, or a block of output rows of one plane), but all global
// traffic is two TMA bulk copies.  The input range comes into shared memory with one
// cp.async.bulk; the threads transpose it shared -> shared into a second buffer that holds the
// job's output range in its final order; one cp.async.bulk stores that buffer.  A thread handles
// four input columns of one strip at a time: FH vector loads (4 consecutive floats of a row) and
// 4*FH contiguous output floats, i.e. a few instructions per 16 bytes instead of a gather per
// element.  Both buffers keep the 16-byte phase of their global ranges, so the bulk copies move
// aligned chunks; the at most 3 + 3 floats outside the aligned part are copied by threads.
struct TileParams {
  const float* in;
  void* out;            // fp32 im2win tensor, or 16-bit words for the bf16 storage variant
  int32_t* status;
  int32_t H, W, s, Ho, L;
  int32_t MB, nblk, PB;
  int32_t QW;           // column quads per row: ceil(W / 4)
  int64_t planes, HW, HoL, n_in_total;
  uint64_t magic_QW;    // ceil(2^32 / QW)
  uint64_t magic_MQ;    // ceil(2^32 / (rows per plane in the job * QW))
  int32_t test_skip_copy;  // test hook, see the kernel
  uint32_t off_out;     // byte offset of the output buffer in shared memory
  uint32_t off_bar;     // byte offset of the mbarrier
};

// OUT16: the output is the bf16 storage variant (P.out then points at 16-bit words).
template <int FH, bool OUT16>
__global__ void __launch_bounds__(kThreads) transform_tile_kernel(const TileParams P) {
  // a convolution launched next as a programmatic dependent may set up (barriers, tensor memory, resident
  // filter) while this grid drains; it waits for this grid's completion before it reads the im2win tensor
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using OutT = typename std::conditional<OUT16, uint16_t, float>::type;
  constexpr int32_t OPC = OUT16 ? 8 : 4;  // output elements per 16-byte chunk
  extern __shared__ __align__(128) uint8_t smem_raw[];
  float* const tin0 = reinterpret_cast<float*>(smem_raw);
  OutT* const tout0 = reinterpret_cast<OutT*>(smem_raw + P.off_out);
  uint64_t* const bar = reinterpret_cast<uint64_t*>(smem_raw + P.off_bar);

  const int64_t job = blockIdx.x;
  const int64_t pg = job / P.nblk;
  const int32_t b = (int32_t)(job - pg * P.nblk);
  const bool whole = P.nblk == 1;
  const int64_t plane0 = pg * P.PB;
  const int32_t npl = whole ? (int32_t)min((int64_t)P.PB, P.planes - plane0) : 1;
  const int32_t m0 = b * P.MB;
  const int32_t mb = whole ? P.Ho : min(P.MB, P.Ho - m0);
  const int32_t rows_in = whole ? P.H : (mb - 1) * P.s + FH;
  const int32_t plane_floats = rows_in * P.W;
  const int32_t n_in = npl * plane_floats;
  const int32_t out_plane = mb * P.L;
  const int32_t n_out = npl * out_plane;

  // ---- input range -> shared memory (one bulk copy of the enclosing aligned range)
  const int64_t src0 = plane0 * P.HW + (int64_t)m0 * P.s * P.W;  // first float of the range
  const int32_t skew = (int32_t)(src0 & 3);                      // P.in is 16-byte aligned
  const float* const tin = tin0 + skew;                           // tin[e] <-> in[src0 + e]
  const int64_t a0 = src0 - skew;
  int32_t nfl = (skew + n_in + 3) & ~3;
  int32_t ntail = 0;                                              // floats past the last whole chunk
  if (a0 + nfl > P.n_in_total) {                                  // the last chunk would pass the tensor's end
    nfl = (int32_t)((P.n_in_total - a0) & ~(int64_t)3);
    ntail = (int32_t)(P.n_in_total - a0) - nfl;
  }
  const uint32_t bar_a = ptx::smem_u32(bar);
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_a, 1);
    ptx::fence_mbar_init();
    ptx::mbar_arrive_expect_tx(bar_a, (uint32_t)nfl * 4u);
    // (test hook: with test_skip_copy the copy is announced but never issued, so that the expiry
    // path of the bounded wait below can be exercised by a kernel that neither faults nor hangs)
    if (nfl > 0 && !P.test_skip_copy) ptx::bulk_g2s(ptx::smem_u32(tin0), P.in + a0, (uint32_t)nfl * 4u, bar_a);
  }
  if ((int32_t)threadIdx.x < ntail) tin0[nfl + threadIdx.x] = __ldg(P.in + a0 + nfl + threadIdx.x);
  __syncthreads();  // the barrier is initialised for everyone; the tail floats are in place
  {
    // bounded wait: about a second by the global timer (and an iteration cap), then report and leave
    bool landed = ptx::mbar_try_wait(bar_a, 0u);
    uint64_t t0 = 0;
    for (uint32_t it = 0; it < (1u << 22) && !landed; ++it) {
      __nanosleep(64);
      landed = ptx::mbar_try_wait(bar_a, 0u);
      if ((it & 63u) == 63u && !landed) {
        uint64_t now;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        else if (now - t0 > 1000000000ull) break;
      }
    }
    if (!__all_sync(0xffffffffu, landed)) {
      if ((threadIdx.x & 31) == 0) atomicCAS(P.status, 0, (int32_t)DEV_TIMEOUT_COPY);
      return;
    }
  }

  // ---- transpose shared -> shared
  const int64_t dst0 = plane0 * P.HoL + (int64_t)m0 * P.L;       // first element of the output range
  const int32_t dskew = (int32_t)(dst0 & (OPC - 1));              // P.out is 16-byte aligned
  OutT* const tout = tout0 + dskew;                               // tout[e] <-> out[dst0 + e]
  const int32_t sW = P.s * P.W;
  const int32_t units_plane = mb * P.QW;
  const int32_t nunits = npl * units_plane;
  const bool in_even = ((P.W | skew) & 1) == 0;                  // every row start is 8-byte aligned
  for (int32_t q = threadIdx.x; q < nunits; q += kThreads) {
    int32_t pl = 0, rem = q;
    if (npl > 1) {
      pl = (int32_t)(((uint64_t)(uint32_t)q * P.magic_MQ) >> 32);
      rem = q - pl * units_plane;
    }
    const int32_t mm = (int32_t)(((uint64_t)(uint32_t)rem * P.magic_QW) >> 32);
    const int32_t k0 = (rem - mm * P.QW) * 4;
    const float* src = tin + pl * plane_floats + mm * sW + k0;
    const int32_t oe = pl * out_plane + mm * P.L + k0 * FH;
    OutT* dst = tout + oe;
    if (k0 + 4 <= P.W) {
      float r[4 * FH];  // r[c*FH + u] = I[m*s + u][k0 + c]: the 4*FH output floats in order
      if (in_even) {
#pragma unroll
        for (int u = 0; u < FH; ++u) {
          const float2 x = *reinterpret_cast<const float2*>(src + u * P.W);
          const float2 y = *reinterpret_cast<const float2*>(src + u * P.W + 2);
          r[0 * FH + u] = x.x; r[1 * FH + u] = x.y; r[2 * FH + u] = y.x; r[3 * FH + u] = y.y;
        }
      } else {
#pragma unroll
        for (int u = 0; u < FH; ++u) {
#pragma unroll
          for (int c = 0; c < 4; ++c) r[c * FH + u] = src[u * P.W + c];
        }
      }
      if constexpr (OUT16) {
        // 4*FH bf16 in order: 32-bit stores of rounded pairs where the run starts on a 4-byte
        // boundary, else element by element
        if (((dskew + oe) & 1) == 0) {
#pragma unroll
          for (int j = 0; j < 2 * FH; ++j) reinterpret_cast<uint32_t*>(dst)[j] = bf16x2_rn(r[2 * j], r[2 * j + 1]);
        } else {
#pragma unroll
          for (int j = 0; j < 4 * FH; ++j) dst[j] = bf16_rn(r[j]);
        }
        continue;
      }
      const int32_t a = (dskew + oe) & 3;  // 16-byte phase of the run in the output buffer
      if constexpr (!OUT16) {
        if (a == 0) {
#pragma unroll
          for (int j = 0; j < FH; ++j)
            reinterpret_cast<float4*>(dst)[j] = make_float4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        } else if (a == 2) {
          *reinterpret_cast<float2*>(dst) = make_float2(r[0], r[1]);
#pragma unroll
          for (int j = 0; j < FH - 1; ++j)
            *reinterpret_cast<float4*>(dst + 2 + 4 * j) = make_float4(r[4 * j + 2], r[4 * j + 3], r[4 * j + 4], r[4 * j + 5]);
          *reinterpret_cast<float2*>(dst + 4 * FH - 2) = make_float2(r[4 * FH - 2], r[4 * FH - 1]);
        } else {
#pragma unroll
          for (int j = 0; j < 4 * FH; ++j) dst[j] = r[j];
        }
      }
    } else {  // the last, partial quad of a row
      for (int32_t c = 0; k0 + c < P.W; ++c)
#pragma unroll
        for (int u = 0; u < FH; ++u) {
          if constexpr (OUT16) dst[c * FH + u] = bf16_rn(src[u * P.W + c]);
          else dst[c * FH + u] = src[u * P.W + c];
        }
    }
  }
  ptx::fence_proxy_async_smem();  // the buffer is about to be read by the bulk copy
  __syncthreads();

  // ---- output buffer -> global: one bulk copy of the aligned part, threads for the ragged ends
  const int32_t head = min((OPC - dskew) & (OPC - 1), n_out);
  const int32_t nvec = (n_out - head) / OPC;
  const int32_t tail0 = head + nvec * OPC;
  OutT* const gout = reinterpret_cast<OutT*>(P.out) + dst0;
  if (threadIdx.x == 0 && nvec > 0) {
    ptx::bulk_s2g(gout + head, ptx::smem_u32(tout + head), (uint32_t)nvec * 16u);
    ptx::bulk_s2g_commit();
  }
  if ((int32_t)threadIdx.x < head) gout[threadIdx.x] = tout[threadIdx.x];
  if ((int32_t)threadIdx.x < n_out - tail0) gout[tail0 + threadIdx.x] = tout[tail0 + threadIdx.x];
  if (threadIdx.x == 0 && nvec > 0) ptx::bulk_s2g_wait_read();  // shared memory must outlive the copy's reads
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

template <int FH, bool OUT16>
int launch_tile_fh(const TileParams& P, int64_t ctas, size_t smem, cudaStream_t st) {
  auto kern = transform_tile_kernel<FH, OUT16>;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  kern<<<(unsigned)ctas, kThreads, smem, st>>>(P);
  return cuda_status(cudaGetLastError());
}

// Tile kernel where a job's input and output ranges fit one shared-memory budget together (a sixth
// or an eighth of an SM's shared memory, so that six or eight CTAs overlap their loads, transposes and stores);
// IM2WIN_EUNSUPPORTED otherwise (the caller then uses the staged-gather kernel).
int launch_transform_tile(const float* in, void* out, bool out16, const Geometry& g, cudaStream_t st) {
  if (g.Fh != 1 && g.Fh != 2 && g.Fh != 3 && g.Fh != 4 && g.Fh != 5 && g.Fh != 7 && g.Fh != 11) return IM2WIN_EUNSUPPORTED;
  int64_t kBudget = 8704 - 16;  // floats for input + output ranges: 34 KB with the phase skews, six CTAs per SM
  const int64_t planes = (int64_t)g.N * g.C;
  const int64_t hw = (int64_t)g.H * g.W;
  // small planes (several whole planes per CTA): 28 KB, eight CTAs per SM, measured 3-8 % faster on the
  // launch- and tail-bound layers; row blocks of larger planes keep 34 KB (shorter blocks re-read more rows)
  if (hw + g.HoL <= 7168 - 16) kBudget = 7168 - 16;
  if (knobs().transform_budget_kb) kBudget = (int64_t)knobs().transform_budget_kb * 256 - 16;  // (test build)
  int32_t PB = 1, MB = g.Ho, nblk = 1;
  if (hw + g.HoL <= kBudget) {
    PB = (int32_t)(kBudget / (hw + g.HoL));
    const int64_t want_ctas = 148 * 8;  // keep enough CTAs to fill the machine
    if (planes / PB < want_ctas) PB = (int32_t)(planes / want_ctas > 0 ? planes / want_ctas : 1);
    if (PB < 1) PB = 1;
  } else {
    const int64_t mbmax = (kBudget - (int64_t)(g.Fh - g.s) * g.W) / ((int64_t)g.s * g.W + g.L);
    if (mbmax < 1) return IM2WIN_EUNSUPPORTED;
    MB = (int32_t)(mbmax < g.Ho ? mbmax : g.Ho);
    nblk = (g.Ho + MB - 1) / MB;
    MB = (g.Ho + nblk - 1) / nblk;  // balance the blocks
    // neighbouring blocks re-read Fh - s rows each; with the output buffer taking most of the
    // budget, wide rows leave blocks so short that this would dominate: leave those to the
    // staged-gather kernel, which stages the input only
    if ((int64_t)(g.Fh - g.s) * 8 > (int64_t)(MB - 1) * g.s + g.Fh) return IM2WIN_EUNSUPPORTED;
  }
  const int64_t ctas = nblk == 1 ? (planes + PB - 1) / PB : planes * nblk;
  if (ctas > INT32_MAX) return IM2WIN_EUNSUPPORTED;
  const int32_t rows_in = nblk == 1 ? g.H : (MB - 1) * g.s + g.Fh;
  const int64_t in_floats = (int64_t)PB * rows_in * g.W + 8;                       // + phase skew and rounding
  const int64_t out_floats = (int64_t)PB * (nblk == 1 ? g.HoL : (int64_t)MB * g.L) + 8;
  TileParams P;
  P.in = in; P.out = out;
  P.status = device_status_word();
  if (!P.status) return IM2WIN_ECUDA;
  P.H = g.H; P.W = g.W; P.s = g.s; P.Ho = g.Ho; P.L = g.L;
  P.MB = MB; P.nblk = nblk; P.PB = PB;
  P.QW = (g.W + 3) / 4;
  {
    // honoured for single-CTA problems only: every CTA would wait out its own second otherwise
    P.test_skip_copy = (knobs().test_skip_copy && ctas == 1) ? 1 : 0;
  }
  P.planes = planes; P.HW = hw; P.HoL = g.HoL; P.n_in_total = g.n_in;
  const int64_t units_plane = (int64_t)(nblk == 1 ? g.Ho : MB) * P.QW;
  if (units_plane * PB * units_plane >= ((int64_t)1 << 32)) return IM2WIN_EUNSUPPORTED;  // reciprocal division exact
  P.magic_QW = magic_for((uint32_t)P.QW);
  P.magic_MQ = magic_for((uint32_t)units_plane);
  P.off_out = (uint32_t)((in_floats * 4 + 127) / 128 * 128);
  P.off_bar = P.off_out + (uint32_t)((out_floats * (out16 ? 2 : 4) + 15) / 16 * 16);
  const size_t smem = P.off_bar + 16;
  switch (g.Fh) {
    case 1: return out16 ? launch_tile_fh<1, true>(P, ctas, smem, st) : launch_tile_fh<1, false>(P, ctas, smem, st);
    case 2: return out16 ? launch_tile_fh<2, true>(P, ctas, smem, st) : launch_tile_fh<2, false>(P, ctas, smem, st);
    case 3: return out16 ? launch_tile_fh<3, true>(P, ctas, smem, st) : launch_tile_fh<3, false>(P, ctas, smem, st);
    case 4: return out16 ? launch_tile_fh<4, true>(P, ctas, smem, st) : launch_tile_fh<4, false>(P, ctas, smem, st);
    case 5: return out16 ? launch_tile_fh<5, true>(P, ctas, smem, st) : launch_tile_fh<5, false>(P, ctas, smem, st);
    case 7: return out16 ? launch_tile_fh<7, true>(P, ctas, smem, st) : launch_tile_fh<7, false>(P, ctas, smem, st);
    default: return out16 ? launch_tile_fh<11, true>(P, ctas, smem, st) : launch_tile_fh<11, false>(P, ctas, smem, st);
  }
}

// Staged-gather path (and, for rows too long to stage, the per-element kernel), writing fp32 (`out`)
// or, when `out16` is given, the bf16 storage variant.
static int launch_transform_staged(const float* in, float* out, uint16_t* out16, const Geometry& g, cudaStream_t st) {
  // Shared-memory budget for the staged input rows.  Small enough for several CTAs per SM so that
  // one CTA's loads overlap another's stores.
  constexpr int32_t kTileFloats = 8192 - 4;      // 32 KB including the phase skew
  constexpr int32_t kTileFloatsMax = 49152 - 4;  // opt-in ceiling for very wide rows
  const int64_t planes = (int64_t)g.N * g.C;
  const int64_t row_floats = (int64_t)g.Fh * g.W;

  if (row_floats > kTileFloatsMax) {
    const int64_t blocks = (g.n_win + kThreads - 1) / kThreads;
    const int grid = (int)(blocks < 148 * 64 ? blocks : 148 * 64);
    if (out16) transform_gather_bf16_kernel<<<grid, kThreads, 0, st>>>(in, out16, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
    else transform_gather_kernel<<<grid, kThreads, 0, st>>>(in, out, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
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
    if (out16) transform_gather_bf16_kernel<<<grid, kThreads, 0, st>>>(in, out16, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
    else transform_gather_kernel<<<grid, kThreads, 0, st>>>(in, out, g.H, g.W, g.Fh, g.s, g.Ho, g.n_win);
    return cuda_status(cudaGetLastError());
  }
  if (smem > 48 * 1024) {
    cudaError_t e = out16 ? cudaFuncSetAttribute(transform_smem_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                          : (g.Fh == 7 ? cudaFuncSetAttribute(transform_smem_kernel<7>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                             : g.Fh == 11 ? cudaFuncSetAttribute(transform_smem_kernel<11>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                          : cudaFuncSetAttribute(transform_smem_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
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
  if (out16) transform_smem_bf16_kernel<<<(unsigned)ctas, kThreads, smem, st>>>(P, out16);
  else if (g.Fh == 7) transform_smem_kernel<7><<<(unsigned)ctas, kThreads, smem, st>>>(P);
  else if (g.Fh == 11) transform_smem_kernel<11><<<(unsigned)ctas, kThreads, smem, st>>>(P);
  else transform_smem_kernel<0><<<(unsigned)ctas, kThreads, smem, st>>>(P);
  return cuda_status(cudaGetLastError());
}

int launch_transform(const float* in, float* out, const Geometry& g, cudaStream_t st) {
  {
    if (!knobs().transform_gather) {
      const int rc = launch_transform_tile(in, out, false, g, st);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
  }
  return launch_transform_staged(in, out, nullptr, g, st);
}

int launch_transform_bf16(const float* in, uint16_t* out, const Geometry& g, cudaStream_t st) {
  {
    if (!knobs().transform_gather) {
      const int rc = launch_transform_tile(in, out, true, g, st);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
  }
  return launch_transform_staged(in, nullptr, out, g, st);
}

}  // namespace im2win
