// Shared pieces of the shared-memory-operand tensor-core kernels (conv_tc_strip.cu, conv_tc_window.cu):
// barrier block, bounded waits, TMA / cluster / tcgen05 pair helpers, the pipelined TMEM -> NCHW store.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <cstdint>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
#ifdef IM2WIN_PROF
extern long long* g_prof;  // debug build: counter buffer (defined in conv_tc_persistent.cu)
#define SPROF_DECL long long pw[7] = {}; const long long pt0 = clock64();
#define SPROF_W(k, ...) { const long long c0_ = clock64(); __VA_ARGS__; pw[k] += clock64() - c0_; }
#define SPROF_DUMP(role) if (P.prof && blockIdx.x < 8 && lane == 0) { long long* o_ = P.prof + ((long long)blockIdx.x * 8 + (role)) * 8; o_[0] = clock64() - pt0; for (int z_ = 0; z_ < 7; ++z_) o_[1 + z_] = pw[z_]; }
#else
#define SPROF_DECL
#define SPROF_W(k, ...) { __VA_ARGS__; }
#define SPROF_DUMP(role)
#endif
namespace stripc {

constexpr int kTW = 8;             // transposer warps
constexpr int kTWarp0 = 4;
constexpr int kEpiWarp0 = kTWarp0 + kTW;
constexpr int kMaxRaw = 12, kMaxB = 12;
constexpr int kTMax = 3;           // transposer tasks per thread and source stage
constexpr uint32_t kSpin = 1u << 22;

struct SBars {
  uint64_t raw_full[kMaxRaw], raw_empty[kMaxRaw];
  uint64_t b_full[kMaxB], b_empty[kMaxB];
  uint64_t t_full[2], t_empty[2];
  uint64_t acc_full[2], acc_empty[2];
};
struct SMisc {
  uint32_t tmem_base;
  int32_t abort;
};

struct Ring {
  int32_t idx = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void advance(int32_t n) {
    if (++idx == n) { idx = 0; phase ^= 1u; }
  }
};

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait (about a second): polls with a back-off; on expiry records `code`, raises the CTA's
// abort flag (which ends every other role's wait at its next look) and returns false.
static __device__ __noinline__ bool wait_slow(int32_t* status, SMisc* misc, uint32_t bar, uint32_t parity, int32_t code,
                                       uint32_t sleep_ns) {
  uint64_t t0 = 0;
  for (uint32_t it = 0; it < kSpin; ++it) {
    __nanosleep(sleep_ns);
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*reinterpret_cast<volatile int32_t*>(&misc->abort)) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 1000000000ull) break;
    }
  }
  atomicCAS(status, 0, code);
  atomicExch(&misc->abort, 1);
  return false;
}
template <class PT>
__device__ __forceinline__ bool wait_bar(const PT& P, SMisc* misc, uint32_t bar, uint32_t parity, int32_t code,
                                         uint32_t sleep_ns = 32) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  return wait_slow(P.status, misc, bar, parity, code, sleep_ns);
}
template <class PT>
__device__ __forceinline__ bool wait_bar_warp(const PT& P, SMisc* misc, uint32_t bar, uint32_t parity, int32_t code,
                                              uint32_t sleep_ns = 32) {
  return __all_sync(0xffffffffu, wait_bar(P, misc, bar, parity, code, sleep_ns));
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
  uint32_t v;
  asm volatile("{\n.reg .b16 h;\nld.shared.u16 h, [%1];\ncvt.u32.u16 %0, h;\n}" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts_v4(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Cluster helpers (pair mode: a cluster of two CTAs).
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA box whose completion is signalled on a barrier of the pair's leader CTA (a shared::cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
// tcgen05.mma with both operands from shared memory (descriptors passed as 32-bit halves) and tcgen05.commit,
// for one CTA or for a CTA pair (cta_group::2: D[tmem of both CTAs] (+)= A[each CTA's own rows] * B[each CTA
// holds half the N rows], M = 256; the commit arrives on both CTAs' barriers).  The role that issues them is run
// by a WHOLE warp (descriptor arithmetic and waits are then
// warp-uniform work, which the compiler can keep in uniform registers: tcgen05.mma takes its operands from
// those): only the lane with `elect` set issues.
template <bool BF16, bool PAIR>
__device__ __forceinline__ void mma_ss_e(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                         uint32_t idesc, uint32_t accumulate, uint32_t elect) {
#define IM2WIN_MMA_E(GROUP, KIND)                                                                                   \
  asm volatile("{\n\t.reg .pred p, q;\n\t.reg .b64 ad, bd;\n\t"                                                    \
               "setp.ne.b32 p, %6, 0;\n\t"                                                                          \
               "setp.ne.b32 q, %7, 0;\n\t"                                                                          \
               "mov.b64 ad, {%1, %2};\n\t"                                                                          \
               "mov.b64 bd, {%3, %4};\n\t"                                                                          \
               "@q tcgen05.mma.cta_group::" GROUP ".kind::" KIND " [%0], ad, bd, %5, p;\n\t}"                        \
               ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(elect) : "memory")
  if constexpr (PAIR) {
    if constexpr (BF16) IM2WIN_MMA_E("2", "f16"); else IM2WIN_MMA_E("2", "tf32");
  } else {
    if constexpr (BF16) IM2WIN_MMA_E("1", "f16"); else IM2WIN_MMA_E("1", "tf32");
  }
#undef IM2WIN_MMA_E
}
template <bool PAIR>
__device__ __forceinline__ void mma_commit_e(uint32_t bar, uint32_t elect) {
  if constexpr (PAIR)
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t"
                 "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
                 ::"r"(bar), "h"((uint16_t)3), "r"(elect) : "memory");
  else
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                 ::"r"(bar), "r"(elect) : "memory");
}

// Stores columns [c_begin, c_end) (multiples of 16) of one warp's 32 accumulator rows: TMEM -> registers
// -> the output (column stride Ho*Wo for NCHW; 1, with 128-bit stores where aligned, for NHWC).  The TMEM load of the next 16 columns is in flight while the current 16 are stored.  With
// zero_behind the columns are zeroed once read (kernels whose MMAs all accumulate).
__device__ __forceinline__ void store16(float* o, int64_t cstride, const uint32_t (&v)[16], int32_t left, bool vec) {
  if (vec && left >= 16) {  // (NHWC: a position's filters are contiguous)
#pragma unroll
    for (int e = 0; e < 16; e += 4)
      *reinterpret_cast<float4*>(o + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]), __uint_as_float(v[e + 2]),
                                                      __uint_as_float(v[e + 3]));
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if (e < left) o[(int64_t)e * cstride] = __uint_as_float(v[e]);
  }
}
__device__ __forceinline__ void store_columns(uint32_t d_tmem, float* orow, int64_t cstride, int32_t c_begin, int32_t c_end,
                                              int32_t k_left, bool valid, bool zero_behind = false, bool vec = false) {
  uint32_t va[16], vb[16];
  if (c_begin >= c_end) return;
  ptx::tmem_ld_x16(d_tmem + (uint32_t)c_begin, va);
#pragma unroll 1
  for (int32_t c0 = c_begin; c0 < c_end; c0 += 32) {
    ptx::tmem_wait_ld();
    const bool more = c0 + 16 < c_end;
    if (more) ptx::tmem_ld_x16(d_tmem + (uint32_t)(c0 + 16), vb);
    if (zero_behind) ptx::tmem_zero_x16(d_tmem + (uint32_t)c0);  // (the columns just read: the next unit accumulates onto zeros)
    if (valid) store16(orow + (int64_t)c0 * cstride, cstride, va, k_left - c0, vec);
    if (more) {
      ptx::tmem_wait_ld();
      if (c0 + 32 < c_end) ptx::tmem_ld_x16(d_tmem + (uint32_t)(c0 + 32), va);
      if (zero_behind) ptx::tmem_zero_x16(d_tmem + (uint32_t)(c0 + 16));
      if (valid) store16(orow + (int64_t)(c0 + 16) * cstride, cstride, vb, k_left - c0 - 16, vec);
    }
  }
  if (zero_behind) ptx::tmem_wait_st();
}

// ---- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline EncodeTiledFn encode_fn() {
  static std::atomic<void*> cached{nullptr};
  void* p = cached.load(std::memory_order_acquire);
  if (!p) {
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    cached.store(p, std::memory_order_release);
  }
  return reinterpret_cast<EncodeTiledFn>(p);
}

}  // namespace stripc
}  // namespace im2win
