// im2win-based convolution (Algorithm 2) on the sm_100a tensor cores: persistent, specialised kernel.
//
// Same GEMM view as the generic kernel (M = output positions, N = filters, K = (r,u,v); A = windows in
// TENSOR MEMORY written by tcgen05.st, B = filters in shared memory, fp32 accumulators in TMEM), with
//   * one persistent CTA per SM walking work units t, t+grid, ... (neighbouring CTAs work on
//     neighbouring tiles at the same time, so the few strip floats two tiles share are L2 hits);
//     tiles are cut per image where that wastes little (one contiguous source range per channel,
//     one 2-D TMA box per channel group where it fits), else they may span images;
//   * the filter operand either RESIDENT in shared memory for the whole kernel (fetched by TMA with
//     the 32-byte swizzle where the native order serves as is, else built once per CTA from the
//     native K,C,Fh,Fw order; any shape, TF32 or BF16) or STREAMED per tile by TMA tensor loads
//     straight from the native filter viewed as a K x (C*Fh*Fw) matrix (128-byte swizzle);
//   * a unit's channel groups optionally cut into reduction slices that add into a zeroed output
//     (under-filled launches); the strip source optionally a bf16 im2win tensor or (fused) the
//     untransformed input;
//   * filter sizes known at compile time, so a window's elements are loads at immediate offsets from
//     one per-thread, per-channel base address (the window is contiguous in its im2win strip);
//   * A columns handed to the MMA thread in sub-slots of a ring in TMEM, independent of the channel
//     grouping of the staged strips;
//   * two accumulator buffers when they fit, so that the epilogue of one tile (tcgen05.ld -> NCHW
//     stores) overlaps the next tile's main loop.
// Warps (20): 0 strip producer (TMA); 1-3 MMA issuers, one per repack set (resident filter), or 1 MMA
// issuer and 2 filter producer (streamed filter); 4-15 window repack in up to three sets of four
// (one warp per TMEM lane quarter), the sets taking channel groups in turn; 16-19 epilogue.
// Every wait is bounded (status word + common teardown on expiry).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {
#ifdef IM2WIN_PROF
__attribute__((weak)) long long* g_prof = nullptr;  // debug build: one counter buffer shared by the parts
#endif

namespace {

constexpr int kThreads = 640;       // 20 warps: see the role list above the kernel
constexpr int kMaxSets = 3;         // repack warp sets (and MMA-issuing threads with a resident filter)
constexpr int kRepackWarp0 = 4;     // first repack warp: sets of four (one per TMEM lane quarter)
constexpr int kEpiWarp0 = kRepackWarp0 + 4 * kMaxSets;
constexpr int kSegMax = 8;
constexpr int kMaxStages = 12;
constexpr int kMaxSub = 16;
constexpr uint32_t kSpinLimit = 1u << 22;

struct PParams {
  const void* xhat;     // strip source: fp32 im2win tensor / untransformed input, or a bf16 im2win tensor
  const float* f;
  float* out;
  int32_t* status;
  int32_t C, K, Ho, Wo;
  int32_t nhwc;         // output layout N x Ho x Wo x K (fp32, no reduction slices)
  int32_t row_mul;      // source floats from one output row to the next: W*Fh (im2win strips) or s*W (raw rows)
  int32_t col_mul;      // source floats from one output column to the next: s*Fh or s
  int32_t win_span;     // floats from a window's first to one past its last element: Fh*Fw or (Fh-1)*W+Fw
  int32_t W;            // input row length (fused source addressing)
  int64_t plane;        // floats per (image, channel) plane of the source: Ho*W*Fh or H*W
  int32_t HoWo;         // output positions per image (fits 32 bits; checked on the host)
  int64_t Kg, Mtot, n_src;
  int32_t TP, NT, n_ntiles;
  int32_t Z, GZ;        // reduction slices per (m-tile, n-tile) and channel groups per slice (Z > 1: results are added into a zeroed output)
  int32_t usub;         // work units per m-tile: n_ntiles * Z
  int64_t ntiles;       // m tiles * n tiles
  int32_t NG;           // channel groups per tile
  int32_t SR, SB;       // raw strip stages; filter stages (streamed mode)
  int32_t NSETS;        // repack warp sets taking channel groups in turn (2 or 3)
  int32_t SS, NSS;      // MMA steps per A slot; slots per repack set in the TMEM ring
  int32_t ND;           // accumulator buffers
  int32_t chan_pitch;
  int32_t pim;          // 1: tiles are cut per image (a tile never spans two images)
  int32_t box;          // 1 (implies pim): strips come as one 2-D TMA box per channel group
  int32_t TPI;          // pim: tiles per image
  uint64_t magic_TPI, magic_Wo;  // pim: ceil(2^32 / d); n / d == (n * magic) >> 32 while n * d < 2^32 (host check)
  int32_t nchunks;      // 128-byte filter chunks per tile
  int32_t l2_ahead;     // box mode: request the next tile's boxes into L2 one tile ahead
  int32_t wait_prev;    // the preceding kernel in the stream is not this call's own filter copy: source reads and output writes wait for it
  int32_t bslice;       // resident filter holds only this CTA's reduction slice (grid is a multiple of Z)
  int32_t b_tma;        // resident filter fetched by TMA (TF32, dense groups) instead of built by the threads
  int32_t tmem_cols;
  uint32_t idesc;
  uint32_t off_raw, off_zero, off_bar, off_misc;  // shared-memory offsets in bytes
#ifdef IM2WIN_PROF
  long long* prof;  // debug build only: per-role wait-cycle counters of the first CTAs
#endif
};

struct PBars {
  uint64_t raw_full[kMaxStages], raw_empty[kMaxStages];
  uint64_t b_full[kMaxStages], b_empty[kMaxStages];
  uint64_t a_full[kMaxSub], a_empty[kMaxSub];
  uint64_t acc_full[2], acc_empty[2];
};

struct PMisc {
  uint32_t tmem_base;
  int32_t abort;
};

struct SegR {
  int64_t start0;
  int64_t virt_a;
  int32_t len;
  int32_t dst_off;
};

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

#ifdef IM2WIN_PROF
#define PROF_DECL(n) long long prof_acc[n] = {}; const long long prof_t0 = clock64();
#define PROF_SLOT(k) (&prof_acc[k])
#define PROF_T0(v) const long long v = clock64();
#define PROF_ADD(k, v) prof_acc[k] += clock64() - (v);
#define PROF_DUMP(role, n)                                                         \
  if (P.prof && blockIdx.x < 8 && lane == 0) {                                     \
    long long* o = P.prof + ((long long)blockIdx.x * 8 + (role)) * 8;              \
    o[0] = clock64() - prof_t0;                                                    \
    for (int z = 0; z < (n); ++z) o[1 + z] = prof_acc[z];                          \
  }
#else
#define PROF_DECL(n)
#define PROF_SLOT(k) nullptr
#define PROF_T0(v)
#define PROF_ADD(k, v)
#define PROF_DUMP(role, n)
#endif

// Bounded wait (about a second).  A warp that is not ready backs off with nanosleep between polls:
// sixteen warps share four schedulers, and a warp that spins on try_wait takes issue slots from the
// MMA-issuing thread on its scheduler, whose instruction rate is what bounds small-N tiles.
// The polling loop lives in one out-of-line copy: the call sites keep only the first poll, which
// keeps the roles' hot loops short (instruction fetch is a visible cost in this kernel).
__device__ __noinline__ bool wait_bar_slow(int32_t* status, PMisc* misc, uint32_t b, uint32_t parity, int32_t code,
                                           uint32_t sleep_ns) {
  uint64_t t0 = 0;
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    __nanosleep(sleep_ns);
    if (ptx::mbar_try_wait(b, parity)) return true;
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

__device__ __forceinline__ bool wait_bar_a(const PParams& P, PMisc* misc, uint32_t b, uint32_t parity,
                                           int32_t code, long long* acc = nullptr, uint32_t sleep_ns = 64) {
#ifdef IM2WIN_PROF
  // try_wait may block inside the instruction, so the clock brackets the first poll too
  const long long c0 = clock64();
  struct Fin { long long* a; long long c; __device__ ~Fin() { if (a) *a += clock64() - c; } } fin{acc, c0};
#endif
  if (ptx::mbar_try_wait(b, parity)) return true;
  return wait_bar_slow(P.status, misc, b, parity, code, sleep_ns);
}

__device__ __forceinline__ bool wait_bar(const PParams& P, PMisc* misc, uint64_t* bar, uint32_t parity,
                                         int32_t code, long long* acc = nullptr, uint32_t sleep_ns = 64) {
  return wait_bar_a(P, misc, ptx::smem_u32(bar), parity, code, acc, sleep_ns);
}

__device__ __forceinline__ bool wait_bar_warp(const PParams& P, PMisc* misc, uint64_t* bar, uint32_t parity,
                                              int32_t code, long long* acc = nullptr, uint32_t sleep_ns = 64) {
  return __all_sync(0xffffffffu, wait_bar(P, misc, bar, parity, code, acc, sleep_ns));
}

__device__ __forceinline__ bool wait_bar_warp_a(const PParams& P, PMisc* misc, uint32_t b, uint32_t parity,
                                                int32_t code, long long* acc = nullptr, uint32_t sleep_ns = 64) {
  return __all_sync(0xffffffffu, wait_bar_a(P, misc, b, parity, code, acc, sleep_ns));
}

// 32-bit load from a shared-space byte address (kept in program order with the waits and the
// tcgen05 stores around it)
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
  uint32_t v;
  asm volatile("{\n.reg .b16 h;\nld.shared.u16 h, [%1];\ncvt.u32.u16 %0, h;\n}" : "=r"(v) : "r"(a) : "memory");
  return v;
}
// two 16-bit loads packed into one register (low half = first address)
__device__ __forceinline__ uint32_t lds_u16x2(uint32_t a_lo, uint32_t a_hi) {
  uint32_t v;
  asm volatile("{\n.reg .b16 l, h;\nld.shared.u16 l, [%1];\nld.shared.u16 h, [%2];\nmov.b32 %0, {l, h};\n}"
               : "=r"(v) : "r"(a_lo), "r"(a_hi) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}

// Position in a ring of n stages together with the parity of the pass over it.
struct Ring {
  int32_t idx = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void advance(int32_t n) {
    if (++idx == n) { idx = 0; phase ^= 1u; }
  }
};
// A group's S MMA steps are handed over in PARTS slots.  With a resident filter, short groups (up
// to 10 steps) use slots of at most 5 steps (40 TMEM columns): small slots let three repack sets
// own two or more slots each, so that a set never waits for the MMAs of the part it has just
// handed over.  Otherwise slots hold up to 13 steps (104 columns), which keeps the number of
// hand-overs per group low for the single MMA-issuing thread of the streamed-filter mode.
template <int S, bool BRES>
struct SlotGeom {
  static constexpr int MAXS = (BRES && S <= 10) ? 5 : 13;
  static constexpr int PARTS = (S + MAXS - 1) / MAXS;
  static constexpr int SLOT_STEPS = (S + PARTS - 1) / PARTS;
};

// n / d for the divisors with a precomputed magic (exact while n * d < 2^32: checked on the host)
__device__ __forceinline__ int32_t fast_div(int32_t n, uint64_t magic) {
  return (int32_t)(((uint64_t)(uint32_t)n * magic) >> 32);
}

// Work unit t = (m-tile, n-tile, reduction slice), the slice fastest (usually one n-tile, one slice).
__device__ __forceinline__ int32_t tile_of(const PParams& P, int32_t t) {
  return P.usub == 1 ? t : t / P.usub;
}
// n-tile and first / one-past-last channel group of unit t
__device__ __forceinline__ void unit_range(const PParams& P, int32_t t, int32_t& nt, int32_t& g0, int32_t& g1) {
  if (__builtin_expect(P.usub == 1, 1)) { nt = 0; g0 = 0; g1 = P.NG; return; }
  const int32_t sub = t - (t / P.usub) * P.usub;
  nt = P.Z == 1 ? sub : sub / P.Z;
  const int32_t z = sub - nt * P.Z;
  g0 = z * P.GZ;
  g1 = min(g0 + P.GZ, P.NG);
}

// Where an m-tile lies: image of its first position, that position's index inside the image, how
// many positions it has, how many images it touches.  One 64-bit division per tile at most; all
// other per-tile arithmetic is 32-bit (a tile holds at most 128 positions and 8 images).
struct TileInfo {
  int64_t i_first;
  int32_t q_first, npos, nseg;
};

// Tiles that may span images (small images).  Out of line: the per-image case below is the hot one.
__device__ __noinline__ TileInfo tile_info_general(int32_t TP, int32_t HoWo, int64_t Mtot, int32_t tile_m) {
  TileInfo ti;
  if (Mtot <= 0x7fffffff) {  // the usual case: 32-bit arithmetic throughout
    const uint32_t P0 = (uint32_t)tile_m * (uint32_t)TP;
    const uint32_t i = P0 / (uint32_t)HoWo;
    ti.i_first = i;
    ti.q_first = (int32_t)(P0 - i * (uint32_t)HoWo);
    ti.npos = min(TP, (int32_t)((uint32_t)Mtot - P0));
    ti.nseg = (ti.q_first + ti.npos - 1) / HoWo + 1;
  } else {
    const int64_t P0 = (int64_t)tile_m * TP;
    ti.i_first = P0 / HoWo;
    ti.q_first = (int32_t)(P0 - ti.i_first * HoWo);
    ti.npos = (int32_t)min((int64_t)TP, Mtot - P0);
    ti.nseg = (ti.q_first + ti.npos - 1) / HoWo + 1;
  }
  return ti;
}

__device__ __forceinline__ TileInfo tile_info(const PParams& P, int32_t tile_m) {
  if (__builtin_expect(P.pim, 1)) {  // tiles are cut per image
    TileInfo ti;
    const int32_t i = fast_div(tile_m, P.magic_TPI);
    ti.i_first = i;
    ti.q_first = (tile_m - i * P.TPI) * P.TP;
    ti.npos = min(P.TP, P.HoWo - ti.q_first);
    ti.nseg = 1;
    return ti;
  }
  return tile_info_general(P.TP, P.HoWo, P.Mtot, tile_m);
}

// Row p of the tile: image (as an offset from the tile's first image) and position inside it.
__device__ __forceinline__ void tile_row(const PParams& P, const TileInfo& ti, int32_t p, int32_t& i_off, int32_t& q) {
  q = ti.q_first + p;
  i_off = 0;
  while (q >= P.HoWo) { q -= P.HoWo; ++i_off; }
}

// Lanes 0..nseg-1 each describe one image segment of the tile; dst_off is the exclusive prefix sum
// of the slot sizes.  Must be called by a converged warp.
__device__ __forceinline__ SegR compute_seg(const PParams& P, const TileInfo& ti, int lane) {
  SegR s{0, 0, 0, 0};
  int32_t slot = 0;
  if (lane < ti.nseg) {
    const int32_t qa = lane == 0 ? ti.q_first : 0;
    const int32_t qb = min(ti.q_first + ti.npos - 1 - lane * P.HoWo, P.HoWo - 1);
    const int32_t m_a = qa / P.Wo, n_a = qa - m_a * P.Wo;
    const int32_t m_b = qb / P.Wo, n_b = qb - m_b * P.Wo;
    s.virt_a = (int64_t)m_a * P.row_mul + (int64_t)n_a * P.col_mul;
    s.start0 = ((ti.i_first + lane) * P.C) * P.plane + s.virt_a;
    s.len = (int32_t)(((int64_t)m_b * P.row_mul + (int64_t)n_b * P.col_mul) - s.virt_a) + P.win_span;
    slot = (s.len + 6) & ~3;
  }
  int32_t incl = slot;
#pragma unroll
  for (int d = 1; d < kSegMax; d <<= 1) {
    const int32_t t = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += t;
  }
  s.dst_off = incl - slot;
  return s;
}

// Repack warps, tiles that may span images: where lane's window starts in a staged channel row, and
// the 16-byte phase of the staged range.  (Kept inline: an out-of-line copy would take the kernel
// parameters by address, which turns every later read of them into a memory load.)
__device__ __forceinline__ void repack_prologue_general(const PParams& P, const TileInfo& ti, int32_t p, int lane,
                                                     bool valid, int32_t& base_off, int32_t& skew0) {
  const SegR seg = compute_seg(P, ti, lane);
  int32_t sg = 0, q = 0;
  if (valid) tile_row(P, ti, p, sg, q);
  const int64_t s_start0 = __shfl_sync(0xffffffffu, seg.start0, sg);
  const int64_t s_virt = __shfl_sync(0xffffffffu, seg.virt_a, sg);
  const int32_t s_dst = __shfl_sync(0xffffffffu, seg.dst_off, sg);
  base_off = 0;
  if (valid) {
    const int32_t m = q / P.Wo, n = q - m * P.Wo;
    base_off = s_dst + (int32_t)(((int64_t)m * P.row_mul + (int64_t)n * P.col_mul) - s_virt);
  }
  skew0 = (int32_t)(s_start0 & 3);  // 16-byte phase of the staged range, per absolute address
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Ask for a box to be brought into L2 (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int32_t c0, int32_t c1) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(c0), "r"(c1) : "memory");
}

template <int FH, int FW, int CB, bool BF16, bool BRES, bool FUSED, bool SRC16, bool OUT16>
__global__ void __launch_bounds__(kThreads, 1)
conv_tc_persistent_kernel(const PParams P, const __grid_constant__ CUtensorMap fmap,
                          const __grid_constant__ CUtensorMap xmap) {
  constexpr int FF = FH * FW;
  // SRC16: the staged source is an im2win tensor stored as bf16 (per-image tiling only; BF16 mode).
  // Source lengths and offsets are in elements; ES bytes each, EPC elements per 16-byte chunk.
  static_assert(!SRC16 || (BF16 && !FUSED), "a 16-bit source is an im2win tensor consumed in BF16 mode");
  constexpr uint32_t ES = SRC16 ? 2u : 4u;
  constexpr int32_t EPC = SRC16 ? 8 : 4;
  constexpr int KSTEP = BF16 ? 16 : 8;        // reduction elements per MMA
  constexpr int KCHUNK = BF16 ? 64 : 32;      // reduction elements per 128-byte filter row
  constexpr int KCG = CB * FF;                // real reduction elements per channel group
  constexpr int KCGP = (KCG + KSTEP - 1) / KSTEP * KSTEP;
  constexpr int S = KCGP / KSTEP;             // MMA steps per channel group
  constexpr int PARTS = SlotGeom<S, BRES>::PARTS;   // a group's A columns go to TMEM in PARTS slots
  constexpr int SLOT_STEPS = SlotGeom<S, BRES>::SLOT_STEPS;
  constexpr int SLOT_COLS = SLOT_STEPS * 8;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* const smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* const b_smem = smem;  // resident: nchunks * NT*128 bytes; streamed: SB stages of NT*128 bytes
  float* const raw = reinterpret_cast<float*>(smem + P.off_raw);
  const float* const zero_pad = reinterpret_cast<const float*>(smem + P.off_zero);  // win_span + 8 zeros
  PBars* const bars = reinterpret_cast<PBars*>(smem + P.off_bar);
  PMisc* const misc = reinterpret_cast<PMisc*>(smem + P.off_misc);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int32_t raw_stage_floats = CB * P.chan_pitch;  // source elements per strip stage
  using SrcT = typename std::conditional<SRC16, uint16_t, float>::type;
  const SrcT* const xsrc = reinterpret_cast<const SrcT*>(P.xhat);
  const uint32_t raw_sa = ptx::smem_u32(raw);
  (void)xsrc; (void)raw_sa;
  const uint32_t b_stage_bytes = (uint32_t)P.NT * 128u;
#ifdef IM2WIN_PROF
  const long long prof_kernel_t0 = clock64();
  if (P.prof && threadIdx.x == 0) { P.prof[512 + blockIdx.x * 4] = (long long)global_ns(); P.prof[512 + blockIdx.x * 4 + 2] = prof_kernel_t0; }
#endif

  // ------------------------------------------------------------------ prologue
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->raw_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->raw_empty[i]), 4);
      ptx::mbar_init(ptx::smem_u32(&bars->b_full[i]), (BRES && i == 0 && !P.b_tma) ? kThreads - 32 : 1);
      ptx::mbar_init(ptx::smem_u32(&bars->b_empty[i]), BRES ? 1 : 2);  // streamed: both issuers release a stage
    }
    for (int i = 0; i < kMaxSub; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->a_full[i]), 4);
      ptx::mbar_init(ptx::smem_u32(&bars->a_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[i]), BRES ? P.NSETS : 2);  // one commit per MMA-issuing thread
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[i]), 4);
    }
    ptx::fence_mbar_init();
    misc->abort = 0;
  }
  for (int32_t i = threadIdx.x; i < P.win_span + 8; i += kThreads) reinterpret_cast<float*>(smem + P.off_zero)[i] = 0.f;
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), (uint32_t)P.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // Slice-resident mode: the grid is a multiple of the number of reduction slices, so every unit of
  // this CTA (t = blockIdx.x + k * gridDim.x) belongs to the same slice, and only that slice's part
  // of the filter is kept in shared memory.
  int32_t bs_g0 = 0, bs_ng = P.NG;
  if constexpr (BRES) {
    if (P.bslice) {
      int32_t nt_b, gb0, gb1;
      unit_range(P, (int32_t)blockIdx.x, nt_b, gb0, gb1);
      (void)nt_b;
      bs_g0 = gb0; bs_ng = gb1 - gb0;
    }
  }
  const int32_t bs_step0 = bs_g0 * S;  // first MMA step held in the resident filter
  if constexpr (BRES) {
    // Build the whole filter operand once, one block of NT rows x 32 bytes per MMA step (padded
    // reduction indices [s*KSTEP, +KSTEP)), K-major with the 32-byte swizzle, so that the MMA thread
    // steps its descriptor by a constant.  (A resident filter implies one n-tile.)  Every warp but
    // the strip producer takes part; the producer already fetches strips meanwhile, and only the
    // MMA thread waits for the build to be complete.
    if (P.b_tma) {
      // TF32 with dense groups: the operand is the native filter itself, so one TMA box per MMA step
      // (NT rows x 32 bytes, 32-byte swizzle) lays it out; the lanes of the otherwise idle warp 2
      // issue them, and no thread waits except the MMA issuers.
      if (warp == 2) {
        const int32_t nsteps_all = bs_ng * S;
        const uint32_t full = ptx::smem_u32(&bars->b_full[0]);
        if (lane == 0) ptx::mbar_arrive_expect_tx(full, (uint32_t)nsteps_all * (uint32_t)P.NT * 32u);
        __syncwarp();
        for (int32_t st = lane; st < nsteps_all; st += 32)
          tma_load_2d(ptx::smem_u32(b_smem) + (uint32_t)st * (uint32_t)P.NT * 32u, &fmap, (bs_step0 + st) * KSTEP, 0, full);
      }
    } else if (warp != 0) {
      constexpr int EPP = BF16 ? 8 : 4;  // elements per 16-byte piece
      const int32_t nsteps_all = bs_ng * S;
      const int32_t pieces = nsteps_all * P.NT * 2;
      const uint32_t step_bytes = (uint32_t)P.NT * 32u;
      const bool vec = (KCG == KCGP) && (P.Kg % 4) == 0;  // padded index == real index, rows 16-byte aligned
      // piece index = [row / 8][step][row % 8][16-byte half]: 16 consecutive threads fill one
      // contiguous 256-byte swizzle atom in shared memory and read 8 sector-sized runs of the filter
      // Four pieces per thread and trip: all loads of a trip are issued before the first store, so
      // that a thread has four requests in flight (every CTA reads the same filter at the same
      // time, and a trip costs one L2 round trip under that load).
      constexpr int U = 4;
      for (int32_t base = (int32_t)threadIdx.x - 32; base < pieces; base += U * (kThreads - 32)) {
        float x[U][8];
        int32_t dst[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int32_t idx = base + u * (kThreads - 32);
          dst[u] = -1;
          if (idx < pieces) {
            const int32_t c = idx & 1, jl = (idx >> 1) & 7;
            const int32_t rest = idx >> 4;
            const int32_t jb = rest / nsteps_all;
            const int32_t sidx = rest - jb * nsteps_all, j = jb * 8 + jl;
            const int32_t kp0 = (bs_step0 + sidx) * KSTEP + c * EPP;
            dst[u] = sidx * (int32_t)step_bytes + (j >> 3) * 256 + (j & 7) * 32 + ((c ^ ((j >> 2) & 1)) << 4);
            if (vec && j < P.K && kp0 + EPP <= P.Kg) {
              const float4 a = __ldg(reinterpret_cast<const float4*>(P.f + (int64_t)j * P.Kg + kp0));
              x[u][0] = a.x; x[u][1] = a.y; x[u][2] = a.z; x[u][3] = a.w;
              if (EPP == 8) {
                const float4 b = __ldg(reinterpret_cast<const float4*>(P.f + (int64_t)j * P.Kg + kp0 + 4));
                x[u][4] = b.x; x[u][5] = b.y; x[u][6] = b.z; x[u][7] = b.w;
              }
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                x[u][e] = 0.f;
                if (e < EPP && j < P.K) {
                  const int32_t kp = kp0 + e;
                  const int32_t g = kp / KCGP, kl = kp - g * KCGP;
                  const int64_t k = (int64_t)g * KCG + kl;
                  if (kl < KCG && k < P.Kg) x[u][e] = __ldg(P.f + (int64_t)j * P.Kg + k);
                }
              }
            }
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (dst[u] >= 0) {
            uint4 piece;
            if (BF16) {
              piece.x = ptx::pack_bf16x2(x[u][0], x[u][1]); piece.y = ptx::pack_bf16x2(x[u][2], x[u][3]);
              piece.z = ptx::pack_bf16x2(x[u][4], x[u][5]); piece.w = ptx::pack_bf16x2(x[u][6], x[u][7]);
            } else {
              piece.x = __float_as_uint(x[u][0]); piece.y = __float_as_uint(x[u][1]);
              piece.z = __float_as_uint(x[u][2]); piece.w = __float_as_uint(x[u][3]);
            }
            *reinterpret_cast<uint4*>(b_smem + dst[u]) = piece;
          }
        }
      }
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(ptx::smem_u32(&bars->b_full[0]));  // resident mode: b_full[0] = "filter built"
    }
  }
  const uint32_t tmem_base = misc->tmem_base;
  const uint32_t tmem_a0 = tmem_base + (uint32_t)(P.ND * P.NT);

  if (warp == 0) {
    // ================================================================ STRIP PRODUCER
    Ring rr;             // raw stage being filled
    int64_t gcount = 0;  // channel groups issued so far (all tiles)
    bool ok = true;
    PROF_DECL(2)
#ifdef IM2WIN_PROF
    prof_acc[1] = prof_t0 - prof_kernel_t0;  // prologue (barrier init, TMEM alloc, resident filter build)
#endif
    // The kernel is launched as a programmatic dependent of whatever precedes it in the stream: where that is
    // the transform kernel (which lets its dependents start while it drains), the prologue above overlapped
    // its tail, and the source is read only once that grid has completed.  After any other kernel: no effect.
    // (Behind this call's own filter-copy kernel, an ordinary launch, everything earlier has completed already.)
    if (P.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (P.box) {
      // One 2-D box per channel group.  The tile lies in one image: x = first needed float of the
      // plane rounded down to 16 bytes (in 8-byte elements), y = plane index of the group's first
      // channel.  Nothing else is needed per tile, and only one lane works.
      // The boxes of this CTA's next tile are requested into L2 one tile ahead, group by group, so
      // that the copies into the few shared-memory stages later meet L2 latency, not DRAM's.
      for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x) {
        const int32_t tile_m = tile_of(P, t);
        const int32_t i = fast_div(tile_m, P.magic_TPI);
        const int32_t q_first = (tile_m - i * P.TPI) * P.TP;
        const int32_t m_a = fast_div(q_first, P.magic_Wo), n_a = q_first - m_a * P.Wo;
        const int32_t box_x = ((m_a * P.row_mul + n_a * P.col_mul) & ~(EPC - 1)) / (EPC / 2);  // in 8-byte units
        const int32_t box_y0 = i * P.C;
        const int32_t tn = t + (int32_t)gridDim.x;
        const bool pf = P.l2_ahead && tn < (int32_t)P.ntiles;
        int32_t pf_x = 0, pf_y0 = 0;
        if (pf) {
          const int32_t tm2 = tile_of(P, tn);
          const int32_t i2 = fast_div(tm2, P.magic_TPI);
          const int32_t q2 = (tm2 - i2 * P.TPI) * P.TP;
          const int32_t m2 = fast_div(q2, P.magic_Wo), n2 = q2 - m2 * P.Wo;
          pf_x = ((m2 * P.row_mul + n2 * P.col_mul) & ~(EPC - 1)) / (EPC / 2);
          pf_y0 = i2 * P.C;
        }
        int32_t nt_, g0, g1;
        unit_range(P, t, nt_, g0, g1);
        (void)nt_;
        for (int32_t g = g0; g < g1 && ok; ++g, ++gcount, rr.advance(P.SR)) {
          const int32_t sr = rr.idx;
          if (pf && lane == 0) tma_prefetch_2d(&xmap, pf_x, pf_y0 + g * CB);
          ok = wait_bar_warp(P, misc, &bars->raw_empty[sr], rr.phase ^ 1u, DEV_TIMEOUT_RAW_EMPTY, PROF_SLOT(0), 128);
          if (!ok) break;
          if (lane == 0) {
            const uint32_t full = ptx::smem_u32(&bars->raw_full[sr]);
            ptx::mbar_arrive_expect_tx(full, (uint32_t)raw_stage_floats * ES);
            tma_load_2d(raw_sa + (uint32_t)(sr * raw_stage_floats) * ES, &xmap, box_x, box_y0 + g * CB, full);
          }
          __syncwarp();
        }
      }
    } else if (P.pim) {
      // Tiles cut per image, strips by bulk copies: lane rl < CB copies the one contiguous range of
      // channel rl that the tile needs; from group to group only the plane moves.
      const int64_t group_step = (int64_t)CB * P.plane;
      for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x) {
        const int32_t tile_m = tile_of(P, t);
        const int32_t i = fast_div(tile_m, P.magic_TPI);
        const int32_t q_first = (tile_m - i * P.TPI) * P.TP;
        const int32_t q_last = min(q_first + P.TP, P.HoWo) - 1;
        const int32_t m_a = fast_div(q_first, P.magic_Wo), n_a = q_first - m_a * P.Wo;
        const int32_t m_b = fast_div(q_last, P.magic_Wo), n_b = q_last - m_b * P.Wo;
        const int32_t virt_a = m_a * P.row_mul + n_a * P.col_mul;
        const int32_t len = m_b * P.row_mul + n_b * P.col_mul - virt_a + P.win_span;
        int32_t nt_, g0, g1;
        unit_range(P, t, nt_, g0, g1);
        (void)nt_;
        int64_t start = ((int64_t)i * P.C + (int64_t)g0 * CB + lane) * P.plane + virt_a;
        for (int32_t g = g0; g < g1 && ok; ++g, ++gcount, rr.advance(P.SR)) {
          const int32_t sr = rr.idx;
          ok = wait_bar_warp(P, misc, &bars->raw_empty[sr], rr.phase ^ 1u, DEV_TIMEOUT_RAW_EMPTY, PROF_SLOT(0), 128);
          if (!ok) break;
          const uint32_t full = ptx::smem_u32(&bars->raw_full[sr]);
          const SrcT* src = nullptr;
          uint32_t dst = 0, bytes = 0;
          if (lane < CB && g * CB + lane < P.C) {
            const int32_t skew = (int32_t)(start & (EPC - 1));
            const int64_t a0 = start - skew;
            int32_t nfl = (skew + len + EPC - 1) & ~(EPC - 1);
            SrcT* d = reinterpret_cast<SrcT*>(raw) + (size_t)sr * raw_stage_floats + lane * P.chan_pitch;
            if (a0 + nfl > P.n_src) {  // the last 16-byte chunk would pass the end of the tensor
              const int32_t nbulk = (int32_t)((P.n_src - a0) & ~(int64_t)(EPC - 1));
              for (int64_t e = a0 + nbulk; e < P.n_src; ++e) d[e - a0] = __ldg(xsrc + e);
              nfl = nbulk;
            }
            src = xsrc + a0;
            dst = ptx::smem_u32(d);
            bytes = (uint32_t)nfl * ES;
          }
          start += group_step;
          const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
          if (lane == 0) ptx::mbar_arrive_expect_tx(full, total);
          __syncwarp();
          if (bytes) ptx::bulk_g2s(dst, src, bytes, full);
        }
      }
    } else if constexpr (!SRC16) {
      for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x) {
        const TileInfo ti = tile_info(P, tile_of(P, t));
        const int32_t nseg = ti.nseg;
        const SegR seg = compute_seg(P, ti, lane);
        // Each lane owns up to two (channel-in-group, image segment) pairs for the whole tile; from
        // group to group only the channel, i.e. the source address, moves (by CB planes).
        const int32_t npairs = CB * nseg;  // <= 64
        bool act[2];
        int32_t rl[2], len[2], dsto[2];
        int64_t start[2];
#pragma unroll
        for (int z = 0; z < 2; ++z) {
          const int32_t idx = z * 32 + lane;
          act[z] = idx < npairs;
          rl[z] = act[z] ? idx / nseg : 0;
          const int32_t sg = act[z] ? idx - rl[z] * nseg : 0;
          const int64_t s_start0 = __shfl_sync(0xffffffffu, seg.start0, sg);
          len[z] = __shfl_sync(0xffffffffu, seg.len, sg);
          dsto[z] = rl[z] * P.chan_pitch + __shfl_sync(0xffffffffu, seg.dst_off, sg);
          start[z] = s_start0 + (int64_t)rl[z] * P.plane;
        }
        const int64_t group_step = (int64_t)CB * P.plane;
        int32_t nt_, g0, g1;
        unit_range(P, t, nt_, g0, g1);
        (void)nt_;
        start[0] += g0 * group_step;
        start[1] += g0 * group_step;
        for (int32_t g = g0; g < g1 && ok; ++g, ++gcount, rr.advance(P.SR)) {
          const int32_t sr = rr.idx;
          ok = wait_bar_warp(P, misc, &bars->raw_empty[sr], rr.phase ^ 1u, DEV_TIMEOUT_RAW_EMPTY, PROF_SLOT(0), 128);
          if (!ok) break;
          const uint32_t full = ptx::smem_u32(&bars->raw_full[sr]);
          float* stage = raw + (size_t)sr * raw_stage_floats;
          const float* src[2];
          uint32_t dst[2], bytes[2];
#pragma unroll
          for (int z = 0; z < 2; ++z) {
            bytes[z] = 0;
            if (act[z] && g * CB + rl[z] < P.C) {
              const int32_t skew = (int32_t)(start[z] & 3);
              const int64_t a0 = start[z] - skew;
              int32_t nfl = (skew + len[z] + 3) & ~3;
              float* d = stage + dsto[z];
              if (a0 + nfl > P.n_src) {  // the last 16-byte chunk would pass the end of the tensor
                const int32_t nbulk = (int32_t)((P.n_src - a0) & ~(int64_t)3);
                for (int64_t e = a0 + nbulk; e < P.n_src; ++e) d[e - a0] = __ldg(xsrc + e);
                nfl = nbulk;
              }
              src[z] = xsrc + a0;
              dst[z] = ptx::smem_u32(d);
              bytes[z] = (uint32_t)nfl * 4u;
            }
            start[z] += group_step;
          }
          // one arrival carrying the byte count of the whole group, then the copies
          const uint32_t total = __reduce_add_sync(0xffffffffu, bytes[0] + bytes[1]);
          if (lane == 0) ptx::mbar_arrive_expect_tx(full, total);
          __syncwarp();
#pragma unroll
          for (int z = 0; z < 2; ++z)
            if (bytes[z]) ptx::bulk_g2s(dst[z], src[z], bytes[z], full);
        }
      }
    }
    PROF_DUMP(0, 2)
    // every copy issued must have landed before the CTA exits
    for (int64_t g = max(gcount - P.SR, (int64_t)0); g < gcount; ++g)
      wait_bar(P, misc, &bars->raw_full[g % P.SR], (uint32_t)(g / P.SR) & 1u, DEV_TIMEOUT_DRAIN);
  } else if (warp == 1 || (BRES && warp >= 2 && warp <= P.NSETS) || (!BRES && warp == 3)) {
    // ================================================================ MMA ISSUER(S)
    // The loop body per MMA is kept to a handful of instructions because a single thread can only
    // issue a tcgen05.mma every few tens of cycles -- more than a narrow (N = 64) MMA takes to run.
    // With a resident filter nothing orders the groups of a tile among themselves (every MMA
    // accumulates onto an accumulator the epilogue has zeroed), so one thread per repack set, in
    // warps 1, 2, (3), issues the groups that set produced.  With a streamed filter two threads (warps
    // 1 and 3; warp 2 feeds the filter ring) share the groups by the parity of the producing set; both
    // walk every filter stage in order -- each waits for a stage when it passes its first step and
    // releases it when it passes its last, also across groups it does not issue, so that every stage
    // barrier sees both of them in every phase.
    const uint32_t me = BRES ? (uint32_t)(warp - 1) : (warp == 3 ? 1u : 0u);
    (void)me;
    // The whole warp runs the role and lane 0 issues: the descriptor arithmetic and the waits are then warp-uniform
    // work (4-7 % on the TF32 layers, whose narrow MMAs the issue rate bounds).  Two families keep the one-thread
    // form, measured slower with it: the 7x7 three-channel stems in TF32 mode from the im2win tensor (7 %), and
    // streamed filters other than 3x3 (the 5x5 layers: 18-22 %).
    constexpr bool WARP_ISSUE = (BRES || FH == 3) && !(FH == 7 && CB == 3 && !BF16 && !FUSED);
    if (WARP_ISSUE || lane == 0) {
      const uint32_t elect = lane == 0 ? 1u : 0u;
      auto wait_role = [&](uint64_t* bar, uint32_t parity, int32_t code, long long* acc, uint32_t sleep_ns) -> bool {
        if constexpr (WARP_ISSUE) return wait_bar_warp(P, misc, bar, parity, code, acc, sleep_ns);
        else return wait_bar(P, misc, bar, parity, code, acc, sleep_ns);
      };
      auto poll_role = [&](uint32_t bar_addr, uint32_t parity) -> bool {
        const bool r = ptx::mbar_try_wait(bar_addr, parity);
        if constexpr (WARP_ISSUE) return __all_sync(0xffffffffu, r);
        else return r;
      };
      Ring ar0, ar1, ar2, br, dr;  // A slot (one ring per repack set), streamed filter stage, accumulator buffer
      uint32_t gset = 0;    // running group count modulo the number of sets = which set produced the group
      const uint32_t nsets = (uint32_t)P.NSETS;
      bool ok = true;
      PROF_DECL(7)
      const uint64_t desc0 = BRES ? ptx::smem_desc_k_sw32(ptx::smem_u32(b_smem)) : ptx::smem_desc_k_sw128(ptx::smem_u32(b_smem));
      const uint32_t desc_lo0 = (uint32_t)desc0, desc_hi = (uint32_t)(desc0 >> 32);
      const uint32_t step16 = (uint32_t)P.NT * 2u;  // resident: one step block (NT*32 bytes) in descriptor units
      uint32_t step_off[SLOT_STEPS];                // resident: j * step16, kept in registers
#pragma unroll
      for (int j = 0; j < SLOT_STEPS; ++j) step_off[j] = (uint32_t)j * step16;
      const uint32_t chunk16 = b_stage_bytes >> 4;  // one filter chunk / stage in descriptor units
      const uint32_t a_full0 = ptx::smem_u32(&bars->a_full[0]), a_empty0 = ptx::smem_u32(&bars->a_empty[0]);
      const uint32_t b_full0 = ptx::smem_u32(&bars->b_full[0]), b_empty0 = ptx::smem_u32(&bars->b_empty[0]);
      (void)b_full0; (void)b_empty0;
      if constexpr (BRES) ok = wait_role(&bars->b_full[0], 0u, DEV_TIMEOUT_B_FULL, PROF_SLOT(1), 64);
      for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x, dr.advance(P.ND)) {
        const int32_t d = dr.idx;
        // the epilogue hands the buffer over zeroed (also before its first use)
        ok = wait_role(&bars->acc_empty[d], dr.phase, DEV_TIMEOUT_ACC, PROF_SLOT(2), 64);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(d * P.NT);
        const uint32_t accum = 1;
        int32_t nt_, g0, g1;
        unit_range(P, t, nt_, g0, g1);
        (void)nt_;
        uint32_t st0 = (uint32_t)(g0 * S - (BRES ? bs_step0 : 0));  // steps before the current part (resident: of the held filter)
        uint32_t b_lo = desc_lo0;           // streamed: descriptor of the current stage
        for (int32_t g = g0; g < g1 && ok; ++g, gset = (gset + 1u == nsets) ? 0u : gset + 1u) {
          if constexpr (BRES) {
            if (gset != me) { st0 += S; continue; }  // another issuer's group
          } else {
            if ((gset & 1u) != me) {
              // the other issuer's group: pass the filter stages that begin or end inside it
              const uint32_t end = st0 + S;
              uint32_t st = st0;
              while (true) {
                if ((st & 3u) == 0) {
                  ok = wait_role(&bars->b_full[br.idx], br.phase, DEV_TIMEOUT_B_FULL, nullptr, 20);
                  if (!ok) break;
                }
                const uint32_t last = st | 3u;  // last step of the stage that holds step st
                if (last >= end) break;         // the stage runs on into the next group
                ptx::mma_commit_if(b_empty0 + (uint32_t)br.idx * 8u, elect);
                br.advance(P.SB);
                st = last + 1u;
                if (st >= end) break;
              }
              st0 = end;
              continue;
            }
            b_lo = desc_lo0 + (uint32_t)br.idx * chunk16;  // (the group may begin inside a stage)
          }
          // the ring of the set that produced this group, held in registers (no indexed array)
          Ring ar = gset == 0 ? ar0 : (gset == 1 ? ar1 : ar2);
          const int32_t slot0 = (int32_t)gset * P.NSS;
#pragma unroll
          for (int h = 0; h < PARTS; ++h) {
            const int nst = (h == PARTS - 1) ? (S - (PARTS - 1) * SLOT_STEPS) : SLOT_STEPS;
            const int32_t slot = slot0 + ar.idx;
            if (!poll_role(a_full0 + (uint32_t)slot * 8u, ar.phase)) {  // usually ready: one poll
              ok = wait_role(&bars->a_full[slot], ar.phase, DEV_TIMEOUT_A_FULL, PROF_SLOT(0), 20);
              if (!ok) break;
            }
            PROF_T0(tf)
            ptx::tc_fence_after();
            PROF_ADD(3, tf)
            const uint32_t a_addr = tmem_a0 + (uint32_t)(slot * SLOT_COLS);
            const uint32_t lo_part = desc_lo0 + st0 * step16;
            (void)lo_part;
            PROF_T0(tm)
#pragma unroll
            for (int j = 0; j < SLOT_STEPS; ++j) {
              if (j < nst) {
                const uint32_t st = st0 + j;  // step within the tile: chunk st >> 2, quarter st & 3
                uint32_t lo;
                if constexpr (BRES) {
                  lo = lo_part + step_off[j];  // one add per MMA, no chain from step to step
                } else {
                  if ((st & 3u) == 0) {
                    if (!poll_role(b_full0 + (uint32_t)br.idx * 8u, br.phase)) {
                      ok = wait_role(&bars->b_full[br.idx], br.phase, DEV_TIMEOUT_B_FULL, PROF_SLOT(1), 20);
                      if (!ok) break;
                    }
                    ptx::tc_fence_after();
                    b_lo = desc_lo0 + (uint32_t)br.idx * chunk16;
                  }
                  lo = b_lo + (st & 3u) * 2u;
                }
                ptx::mma_ts_lohi_if<BF16>(d_tmem, a_addr + j * 8, lo, desc_hi, P.idesc, accum, elect);
                if constexpr (!BRES) {
                  if ((st & 3u) == 3u) { ptx::mma_commit_if(b_empty0 + (uint32_t)br.idx * 8u, elect); br.advance(P.SB); }
                }
              }
            }
            if (!ok) break;
            PROF_ADD(4, tm)
            st0 += nst;
            PROF_T0(tc)
            ptx::mma_commit_if(a_empty0 + (uint32_t)slot * 8u, elect);
            PROF_ADD(5, tc)
            ar.advance(P.NSS);
          }
          if (gset == 0) ar0 = ar; else if (gset == 1) ar1 = ar; else ar2 = ar;
        }
        if (!ok) break;
        if constexpr (!BRES) {
          if ((st0 & 3u) != 0) { ptx::mma_commit_if(ptx::smem_u32(&bars->b_empty[br.idx]), elect); br.advance(P.SB); }
        }
        ptx::mma_commit_if(ptx::smem_u32(&bars->acc_full[d]), elect);
      }
      if (me == 0 && lane == 0) { PROF_DUMP(1, 7) }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ================================================================ FILTER PRODUCER (streamed mode)
    // (with a resident filter this warp is an MMA issuer, and the copies it issued in the prologue
    // have landed before its first MMA)
    if constexpr (!BRES) {
      if (lane == 0) {
        PROF_DECL(2)
        int64_t bcount = 0;
        Ring br;
        bool ok = true;
        // BF16 mode: the bf16 copy of the filter is written by the kernel launched just before this one,
        // which this kernel may overlap (programmatic dependent launch); without such a launch: no effect
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x) {
          int32_t nt, g0, g1;
          unit_range(P, t, nt, g0, g1);
          const int32_t n0 = nt * P.NT;
          // the slice's 128-byte filter chunks (a slice starts on a chunk boundary: host check)
          const int32_t c0 = (g0 * S) >> 2, c1 = (g1 * S + 3) >> 2;
          for (int32_t c = c0; c < c1 && ok; ++c, ++bcount, br.advance(P.SB)) {
            const int32_t sb = br.idx;
            ok = wait_bar(P, misc, &bars->b_empty[sb], br.phase ^ 1u, DEV_TIMEOUT_B_EMPTY, PROF_SLOT(0));
            if (!ok) break;
            const uint32_t full = ptx::smem_u32(&bars->b_full[sb]);
            ptx::mbar_expect_tx(full, b_stage_bytes);
            tma_load_2d(ptx::smem_u32(b_smem) + (uint32_t)sb * b_stage_bytes, &fmap, c * KCHUNK, n0, full);
            ptx::mbar_arrive(full);
          }
        }
        for (int64_t c = max(bcount - P.SB, (int64_t)0); c < bcount; ++c)
          wait_bar(P, misc, &bars->b_full[c % P.SB], (uint32_t)(c / P.SB) & 1u, DEV_TIMEOUT_DRAIN);
        PROF_DUMP(7, 1)
      }
      __syncwarp();
    }
  } else if (warp >= kRepackWarp0 && warp < kRepackWarp0 + 4 * P.NSETS) {
    // ================================================================ WINDOW REPACK: strips -> TMEM (A)
    // Sets of four warps (one per TMEM lane quarter); the sets take channel groups in turn.
    const int32_t set = (warp - kRepackWarp0) >> 2;
    const int32_t q4 = (warp - kRepackWarp0) & 3;
    const int32_t p = q4 * 32 + lane;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    const int32_t skew_step = P.box ? 0 : (int32_t)(P.plane & (EPC - 1));
    Ring rr, ar;      // raw stage of the current group, A slot of the current part (this set's own ring)
    const uint32_t slot0 = (uint32_t)(set * P.NSS);
    const uint32_t raw_a = ptx::smem_u32(raw), zero_a = ptx::smem_u32(zero_pad);
    const uint32_t W4 = (uint32_t)P.W * 4u;
    (void)W4;
    const uint32_t raw_full0 = ptx::smem_u32(&bars->raw_full[0]), raw_empty0 = ptx::smem_u32(&bars->raw_empty[0]);
    const uint32_t a_full0 = ptx::smem_u32(&bars->a_full[0]), a_empty0 = ptx::smem_u32(&bars->a_empty[0]);
    int32_t gset = 0;  // running group count modulo the number of sets
    bool ok = true;
    PROF_DECL(7)
    for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x) {
      PROF_T0(tt)
      const TileInfo ti = tile_info(P, tile_of(P, t));
      const bool valid = p < ti.npos;
      int32_t base_off = 0, skew0 = 0;
      if (P.pim) {
        // one image, one segment: everything follows from the tile's first position
        const int32_t m_a = fast_div(ti.q_first, P.magic_Wo), n_a = ti.q_first - m_a * P.Wo;
        const int32_t virt_a = m_a * P.row_mul + n_a * P.col_mul;  // a plane fits 32 bits (host check)
        if (valid) {
          const int32_t q = ti.q_first + p;
          const int32_t m = fast_div(q, P.magic_Wo), n = q - m * P.Wo;
          // box: the staged range starts at the 16-byte boundary below the first float (same phase
          // in every plane); bulk copies: the phase is per channel, added to the pointers below
          base_off = m * P.row_mul + n * P.col_mul - (P.box ? (virt_a & ~(EPC - 1)) : virt_a);
        }
        if (!P.box) skew0 = (int32_t)((ti.i_first * P.C * P.plane + virt_a) & (EPC - 1));
      } else {
        repack_prologue_general(P, ti, p, lane, valid, base_off, skew0);
      }
      PROF_ADD(2, tt)

      int32_t nt_, g0, g1;
      unit_range(P, t, nt_, g0, g1);
      (void)nt_;
      for (int32_t g = g0; g < g1 && ok; ++g, gset = (gset + 1 == P.NSETS) ? 0 : gset + 1) {
        if (gset != set) {  // another set's group
          rr.advance(P.SR);
          continue;
        }
        const int32_t sr = rr.idx;
        PROF_T0(twhole)
        ok = wait_bar_warp_a(P, misc, raw_full0 + (uint32_t)sr * 8u, rr.phase, DEV_TIMEOUT_RAW_FULL, PROF_SLOT(0));
        if (!ok) break;
        PROF_T0(ts)
        // Shared-space byte address of this lane's window start in each channel of the group.
        // element kl of the group: channel kl / FF, tap (u, v) = ((kl % FF) / FW, (kl % FF) % FW),
        // stored in the strip at offset v*FH + u from the window start
        // (fused source: the raw input rows are staged instead, and tap (u, v) is at u*W + v)
        const int32_t r0 = g * CB;
        const uint32_t stage_a = raw_a + (uint32_t)(sr * raw_stage_floats + base_off) * ES;
        uint32_t ca[CB];
        if (skew_step == 0) {  // every plane starts on a 16-byte boundary: one phase for all channels
#pragma unroll
          for (int rl = 0; rl < CB; ++rl) ca[rl] = stage_a + (uint32_t)(rl * P.chan_pitch + skew0) * ES;
        } else {
#pragma unroll
          for (int rl = 0; rl < CB; ++rl)
            ca[rl] = stage_a + (uint32_t)(rl * P.chan_pitch + ((skew0 + (r0 + rl) * skew_step) & (EPC - 1))) * ES;
        }
        // channels past C (last group of a C that CB does not divide) read as zero: their addresses
        // are parked on a zeroed pad so that the hot loop carries no per-element select
        if (r0 + CB > P.C) {
#pragma unroll
          for (int rl = 0; rl < CB; ++rl)
            if (r0 + rl >= P.C) ca[rl] = zero_a;
        }
        // (16-bit source) shared address of element kl, and a packed pair of consecutive elements
        auto addr16 = [&](int kl) -> uint32_t {
          const int rl = kl / FF, w = kl % FF;
          return ca[rl] + (uint32_t)(((w % FW) * FH + (w / FW)) * 2);
        };
        auto pair16 = [&](int kl) -> uint32_t {
          if (kl >= KCG) return 0u;
          if (kl + 1 >= KCG) return lds_u16(addr16(kl));
          return lds_u16x2(addr16(kl), addr16(kl + 1));
        };
        (void)pair16;
        auto elem = [&](int kl) -> uint32_t {
          if (kl >= KCG) return 0u;
          const int rl = kl / FF, w = kl % FF;
          if constexpr (SRC16) return lds_u16(ca[rl] + (uint32_t)(((w % FW) * FH + (w / FW)) * 2));  // bf16 bits
          else return lds_u32(FUSED ? ca[rl] + (uint32_t)(w / FW) * W4 + (uint32_t)((w % FW) * 4)
                                    : ca[rl] + (uint32_t)(((w % FW) * FH + (w / FW)) * 4));
        };
#pragma unroll
        for (int h = 0; h < PARTS; ++h) {
          const int j0 = h * SLOT_STEPS;                         // first step of this part in the group
          const int nst = (h == PARTS - 1) ? (S - (PARTS - 1) * SLOT_STEPS) : SLOT_STEPS;
          const uint32_t slot = slot0 + (uint32_t)ar.idx;
          if (h == 0) { PROF_ADD(5, ts) }
          PROF_T0(tl)
          // In register batches of at most 7 steps; the first batch's windows are loaded before the
          // slot is waited for (the slot is only needed for the stores).
          constexpr int NB = (SLOT_STEPS + 6) / 7;
          constexpr int BATCH = (SLOT_STEPS + NB - 1) / NB;
          uint32_t a_slot = 0;
#pragma unroll
          for (int b = 0; b < NB; ++b) {
            uint32_t v[BATCH][8];
#pragma unroll
            for (int jj = 0; jj < BATCH; ++jj) {
              const int j = b * BATCH + jj;
              if (j < nst) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  if constexpr (SRC16)  // already bf16: low half = even k
                    v[jj][e] = pair16((j0 + j) * 16 + 2 * e);
                  else if constexpr (BF16)
                    v[jj][e] = ptx::pack_bf16x2(__uint_as_float(elem((j0 + j) * 16 + 2 * e)),
                                                __uint_as_float(elem((j0 + j) * 16 + 2 * e + 1)));
                  else
                    v[jj][e] = elem((j0 + j) * 8 + e);
                }
              }
            }
            if (b == 0) {
              ok = wait_bar_warp_a(P, misc, a_empty0 + slot * 8u, ar.phase ^ 1u, DEV_TIMEOUT_A_EMPTY, PROF_SLOT(1));
              if (!ok) break;
              ptx::tc_fence_after();
              a_slot = tmem_a0 + lane_base + slot * (uint32_t)SLOT_COLS;
            }
#pragma unroll
            for (int jj = 0; jj < BATCH; ++jj) {
              const int j = b * BATCH + jj;
              if (j < nst) ptx::tmem_st_x8(a_slot + (uint32_t)(j * 8), v[jj]);
            }
          }
          if (!ok) break;
          PROF_ADD(3, tl)
          PROF_T0(tw)
          ptx::tmem_wait_st();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            ptx::mbar_arrive(a_full0 + slot * 8u);
            // every lane's loads of the stage are done too (their values went into the stores)
            if (h == PARTS - 1) ptx::mbar_arrive(raw_empty0 + (uint32_t)sr * 8u);
          }
          PROF_ADD(4, tw)
          ar.advance(P.NSS);
        }
        if (!ok) break;
        rr.advance(P.SR);
        PROF_ADD(6, twhole)
      }
    }
    if (set == 0) { PROF_DUMP(2 + q4, 7) }
  } else if (warp >= kEpiWarp0) {
    // ================================================================ EPILOGUE: TMEM -> NCHW
    const int32_t q4 = warp - kEpiWarp0;
    const int32_t p = q4 * 32 + lane;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    // The role exists in two copies, chosen once: plain stores, or (reduction slices, Z > 1) additions
    // into the zeroed output.  A choice inside the store loop, or an out-of-line call next to it,
    // slowed the C = 3 stem layers, which this loop bounds, by 20 %.
    PROF_DECL(6)
    auto epilogue_role = [&](auto kind_tag) {
      constexpr int EK = decltype(kind_tag)::value;  // 0 fp32 stores, 1 fp32 reductions, 2 bf16 stores, 3 fp32 stores in NHWC order
      constexpr bool REDUCE = EK == 1;
      Ring dr;
      bool ok = true;
      if (P.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");  // (the output is written only after the preceding grid has completed)
      const int32_t eK = P.K, eNT = P.NT, eHoWo = P.HoWo;  // kept in registers for the store loop
      // hand both accumulator buffers to the MMA side zeroed: every MMA accumulates
      for (int32_t d = 0; d < P.ND; ++d) {
        for (int32_t c0 = 0; c0 < P.NT; c0 += 16) ptx::tmem_zero_x16(tmem_base + lane_base + (uint32_t)(d * P.NT + c0));
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->acc_empty[d]));
      }
      for (int32_t t = blockIdx.x; t < (int32_t)P.ntiles && ok; t += gridDim.x, dr.advance(P.ND)) {
        PROF_T0(tp)
        const int32_t tile_m = tile_of(P, t);
        int32_t nt, g0_, g1_;
        unit_range(P, t, nt, g0_, g1_);
        (void)g0_; (void)g1_;
        const int32_t n0 = nt * P.NT;
        const TileInfo ti = tile_info(P, tile_m);
        const bool valid = p < ti.npos;
        float* orow = P.out;
        if (valid) {
          int32_t i_off, q;
          tile_row(P, ti, p, i_off, q);
          if constexpr (EK == 3) orow += ((ti.i_first + i_off) * (int64_t)P.HoWo + q) * P.K + n0;
          else orow += ((ti.i_first + i_off) * P.K + n0) * (int64_t)P.HoWo + q;
        }
        const int32_t d = dr.idx;
        PROF_ADD(1, tp)
        ok = wait_bar_warp(P, misc, &bars->acc_full[d], dr.phase, DEV_TIMEOUT_ACC, PROF_SLOT(0), 256);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + lane_base + (uint32_t)(d * P.NT);
        // 16 columns per trip.  Deliberately a rolled loop with a small body: this code runs once per
        // tile, and a fully unrolled store sequence (hundreds of instructions executed once) spent its
        // time on instruction fetch, the other roles' code having evicted it in between.
  #pragma unroll 1
        for (int32_t c0 = 0; c0 < eNT; c0 += 16) {
          uint32_t v[16];
          PROF_T0(t1)
          ptx::tmem_ld_x16(d_tmem + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
          PROF_ADD(2, t1)
          ptx::tmem_zero_x16(d_tmem + (uint32_t)c0);  // leave the columns zeroed for the next tile
          PROF_T0(t3)
          if constexpr (EK == 2) {
            // bf16 output: every lane rounds its own value and stores 16 bits; the 32 lanes of a
            // warp write 64 contiguous bytes per filter.  (Pairing neighbouring positions into 32-bit
            // stores through shuffles was slower: this loop is bound by its instruction count.)
            if (valid) {
              uint16_t* const o16 = reinterpret_cast<uint16_t*>(P.out) + (orow - P.out) + (int64_t)c0 * eHoWo;
              const int32_t left = eK - n0 - c0;
#pragma unroll
              for (int e = 0; e < 16; e += 2) {
                const uint32_t pk = ptx::pack_bf16x2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                if (e < left) o16[(int64_t)e * eHoWo] = (uint16_t)(pk & 0xffffu);
                if (e + 1 < left) o16[(int64_t)(e + 1) * eHoWo] = (uint16_t)(pk >> 16);
              }
            }
          } else if constexpr (EK == 3) {
            // NHWC: the thread's 16 filters of one position are contiguous
            if (valid) {
              float* o = orow + c0;
              const int32_t left = eK - n0 - c0;
              if (left >= 16 && (eK & 3) == 0) {
#pragma unroll
                for (int e = 0; e < 16; e += 4)
                  *reinterpret_cast<float4*>(o + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                                                  __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
              } else {
#pragma unroll
                for (int e = 0; e < 16; ++e)
                  if (e < left) o[e] = __uint_as_float(v[e]);
              }
            }
          } else
          if (valid) {
            float* o = orow + (int64_t)c0 * eHoWo;
            const int32_t left = eK - n0 - c0;  // filters of this block that exist
  #pragma unroll
            for (int e = 0; e < 16; ++e) {
              if (e < left) {
                if constexpr (REDUCE) atomicAdd(o + (int64_t)e * eHoWo, __uint_as_float(v[e]));  // fp32 reduction in L2
                else o[(int64_t)e * eHoWo] = __uint_as_float(v[e]);
              }
            }
          }
          PROF_ADD(4, t3)
        }
        PROF_T0(t4)
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->acc_empty[d]));
        PROF_ADD(5, t4)
      }
    };
    if constexpr (OUT16) {  // (separate instantiations: the fp32 kernels' code is not touched by this variant)
      epilogue_role(std::integral_constant<int, 2>{});
    } else {
      if (P.nhwc) epilogue_role(std::integral_constant<int, 3>{});
      else if (P.Z == 1) epilogue_role(std::integral_constant<int, 0>{});
      else epilogue_role(std::integral_constant<int, 1>{});
    }
    if (q4 == 0) { PROF_DUMP(6, 6) }
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  __syncthreads();
#ifdef IM2WIN_PROF
  if (P.prof && threadIdx.x == 0) { P.prof[512 + blockIdx.x * 4 + 1] = (long long)global_ns(); P.prof[512 + blockIdx.x * 4 + 3] = clock64(); }
#endif
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
  }
}

// fp32 -> bf16 (round to nearest even) copy of the filter, for the TMA-streamed BF16 filter operand
__global__ void __launch_bounds__(256) filter_to_bf16_kernel(const float* __restrict__ f, __nv_bfloat16* __restrict__ o,
                                                             int64_t n) {
  // the convolution kernel that follows may start now (its filter producer waits for this grid's completion)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256)
    o[i] = __float2bfloat16_rn(f[i]);
}

// The same copy with every channel group's KCG reduction elements padded with zeros to the KCGP the
// MMA steps cover, so that a filter row is indexed by (group, step) exactly as the kernel counts them.
__global__ void __launch_bounds__(256) filter_to_bf16_padded_kernel(const float* __restrict__ f,
                                                                    __nv_bfloat16* __restrict__ o, int64_t n_pad,
                                                                    int32_t Kg, int32_t KCG, int32_t KCGP, int32_t NG) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int32_t Kgp = NG * KCGP;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_pad; i += (int64_t)gridDim.x * 256) {
    const int64_t j = i / Kgp;
    const int32_t r = (int32_t)(i - j * Kgp);
    const int32_t grp = r / KCGP, kl = r - grp * KCGP;
    o[i] = kl < KCG ? __float2bfloat16_rn(f[j * Kg + (int64_t)grp * KCG + kl]) : __float2bfloat16_rn(0.f);
  }
}

// ---------------------------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}

template <int FH, int FW, int CB, bool BF16, bool FUSED, bool SRC16 = false, bool OUT16 = false>
int launch_spec_impl(const void* xhat, const float* f, float* out, const Geometry& g, cudaStream_t st, Scratch scratch) {
  constexpr bool out16 = OUT16;
  constexpr int FF = FH * FW;
  constexpr int64_t ES = SRC16 ? 2 : 4;    // bytes per source element
  constexpr int64_t EPC = 16 / ES;         // source elements per 16-byte chunk
  constexpr int KSTEP = BF16 ? 16 : 8;
  constexpr int KCG = CB * FF;
  constexpr int KCGP = (KCG + KSTEP - 1) / KSTEP * KSTEP;
  constexpr int S = KCGP / KSTEP;

  PParams P{};
  P.xhat = xhat; P.f = f; P.out = out;  // (OUT16: `out` points at 16-bit words)
  P.nhwc = g.out_nhwc;
  P.status = device_status_word();
  if (!P.status) return IM2WIN_ECUDA;
#ifdef IM2WIN_PROF
  P.prof = g_prof;
#endif
  P.C = g.C; P.K = g.K; P.Ho = g.Ho; P.Wo = g.Wo; P.W = g.W;
  if (g.HoWo > (1 << 30)) return IM2WIN_EUNSUPPORTED;
  P.HoWo = (int32_t)g.HoWo; P.Kg = g.Kg; P.Mtot = g.Mtot;
  if (FUSED) {  // source = the untransformed input: windows are read from Fh staged rows
    P.row_mul = g.s * g.W; P.col_mul = g.s; P.win_span = (g.Fh - 1) * g.W + g.Fw;
    P.plane = (int64_t)g.H * g.W; P.n_src = g.n_in;
  } else {      // source = the im2win tensor: a window is Fh*Fw contiguous floats of its strip
    P.row_mul = g.L; P.col_mul = g.sFh; P.win_span = FF;
    P.plane = g.HoL; P.n_src = g.n_win;
  }
  int64_t tp = 128;
  if ((kSegMax - 1) * g.HoWo + 1 < tp) tp = (kSegMax - 1) * g.HoWo + 1;
  P.TP = (int32_t)tp;
  P.n_ntiles = (g.K + 255) / 256;
  P.NT = ((g.K + P.n_ntiles - 1) / P.n_ntiles + 15) / 16 * 16;
  {
    // Filter tiles stay as wide as the MMA allows (256): a unit of work costs the same number of MMA
    // instructions and window repacks whatever its width, and narrow MMAs are bound by the issuing
    // thread, so splitting K further to even out the last wave loses (measured).  Tuning aid only:
    const int fix = knobs().ntiles;
    if (fix >= 1 && fix <= 8 && (g.K + fix - 1) / fix <= 256) {
      P.n_ntiles = fix;
      P.NT = ((g.K + P.n_ntiles - 1) / P.n_ntiles + 15) / 16 * 16;
    }
  }
  P.NG = (g.C + CB - 1) / CB;
  const int32_t steps_tile = P.NG * S;
  P.nchunks = (steps_tile + 3) / 4;

  // worst-case floats one channel contributes to a tile
  const int64_t rowwrap = (int64_t)P.row_mul - (int64_t)(g.Wo - 1) * P.col_mul;
  const int64_t wraps = (tp + g.Wo - 2) / g.Wo;
  int64_t nseg_max = (tp - 1) / g.HoWo + 2;
  if (nseg_max > kSegMax) nseg_max = kSegMax;
  int64_t pitch = (tp - 1) * P.col_mul + wraps * (rowwrap > P.col_mul ? rowwrap - P.col_mul : 0) + nseg_max * (P.win_span + 6) + 4;
  pitch = (pitch + 3) & ~(int64_t)3;
  if (pitch > (1 << 20)) return IM2WIN_EUNSUPPORTED;
  // Per-image tiling: where images are large enough that cutting tiles per image wastes little, a
  // tile lies in one image and needs one contiguous range per channel; the per-tile index work of
  // every role then is a few multiplications (divisions by precomputed reciprocals).
  // Box mode (on top of it): one 2-D TMA box (CB planes x one contiguous range) per channel group
  // instead of CB bulk copies.  Needs planes that are multiples of 16 bytes and a range of at most
  // 256 8-byte elements.
  {
    const int64_t tpi = (g.HoWo + 127) / 128;
    // (+ the 16-byte phase in front and the rounding up to whole 16-byte chunks behind)
    const int64_t one_seg = 127 * (int64_t)P.col_mul + wraps * (rowwrap > P.col_mul ? rowwrap - P.col_mul : 0) +
                            P.win_span + 2 * (EPC - 1) + EPC;
    // A box row is a whole number of 16-byte units, and CB rows (one stage) a whole number of 128
    // bytes, so that every stage starts on the 128-byte boundary a tiled TMA destination needs.
    int64_t row_align = EPC;
    while ((CB * row_align * ES) % 128 != 0) row_align *= 2;
    const int64_t boxf = (one_seg + row_align - 1) / row_align * row_align;
    const bool little_waste = tpi * 128 * 100 <= g.HoWo * 107;
    if (little_waste && tp == 128 && P.plane < ((int64_t)1 << 30) && (g.HoWo + 128) * g.Wo < ((int64_t)1 << 32) &&
        (int64_t)g.N * tpi * tpi < ((int64_t)1 << 32) && one_seg <= (1 << 20) && !knobs().no_pim) {
      P.pim = 1;
      P.TPI = (int32_t)tpi;
      P.magic_TPI = (((uint64_t)1 << 32) + (uint64_t)tpi - 1) / (uint64_t)tpi;
      P.magic_Wo = (((uint64_t)1 << 32) + (uint64_t)g.Wo - 1) / (uint64_t)g.Wo;
      pitch = (one_seg + EPC - 1) / EPC * EPC;
      if (CB >= 2 && (P.plane % EPC) == 0 && boxf * ES <= 2048 && encode_fn() != nullptr && (int64_t)g.N * g.C <= INT32_MAX &&
          !knobs().no_box) {
        P.box = 1;
        P.l2_ahead = !knobs().no_l2ahead;
        pitch = boxf;
      }
    }
  }
  if (SRC16 && !P.pim) return IM2WIN_EUNSUPPORTED;  // the 16-bit source is implemented for per-image tiling only
  // Tiles that span images: each of the strip producer's 32 lanes owns at most two (channel, image
  // segment) pairs of a group, so a group holds at most 64 of them.  (Sixteen-channel groups on images
  // of fewer than ~40 positions exceed that; the dispatcher then takes the eight-channel variant.)
  if (!P.pim && (int64_t)CB * nseg_max > 64) return IM2WIN_EUNSUPPORTED;
  P.chan_pitch = (int32_t)pitch;
  const int64_t tiles_m = P.pim ? (int64_t)g.N * P.TPI : (g.Mtot + P.TP - 1) / P.TP;
  P.ntiles = tiles_m * P.n_ntiles;
  const int64_t raw_stage = (int64_t)CB * pitch * ES;

  // filter operand: resident if it fits next to two strip stages, else streamed by TMA (TF32, dense groups)
  const int64_t cap = 227 * 1024 - 1024 - 1024 - ((int64_t)(P.win_span + 8) * 4 + 16);  // alignment slack, barriers, zero pad
  const int64_t b_res = (int64_t)steps_tile * P.NT * 32;  // one 32-byte-swizzled block per MMA step
  bool resident = P.n_ntiles == 1 && b_res + 2 * raw_stage <= cap;
  if (knobs().force_stream) resident = false;  // test knob
  // Streaming the native TF32 filter needs dense groups (padded reduction index == real index) and
  // 16-byte aligned filter rows.  In BF16 mode the TMA source is a bf16 copy of the filter, written at
  // the start of the call into scratch memory the caller supplied beyond the im2win tensor (without
  // enough scratch this kernel does not apply); that copy has padded groups where the groups are not dense.
  const bool pad_copy = BF16 && KCG != KCGP;
  const int64_t copy_row = pad_copy ? (int64_t)((g.C + CB - 1) / CB) * KCGP : g.Kg;
  const bool have_copy_room = scratch.ptr && (int64_t)scratch.bytes >= (int64_t)g.K * copy_row * 2;
  const bool can_stream = (g.C % CB) == 0 && encode_fn() != nullptr &&
                          (BF16 ? have_copy_room && (pad_copy || (g.Kg % 8) == 0) : KCG == KCGP && (g.Kg % 4) == 0);
  if (!resident && !can_stream) return IM2WIN_EUNSUPPORTED;
  // Slice-resident mode.  A filter that does not fit whole may fit as one reduction slice per CTA:
  // the units are (tile, slice) with the slice fastest, so with a grid that is a multiple of Z every
  // CTA keeps to one slice, holds that slice of the filter for the whole kernel and adds its partial
  // sums into the zeroed output.  The price is Z epilogues per tile, each of atomic adds: an SM
  // passes about one 32-bit add per cycle, so an epilogue warp spends ~85 cycles per accumulator
  // column (measured; ~31 with plain stores).  It pays only for long reductions onto few output
  // channels (Table I Conv4: C = 64, 7x7, K = 64) -- estimated against the streamed mode, whose
  // issuing threads spend about 200 cycles per MMA (measured), in microseconds at 1.9 GHz.
  int32_t bs_z = 0, bs_gz = 0;
  const bool bs_force = knobs().bslice != 0;  // test knob
  if ((!resident || bs_force) && P.n_ntiles == 1 && !out16 && !g.out_nhwc && !knobs().no_bslice) {
    const int nsm = sm_count();
    for (int32_t z = 2; z <= 16 && z <= P.NG && z <= nsm; ++z) {
      const int32_t gz = (P.NG + z - 1) / z;
      const int32_t z_eff = (P.NG + gz - 1) / gz;
      if ((int64_t)gz * S * P.NT * 32 + 2 * raw_stage > cap) continue;
      const double pipe = BF16 ? P.NT / 4.0 : P.NT / 2.0;  // cycles of one MMA in the tensor pipe
      const int64_t grid_z = (int64_t)(nsm / z_eff) * z_eff;
      const double units_cta = (double)((P.ntiles * z_eff + grid_z - 1) / grid_z);
      const double mma_u = (double)gz * S * (pipe > 30.0 ? pipe : 30.0);
      const double epi_u = P.NT * 85.0;
      const bool two_acc = 2 * P.NT + 2 * 40 <= 512;
      const double work_us = units_cta * (two_acc ? (mma_u > epi_u ? mma_u : epi_u) : mma_u + epi_u) / 1900.0;
      const double zero_us = 3.0 + (double)g.n_out * 4.0 / 3.0e6;
      const double t_slice = work_us + zero_us;
      const double t_stream = (double)((P.ntiles + nsm - 1) / nsm) * P.NG * S * (pipe > 200.0 ? pipe : 200.0) / 1900.0;
      if (bs_force || t_slice < 0.8 * t_stream) { bs_z = z_eff; bs_gz = gz; }
      break;  // the smallest Z that fits
    }
    if (bs_z) resident = true;
  }
  int64_t b_bytes;
  if (resident) {
    b_bytes = bs_z ? (int64_t)bs_gz * S * P.NT * 32 : b_res;
    P.bslice = bs_z ? 1 : 0;
    P.SB = 1;
  } else {
    P.SB = 6;
    while (P.SB > 3 && (int64_t)P.SB * P.NT * 128 + 4 * raw_stage > cap) --P.SB;
    b_bytes = (int64_t)P.SB * P.NT * 128;
  }
  // Repack sets and strip stages.  The sets take groups in turn, so with a stage count that is a
  // multiple of the number of sets a stage is always read by the same set, which then sees every
  // phase of the stage's barrier.  (A waiter that skips phases can poll before the previous phase
  // has completed and would take it for its own.)  Three sets where that leaves at least six
  // stages in flight, else two.
  const int SLOT_STEPS = resident ? SlotGeom<S, true>::SLOT_STEPS : SlotGeom<S, false>::SLOT_STEPS;
  const int SLOT_COLS = SLOT_STEPS * 8;
  int32_t sr_max = (int32_t)((cap - b_bytes) / raw_stage);
  if (sr_max > kMaxStages) sr_max = kMaxStages;
  P.NSETS = (sr_max / 3 * 3 >= 6 || sr_max == 3) ? 3 : 2;
  const bool nsets_fixed = knobs().nsets == 2 || knobs().nsets == 3;
  if (nsets_fixed) P.NSETS = knobs().nsets;
  // TMEM: accumulators first, then the rings of A slots, one ring of NSS slots per set (a barrier
  // must be waited on by one party that sees every one of its phases, so the sets cannot share slots)
  P.ND = (2 * P.NT + P.NSETS * SLOT_COLS <= 512) ? 2 : 1;
  // a third set only pays where every set still owns at least two slots (a set with one slot waits
  // for the MMAs of each part before it can store the next)
  if ((512 - P.ND * P.NT) / SLOT_COLS / P.NSETS < 2 && !nsets_fixed) P.NSETS = 2;
  P.ND = (2 * P.NT + P.NSETS * SLOT_COLS <= 512) ? 2 : 1;
  if (P.ND * P.NT + P.NSETS * SLOT_COLS > 512) P.NSETS = 2;
  P.SR = sr_max / P.NSETS * P.NSETS;
  if (P.SR < 2) return IM2WIN_EUNSUPPORTED;
  P.NSS = (512 - P.ND * P.NT) / SLOT_COLS / P.NSETS;
  if (P.NSS > 4) P.NSS = 4;
  if (P.NSS < 1) return IM2WIN_EUNSUPPORTED;
  P.SS = SLOT_STEPS;

  // Reduction slices.  When the (m-tile, n-tile) units do not fill the SMs evenly -- few tiles at
  // small batch, or a last wave that is mostly idle -- a unit's channel groups are cut into Z slices
  // that run as separate units and add their partial sums into the zeroed output.  Z is picked with
  // a small cost model: waves x (groups per slice x cycles per group + per-unit overhead), where a
  // group costs its MMA time (or the repack floor) and the overhead is the pipeline fill plus, with a
  // single accumulator buffer, the epilogue that nothing overlaps; a split also pays for zeroing the
  // output.  A slice of a streamed filter must start on a 128-byte filter chunk (4 MMA steps).
  P.Z = 1; P.GZ = P.NG;
  {
    const int64_t units1 = P.ntiles;
    const int nsm = sm_count();
    const double group_cyc = (double)S * P.NT * 0.7 > 600.0 ? (double)S * P.NT * 0.7 : 600.0;
    const double ov_cyc = (P.ND == 1 ? P.NT * 31.0 : 0.0) + 3000.0;
    const double zero_cyc = 5000.0 + (double)g.n_out * 4.0 / 1600.0;  // the extra launch that zeroes the output
    auto cost = [&](int64_t z_eff, int32_t gz) {
      const int64_t waves = (units1 * z_eff + nsm - 1) / nsm;
      const double c = (double)waves * (gz * group_cyc + ov_cyc);
      return z_eff > 1 ? c * 1.05 + zero_cyc : c;
    };
    int32_t gmul = 1;
    if (!resident) while ((gmul * S) % 4 != 0) ++gmul;
    double best = cost(1, P.NG) * 0.92;  // a split must win clearly
    int forced = knobs().splitk;
    if (out16 || g.out_nhwc) forced = 1;  // partial sums cannot be added into a bf16 output; the NHWC epilogue has no adding copy
    for (int32_t z = 2; z <= 16 && z <= P.NG; ++z) {
      int32_t gz = (P.NG + z - 1) / z;
      gz = (gz + gmul - 1) / gmul * gmul;
      const int32_t z_eff = (P.NG + gz - 1) / gz;
      if (z_eff < 2) continue;
      const double c = cost(z_eff, gz);
      if (forced >= 0 ? z == forced : c < best) { best = c; P.Z = z_eff; P.GZ = gz; }
    }
    if (forced == 0 || forced == 1) { P.Z = 1; P.GZ = P.NG; }
    if (bs_z) { P.Z = bs_z; P.GZ = bs_gz; }
  }
  P.usub = P.n_ntiles * P.Z;
  P.ntiles *= P.Z;
  // the roles count work units in 32 bits (t, t + grid, ...): decline what does not fit, instead of wrapping
  if (P.ntiles > (int64_t)INT32_MAX - sm_count()) return IM2WIN_EUNSUPPORTED;
  const int32_t cols = P.ND * P.NT + P.NSETS * P.NSS * SLOT_COLS;
  P.tmem_cols = 32;
  while (P.tmem_cols < cols) P.tmem_cols *= 2;
  P.idesc = ptx::make_idesc(128, P.NT, BF16 ? 1 : 2);

  uint32_t off = (uint32_t)b_bytes;
  P.off_raw = off; off += (uint32_t)(P.SR * raw_stage);
  P.off_zero = off; off += (uint32_t)(((P.win_span + 8) * 4 + 15) / 16 * 16);
  P.off_bar = off; off += (uint32_t)((sizeof(PBars) + 15) / 16 * 16);
  P.off_misc = off; off += 64;
  const size_t smem_bytes = off + 1024;

  // reduction slices add into a zeroed output (before the filter copy's launch, so that the convolution
  // kernel can follow that copy as a programmatic dependent)
  if (P.Z > 1 && cudaMemsetAsync(out, 0, (size_t)g.n_out * 4, st) != cudaSuccess) {  // (Z > 1 implies an fp32 output)
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  CUtensorMap fmap;
  memset(&fmap, 0, sizeof(fmap));
  void* f_bf16 = nullptr;  // BF16 streamed mode: bf16 copy of the filter in the caller's scratch
  if (resident && !BF16 && KCG == KCGP && (g.C % CB) == 0 && (g.Kg % 4) == 0 && encode_fn() != nullptr &&
      !knobs().no_btma) {
    // the native filter as a K x Kg matrix, fetched one MMA step (8 reduction elements) at a time
    const cuuint64_t gdim[2] = {(cuuint64_t)g.Kg, (cuuint64_t)g.K};
    const cuuint64_t gstr[1] = {(cuuint64_t)g.Kg * 4};
    const cuuint32_t box[2] = {8u, (cuuint32_t)P.NT};
    const cuuint32_t estr[2] = {1, 1};
    if (encode_fn()(&fmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(f), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
      P.b_tma = 1;
  }
  if (!resident) {
    const int64_t row = pad_copy ? (int64_t)P.NG * KCGP : g.Kg;  // filter row length seen by the TMA
    const cuuint64_t gdim[2] = {(cuuint64_t)row, (cuuint64_t)g.K};
    const cuuint64_t gstr[1] = {(cuuint64_t)row * (BF16 ? 2 : 4)};
    const cuuint32_t box[2] = {BF16 ? 64u : 32u, (cuuint32_t)P.NT};  // one 128-byte row of the swizzle
    const cuuint32_t estr[2] = {1, 1};
    void* base = const_cast<float*>(f);
    if (BF16) {
      const int64_t n_copy = (int64_t)g.K * row;
      f_bf16 = scratch.ptr;
      const int64_t blocks = (n_copy + 255) / 256;
      const unsigned nb = (unsigned)(blocks < 148 * 8 ? blocks : 148 * 8);
      if (pad_copy)
        filter_to_bf16_padded_kernel<<<nb, 256, 0, st>>>(f, static_cast<__nv_bfloat16*>(f_bf16), n_copy, (int32_t)g.Kg,
                                                         KCG, KCGP, P.NG);
      else
        filter_to_bf16_kernel<<<nb, 256, 0, st>>>(f, static_cast<__nv_bfloat16*>(f_bf16), g.n_flt);
      base = f_bf16;
    }
    if (encode_fn()(&fmap, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, gdim,
                    gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      return IM2WIN_EUNSUPPORTED;
    }
  }
  CUtensorMap xmap;
  memset(&xmap, 0, sizeof(xmap));
  if (P.box) {
    // the source as [N*C planes][plane bytes / 8 8-byte elements]
    const cuuint64_t gdim[2] = {(cuuint64_t)(P.plane * ES / 8), (cuuint64_t)g.N * g.C};
    const cuuint64_t gstr[1] = {(cuuint64_t)P.plane * ES};
    const cuuint32_t box[2] = {(cuuint32_t)(P.chan_pitch * ES / 8), (cuuint32_t)CB};
    const cuuint32_t estr[2] = {1, 1};
    if (encode_fn()(&xmap, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(xhat), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      return IM2WIN_ECUDA;
    }
  }
  int64_t grid = P.ntiles < sm_count() ? P.ntiles : sm_count();
  if (P.bslice) grid = grid / P.Z * P.Z;  // every CTA keeps to one slice
  cudaError_t e;
  // Programmatic dependent launch: behind the filter-copy kernel (BF16 streamed mode) the prologue, strip copies
  // and repacking overlap that copy, and the filter producer waits for it; behind the transform kernel the
  // prologue overlaps that kernel's tail, and the strip producer and the epilogue wait (griddepcontrol.wait).
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // (the filter copy itself is an ordinary launch: when it runs, everything before it has completed)
  P.wait_prev = f_bf16 ? 0 : 1;
  if (resident) {
    auto kern = conv_tc_persistent_kernel<FH, FW, CB, BF16, true, FUSED, SRC16, OUT16>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
    if (cudaLaunchKernelEx(&cfg, kern, P, fmap, xmap) != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  } else {
    auto kern = conv_tc_persistent_kernel<FH, FW, CB, BF16, false, FUSED, SRC16, OUT16>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
    if (cudaLaunchKernelEx(&cfg, kern, P, fmap, xmap) != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  }
  note_kernel(KERNEL_PERSISTENT);
  return cuda_status(cudaGetLastError());
}

// src_kind: 0 = im2win tensor (fp32), 1 = untransformed input consumed fused, 2 = im2win tensor stored as bf16
template <int FH, int FW, int CB, bool BF16>
int launch_spec(const void* src, const float* f, float* out, const Geometry& g, cudaStream_t st, Scratch scratch,
                int src_kind, bool out16) {
  if (out16) {  // the bf16 epilogue exists for the unfused sources
    if (src_kind == 1) return IM2WIN_EUNSUPPORTED;
    if (src_kind == 2) {
      if constexpr (BF16) return launch_spec_impl<FH, FW, CB, true, false, true, true>(src, f, out, g, st, scratch);
      else return IM2WIN_EUNSUPPORTED;
    }
    return launch_spec_impl<FH, FW, CB, BF16, false, false, true>(src, f, out, g, st, scratch);
  }
  if (src_kind == 2) {
    if constexpr (BF16) return launch_spec_impl<FH, FW, CB, true, false, true>(src, f, out, g, st, scratch);
    else return IM2WIN_EUNSUPPORTED;
  }
  return src_kind == 1 ? launch_spec_impl<FH, FW, CB, BF16, true>(src, f, out, g, st, scratch)
                       : launch_spec_impl<FH, FW, CB, BF16, false>(src, f, out, g, st, scratch);
}

}  // namespace

// Returns IM2WIN_EUNSUPPORTED when no specialisation applies (the caller then uses the generic kernel).
// scratch: device memory of the caller's (beyond the im2win tensor) for the bf16 copy of a filter that
// is too large to stay in shared memory (BF16 mode); without it those shapes are declined.
// fused: `xhat` is the untransformed NCHW input and the windows are built from staged input rows
// (no im2win tensor exists in global memory).
// The filter-size families are separate functions so that the build can compile them as separate
// translation units in parallel (-DIM2WIN_PART=0..5: part 0 = 3x3 + this dispatcher, 1 = 5x5,
// 2 = 7x7, 3 = 11x11, 4 = 1x1 / 1x3 / 3x1, 5 = 1x7 / 7x1, 6 = 2x2 / 4x4, 7 = 3x5 / 5x3; without the macro
// everything is compiled here).
#ifndef IM2WIN_PART
#define IM2WIN_PART -1
#endif
#define IM2WIN_SPEC_ARGS const void* xhat, const float* f, float* out, const Geometry& g, cudaStream_t st, \
                         Scratch scratch, int kind, bool out_bf16, bool bf16
int launch_spec_3x3(IM2WIN_SPEC_ARGS);
int launch_spec_5x5(IM2WIN_SPEC_ARGS);
int launch_spec_7x7(IM2WIN_SPEC_ARGS);
int launch_spec_11x11(IM2WIN_SPEC_ARGS);
int launch_spec_rect_a(IM2WIN_SPEC_ARGS);
int launch_spec_rect_b(IM2WIN_SPEC_ARGS);
int launch_spec_rect_c(IM2WIN_SPEC_ARGS);
int launch_spec_rect_d(IM2WIN_SPEC_ARGS);

#if IM2WIN_PART == -1 || IM2WIN_PART == 0
int launch_spec_3x3(IM2WIN_SPEC_ARGS) {
  // BF16 MMAs take 16 reduction elements: sixteen channels (144 = 9 steps) leave no padding
  if (bf16 && g.C % 16 == 0) {
    const int rc = launch_spec<3, 3, 16, true>(xhat, f, out, g, st, scratch, kind, out_bf16);
    if (rc != IM2WIN_EUNSUPPORTED) return rc;
  }
  if (g.C >= 8) return bf16 ? launch_spec<3, 3, 8, true>(xhat, f, out, g, st, scratch, kind, out_bf16)
                            : launch_spec<3, 3, 8, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  if (g.C == 3) return bf16 ? launch_spec<3, 3, 3, true>(xhat, f, out, g, st, scratch, kind, out_bf16)
                            : launch_spec<3, 3, 3, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif
#if IM2WIN_PART == -1 || IM2WIN_PART == 1
int launch_spec_5x5(IM2WIN_SPEC_ARGS) {
  if (bf16 && g.C % 16 == 0) {
    const int rc = launch_spec<5, 5, 16, true>(xhat, f, out, g, st, scratch, kind, out_bf16);
    if (rc != IM2WIN_EUNSUPPORTED) return rc;
  }
  if (g.C >= 8) return bf16 ? launch_spec<5, 5, 8, true>(xhat, f, out, g, st, scratch, kind, out_bf16)
                            : launch_spec<5, 5, 8, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif
#if IM2WIN_PART == -1 || IM2WIN_PART == 2
int launch_spec_7x7(IM2WIN_SPEC_ARGS) {
  if (g.C % 8 == 0) {
    if (bf16) {
      // sixteen channels per group leave no padding (784 = 49 steps); where two strip stages of
      // sixteen channels do not fit (wide images), eight channels with a padded filter copy do
      int rc = IM2WIN_EUNSUPPORTED;
      if (g.C % 16 == 0) rc = launch_spec<7, 7, 16, true>(xhat, f, out, g, st, scratch, kind, out_bf16);
      if (rc == IM2WIN_EUNSUPPORTED) rc = launch_spec<7, 7, 8, true>(xhat, f, out, g, st, scratch, kind, out_bf16);
      return rc;
    }
    return launch_spec<7, 7, 8, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  }
  if (g.C == 3) return bf16 ? launch_spec<7, 7, 3, true>(xhat, f, out, g, st, scratch, kind, out_bf16)
                            : launch_spec<7, 7, 3, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif
#if IM2WIN_PART == -1 || IM2WIN_PART == 3
int launch_spec_11x11(IM2WIN_SPEC_ARGS) {
  if (g.C <= 4) return bf16 ? launch_spec<11, 11, 1, true>(xhat, f, out, g, st, scratch, kind, out_bf16)
                            : launch_spec<11, 11, 1, false>(xhat, f, out, g, st, scratch, kind, out_bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif

// Pointwise, factorised, patch and other small rectangular filters (1x1; 1x3 / 3x1; 1x7 / 7x1; 2x2, 4x4; 3x5 / 5x3):
// the same kernel, from the fp32 im2win tensor or
// fused, fp32 NCHW or NHWC output (the bf16 storage variants of these shapes go to the generic kernel).
// Sixteen channels per group (TF32: two to six MMA steps, BF16: one to seven, no padding); 1x7 / 7x1 in TF32
// mode: eight (seven steps).
template <int FH, int FW>
int launch_spec_rect(IM2WIN_SPEC_ARGS) {
  if (kind == 2 || out_bf16 || g.C % 8 != 0) return IM2WIN_EUNSUPPORTED;
  if constexpr (FH * FW == 1) {  // pointwise: thirty-two channels per group where they divide C
    if (g.C % 32 == 0) {
      int rc;
      if (bf16) rc = kind == 1 ? launch_spec_impl<1, 1, 32, true, true>(xhat, f, out, g, st, scratch)
                               : launch_spec_impl<1, 1, 32, true, false>(xhat, f, out, g, st, scratch);
      else rc = kind == 1 ? launch_spec_impl<1, 1, 32, false, true>(xhat, f, out, g, st, scratch)
                          : launch_spec_impl<1, 1, 32, false, false>(xhat, f, out, g, st, scratch);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
  }
  if (bf16) {
    int rc = IM2WIN_EUNSUPPORTED;
    if (g.C % 16 == 0)
      rc = kind == 1 ? launch_spec_impl<FH, FW, 16, true, true>(xhat, f, out, g, st, scratch)
                     : launch_spec_impl<FH, FW, 16, true, false>(xhat, f, out, g, st, scratch);
    // an even number of taps: eight channels are whole MMA steps too, for strips too long for sixteen-channel
    // stages (4x4 with stride 4: 16 floats per position)
    if constexpr ((8 * FH * FW) % 16 == 0 && FH * FW >= 4) {
      if (rc == IM2WIN_EUNSUPPORTED)
        rc = kind == 1 ? launch_spec_impl<FH, FW, 8, true, true>(xhat, f, out, g, st, scratch)
                       : launch_spec_impl<FH, FW, 8, true, false>(xhat, f, out, g, st, scratch);
    }
    return rc;
  }
  constexpr int CBT = FH * FW >= 7 ? 8 : 16;
  if (g.C % CBT != 0) return IM2WIN_EUNSUPPORTED;
  return kind == 1 ? launch_spec_impl<FH, FW, CBT, false, true>(xhat, f, out, g, st, scratch)
                   : launch_spec_impl<FH, FW, CBT, false, false>(xhat, f, out, g, st, scratch);
}
#if IM2WIN_PART == -1 || IM2WIN_PART == 4
int launch_spec_rect_a(IM2WIN_SPEC_ARGS) {
  if (g.Fh == 1 && g.Fw == 1) return launch_spec_rect<1, 1>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 1 && g.Fw == 3) return launch_spec_rect<1, 3>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 3 && g.Fw == 1) return launch_spec_rect<3, 1>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif
#if IM2WIN_PART == -1 || IM2WIN_PART == 5
int launch_spec_rect_b(IM2WIN_SPEC_ARGS) {
  if (g.Fh == 1 && g.Fw == 7) return launch_spec_rect<1, 7>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 7 && g.Fw == 1) return launch_spec_rect<7, 1>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif

#if IM2WIN_PART == -1 || IM2WIN_PART == 6
int launch_spec_rect_c(IM2WIN_SPEC_ARGS) {  // the patch / downsampling filters
  if (g.Fh == 2 && g.Fw == 2) return launch_spec_rect<2, 2>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 4 && g.Fw == 4) return launch_spec_rect<4, 4>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif
#if IM2WIN_PART == -1 || IM2WIN_PART == 7
int launch_spec_rect_d(IM2WIN_SPEC_ARGS) {
  if (g.Fh == 3 && g.Fw == 5) return launch_spec_rect<3, 5>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 5 && g.Fw == 3) return launch_spec_rect<5, 3>(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  return IM2WIN_EUNSUPPORTED;
}
#endif

#if IM2WIN_PART == -1 || IM2WIN_PART == 0
int launch_conv_tc_persistent(const void* xhat, const float* f, float* out, const Geometry& g, int mode,
                              cudaStream_t st, Scratch scratch, bool fused, bool src_bf16, bool out_bf16) {
  const int kind = src_bf16 ? 2 : (fused ? 1 : 0);
  if (src_bf16 && (fused || mode != IM2WIN_MODE_BF16)) return IM2WIN_EUNSUPPORTED;
  const bool bf16 = mode == IM2WIN_MODE_BF16;
  if (g.Fh == 3 && g.Fw == 3) return launch_spec_3x3(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 5 && g.Fw == 5) return launch_spec_5x5(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 7 && g.Fw == 7) return launch_spec_7x7(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 11 && g.Fw == 11) return launch_spec_11x11(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == 1 && g.Fw == 7 || g.Fh == 7 && g.Fw == 1) return launch_spec_rect_b(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh * g.Fw <= 3 && (g.Fh == 1 || g.Fw == 1) && g.Fh * g.Fw != 2)
    return launch_spec_rect_a(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh == g.Fw && (g.Fh == 2 || g.Fh == 4)) return launch_spec_rect_c(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  if (g.Fh * g.Fw == 15 && (g.Fh == 3 || g.Fh == 5)) return launch_spec_rect_d(xhat, f, out, g, st, scratch, kind, out_bf16, bf16);
  return IM2WIN_EUNSUPPORTED;
}

// Upper bound of the scratch bytes any BF16 specialisation asks for: a bf16 copy of the filter whose
// channel groups (8 or 16 channels, or fewer for tiny C) are padded to whole MMA steps of 16.
size_t persistent_scratch_bytes(const Geometry& g, int mode) {
  if (mode != IM2WIN_MODE_BF16) return 0;
  const int64_t ff = g.FF;
  const int64_t row = g.C >= 8 ? (int64_t)((g.C + 7) / 8) * ((8 * ff + 15) / 16 * 16) : (int64_t)g.C * ((ff + 15) / 16 * 16);
  return (size_t)((int64_t)g.K * row * 2 + 255) / 256 * 256;
}

#ifdef IM2WIN_PROF
// (debug build only)
extern "C" void im2win_debug_set_prof(long long* device_buf) { g_prof = device_buf; }
#endif
#endif  // IM2WIN_PART == -1 || IM2WIN_PART == 0

}  // namespace im2win
