// im2win-based convolution (Algorithm 2) on the sm_100a tensor cores: the WINDOW-OFFSET kernel (stride 1).
//
// Section III-A's observation, taken one step further than the strip-matrix kernel does: with stride 1 the
// im2win tensor holds every input element Fh times (element (h, k) of a channel is entry u of the strip of
// output row m for every m + u = h), and a dot-product window is Fh*Fw of those elements at fixed distances.
// So ONE copy of each element in shared memory is enough.  A stage holds, for G channels, the matrix
//     X[e][r] = I[r][h][k],   e = h*W + k   (all input positions a tile of outputs needs, channels fastest),
// stored as 16-byte chunks of NCH channels, chunk-major without swizzle (chunk c of row e at c*LBO + e*16).
// The window element (u, v) of output position p = m*W + n is row p + u*W + v of X, so each of the Fh*Fw
// taps is the same MMA operand with the descriptor's start address moved by u*W + v rows:
//     O[p, j] = sum_{u,v} sum_r X[p + u*W + v][r] * F[j][r][u][v],
// a tcgen05.mma (A and B from shared memory) per (tap, 8 or 16 channels, 128 rows).  Rows p with n >= Wo
// are computed and dropped.  Nothing is expanded anywhere: an element is staged once (TMA), interleaved
// once (four or eight channels -> one 16-byte store) and then read by the tensor core Fh*Fw times.
//
// Sources: the fp32 or bf16 im2win tensor (entry u = 0 of strip h supplies (h, k); the last Fh-1 input
// rows of a tile come from entries u > 0 of its last strip, so every byte of the tensor is fetched once
// and nothing outside the tile's own strips is touched), or the untransformed input (the fused kind).
// The filter operand is a tap-major copy F9[(u,v)][j][r] that a small kernel writes into the caller's
// scratch at the start of the call, streamed by TMA boxes with the 64-byte swizzle.
//
// Roles (one persistent CTA per SM, units t, t+grid, ...; a unit = 128*MH positions x one filter tile):
//   warp 0       source producer (2-D TMA boxes, or one bulk copy per channel)
//   warp 1       MMA issuer (one thread, fully unrolled over one filter stage, fixed summation order)
//   warp 2       filter producer
//   warps 4-11   interleavers: staged channel rows -> X (fp32 as is for TF32, cvt.rn.bf16x2 for BF16)
//   warps 12-19  epilogue: tcgen05.ld -> coalesced NCHW stores
// Every wait is bounded (status word + common teardown on expiry).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>
#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "strip_common.cuh"

namespace im2win {
namespace {

using namespace stripc;

constexpr int kXMax = 3;  // X rows per interleaver thread and stage

struct WParams {
  const void* src;
  float* out;
  int32_t* status;
  int32_t C, K, Ho, Wo, W, H;
  int32_t RPI;        // positions per image, counted with the full row length: Ho * W
  int32_t TPI;        // row tiles per image
  int32_t MH;         // 128-row blocks per tile
  int32_t RX;         // X rows a tile uses: 128*MH + (Fh-1)*W + Fw-1
  int32_t RA;         // X rows allocated (RX rounded up to 8)
  int32_t NT, n_ntiles, Kp;
  int32_t NTB;        // filter rows one CTA holds per block: NT, or NT/2 when two CTAs share an MMA
  int32_t nhwc;       // output layout N x Ho x Wo x K
  int32_t bres;       // the whole filter tile stays in shared memory: SB stages = one unit's, loaded once per CTA
  int32_t two;        // two MMA-issuing threads share the filter stages by parity; every MMA accumulates, the epilogue zeroes behind its reads
  int32_t pair;       // two CTAs (a cluster) work as one: tcgen05.mma.cta_group::2, M = 256, each CTA its own rows and half the filter tile
  int32_t G, GR, NSUB, NXS;  // channels per X stage / per source stage, source stages per X stage, X stages per unit
  int32_t TPS;        // taps per filter stage (Fw: one filter row per stage; 1: one tap per stage)
  int32_t SR, SB, ND;
  int32_t n_epi;      // epilogue warps in use
  int32_t epi_split;  // the epilogue warps store columns [0, epi_split); with one accumulator buffer the (then idle)
                      // interleaver warps store [epi_split, NT); epi_split == NT: no help
  int32_t box;        // source stages come as 2-D TMA boxes
  int32_t NBX, BXE;   // boxes per source stage; elements per box row (bulk copies: one "box" of CP elements)
  int32_t pm;         // plane length modulo the elements of a 16-byte chunk (bulk copies: per-channel phase)
  int64_t plane;      // source elements per (image, channel)
  int64_t n_src;
  int64_t tiles, units;
  uint32_t idesc, tmem_cols;
  uint32_t raw_stage_bytes, x_stage_bytes, b_stage_bytes;
  uint32_t off_x, off_raw, off_bar, off_misc;
#ifdef IM2WIN_PROF
  long long* prof;
  int32_t skip;   // ablation (profiling build only): 1 = interleavers copy nothing, 2 = no filter loads, 4 = no source loads
#endif
};

struct WUnit {
  int32_t nt, img, R0;
  bool store;
};
// Single-CTA mode: units t = blockIdx.x + it*grid, the filter tile fastest.  Pair mode: the pair (cluster)
// takes two consecutive row tiles of one filter tile, one per CTA; where the number of row tiles is odd the
// last pair's second CTA repeats the last tile without storing.
template <bool PAIR>
__device__ __forceinline__ bool wunit_at(const WParams& P, int64_t it, uint32_t rank, WUnit& u) {
  // (32-bit arithmetic: the host declines problems of 2^31 units or more; a 64-bit division costs a role
  // some 250 cycles, and every role does this once per unit)
  uint32_t tile;
  if (PAIR) {
    const uint32_t pu = (blockIdx.x >> 1) + (uint32_t)it * (gridDim.x >> 1);
    if (pu >= (uint32_t)P.units) return false;
    const uint32_t half = ((uint32_t)P.tiles + 1u) >> 1;
    const uint32_t nt = pu / half;
    tile = 2u * (pu - nt * half) + rank;
    u.store = tile < (uint32_t)P.tiles;
    if (!u.store) tile = (uint32_t)P.tiles - 1u;
    u.nt = (int32_t)nt;
  } else {
    const uint32_t t = blockIdx.x + (uint32_t)it * gridDim.x;
    if (t >= (uint32_t)P.units) return false;
    if (P.n_ntiles == 1) { tile = t; u.nt = 0; }
    else { tile = t / (uint32_t)P.n_ntiles; u.nt = (int32_t)(t - tile * (uint32_t)P.n_ntiles); }
    u.store = true;
  }
  const uint32_t img = tile / (uint32_t)P.TPI;
  u.img = (int32_t)img;
  u.R0 = (int32_t)(tile - img * (uint32_t)P.TPI) * 128 * P.MH;
  return true;
}
// Source elements [e_lo, e_hi) of a channel plane that the tile starting at position R0 needs, and (im2win
// sources) the last strip row it reads.
template <int FH, bool FUSED>
__device__ __forceinline__ void wtile_range(const WParams& P, int32_t R0, int32_t& e_lo, int32_t& e_hi, int32_t& m_last) {
  m_last = min((R0 + 128 * P.MH - 1) / P.W, P.Ho - 1);
  if (FUSED) {
    e_lo = R0;
    e_hi = min(R0 + P.RX, P.H * P.W);
  } else {
    e_lo = R0 * FH;
    e_hi = (m_last + 1) * P.W * FH;
  }
}

// The MMA-issuing thread's whole life.  A filter stage holds the NBLK blocks of TPS taps.
template <int FH, int FW, bool BF16, int MH, int NBLK, int TPS, bool PAIR, bool TWO>
__device__ __forceinline__ void wmma_role(const WParams& P, SBars* bars, SMisc* misc, uint32_t tmem_base, uint32_t x_sa,
                                          uint32_t b_sa, uint32_t which) {
  Ring xr, br, dr;
  bool ok = true;
  constexpr bool two = TWO;
  const bool bres = P.bres != 0;  // resident filter: the stages of a unit are the ring, filled once
  uint32_t bc = 0;  // filter stages so far: with two issuing threads, thread `which` takes those of its parity
  (void)bc; (void)which;
  SPROF_DECL
  const int32_t lane = (int32_t)(threadIdx.x & 31);
  const uint32_t elect = lane == 0 ? 1u : 0u;  // the whole warp runs this role; one lane issues
  const uint32_t RA = (uint32_t)P.RA, NT = (uint32_t)P.NT, idesc = P.idesc, W = (uint32_t)P.W;
  const uint64_t ad0 = ptx::smem_desc_k_chunkmajor(x_sa, RA * 16u);
  const uint64_t bd0 = ptx::smem_desc_k_sw64(b_sa);
  const uint32_t a_lo0 = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32);
  const uint32_t b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
  const uint32_t x16 = P.x_stage_bytes >> 4, b16 = P.b_stage_bytes >> 4;
  const uint32_t blk16 = (uint32_t)P.NTB * 4u;  // one filter block (NTB rows x 64 bytes) in 16-byte units
  const uint32_t kstep16 = 2u * RA;     // one MMA K step (two chunks) of X in 16-byte units
  const uint32_t x_full0 = ptx::smem_u32(&bars->t_full[0]), x_empty0 = ptx::smem_u32(&bars->t_empty[0]);
  const uint32_t b_full0 = ptx::smem_u32(&bars->b_full[0]), b_empty0 = ptx::smem_u32(&bars->b_empty[0]);
  for (int64_t it = 0; ok; ++it, dr.advance(P.ND)) {
    WUnit u;
    if (!wunit_at<PAIR>(P, it, 0, u)) break;
    SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_empty[dr.idx]), dr.phase ^ 1u, DEV_TIMEOUT_ACC))
    if (!ok) break;
    ptx::tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(dr.idx * MH) * NT;
    uint32_t accum = two ? 1u : 0u;
    for (int32_t xs = 0; xs < P.NXS && ok; ++xs, xr.advance(2)) {
      SPROF_W(1, ok = wait_bar_warp(P, misc, x_full0 + (uint32_t)xr.idx * 8u, xr.phase, DEV_TIMEOUT_A_FULL, 20))
      if (!ok) break;
      uint32_t a_u = a_lo0 + (uint32_t)xr.idx * x16;
#pragma unroll 1
      for (int uu = 0; uu < FH && ok; ++uu, a_u += W) {
#pragma unroll
        for (int v0 = 0; v0 < FW; v0 += TPS) {
          if constexpr (TWO) {
            if ((bc++ & 1u) != which) { br.advance(P.SB); continue; }
          }
          SPROF_W(2, ok = wait_bar_warp(P, misc, b_full0 + (uint32_t)br.idx * 8u, bres ? 0u : br.phase, DEV_TIMEOUT_B_FULL, 20))
          if (!ok) break;
          ptx::tc_fence_after();
          // (block by block: consecutive MMAs onto the same accumulator run faster than alternating ones)
          const uint32_t b_s = b_lo0 + (uint32_t)br.idx * b16;
          const uint32_t accum0 = accum;
#ifdef IM2WIN_PROF
          const long long cm0 = clock64();
#endif
#pragma unroll
          for (int h = 0; h < MH; ++h) {
            uint32_t b_k = b_s;
            uint32_t acc = accum0;
#pragma unroll
            for (int dv = 0; dv < TPS; ++dv) {
              uint32_t a_k = a_u + (uint32_t)(v0 + dv) + (uint32_t)h * 128u;
#pragma unroll
              for (int blk = 0; blk < NBLK; ++blk) {
#pragma unroll
                for (int k2 = 0; k2 < 2; ++k2) {
                  mma_ss_e<BF16, PAIR>(d_tmem + (uint32_t)h * NT, a_k, a_hi, b_k + (uint32_t)k2 * 2u, b_hi, idesc, acc, elect);
                  acc = 1;
                  a_k += kstep16;
                }
                b_k += blk16;
              }
            }
          }
          accum = 1;
#ifdef IM2WIN_PROF
          pw[3] += clock64() - cm0;
#endif
          if (!bres) {
            SPROF_W(4, mma_commit_e<PAIR>(b_empty0 + (uint32_t)br.idx * 8u, elect))
          }
          br.advance(P.SB);
        }
      }
      if (!ok) break;
      mma_commit_e<PAIR>(x_empty0 + (uint32_t)xr.idx * 8u, elect);
    }
    if (!ok) break;
    mma_commit_e<PAIR>(ptx::smem_u32(&bars->acc_full[dr.idx]), elect);
  }
  SPROF_DUMP(1)
}

// SRCK: 0 = fp32 im2win tensor, 1 = untransformed input (fused), 2 = bf16 im2win tensor (BF16 mode).
template <int FH, int FW, bool BF16, int SRCK, bool PAIR>
__global__ void __launch_bounds__(640, 1)
conv_tc_window_kernel(const WParams P, const __grid_constant__ CUtensorMap fmap, const __grid_constant__ CUtensorMap xmap) {
  constexpr bool FUSED = SRCK == 1;
  constexpr bool SRC16 = SRCK == 2;
  static_assert(!SRC16 || BF16, "a 16-bit source feeds the BF16 mode");
  constexpr uint32_t ES = SRC16 ? 2u : 4u;       // bytes per source element
  constexpr int32_t EPC = SRC16 ? 8 : 4;          // source elements per 16-byte chunk
  constexpr int NCH = BF16 ? 8 : 4;               // channels per 16-byte chunk of X

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* const smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  SBars* const bars = reinterpret_cast<SBars*>(smem + P.off_bar);
  SMisc* const misc = reinterpret_cast<SMisc*>(smem + P.off_misc);
  const uint32_t b_sa = ptx::smem_u32(smem), x_sa = b_sa + P.off_x, raw_sa = b_sa + P.off_raw;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;  // pair mode: 0 = the leader, whose thread issues the MMAs of both
  constexpr uint32_t kShare = PAIR ? 2u : 1u;            // CTAs that arrive on the leader's "full"-side barriers
  const bool remote = PAIR && rank != 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxRaw; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->raw_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->raw_empty[i]), kTW);
    }
    for (int i = 0; i < kMaxB; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->b_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->b_empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->t_full[i]), kTW * kShare);
      ptx::mbar_init(ptx::smem_u32(&bars->t_empty[i]), 1u + (uint32_t)P.two);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[i]), 1u + (uint32_t)P.two);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[i]), (uint32_t)P.n_epi * kShare * (P.epi_split < P.NT ? 2u : 1u));
    }
    ptx::fence_mbar_init();
    misc->abort = 0;
  }
  if (warp == 1) {
    if constexpr (PAIR) {  // (the same warp of both CTAs)
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(&misc->tmem_base)), "r"(P.tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), P.tmem_cols);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();  // both CTAs' barriers exist before either signals the other's
  ptx::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  if (P.two) {  // every MMA accumulates: the accumulators start as zeros (one warp per TMEM lane quarter)
    if (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4) {
      const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
      for (uint32_t c = 0; c < P.tmem_cols; c += 16) ptx::tmem_zero_x16(tmem_base + lane_base + c);
      ptx::tmem_wait_st();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
  }

  if (warp == 0) {
    // ================================================================ SOURCE PRODUCER
    using SrcT = typename std::conditional<SRC16, uint16_t, float>::type;
    const SrcT* const xsrc = reinterpret_cast<const SrcT*>(P.src);
    Ring rr;
    int64_t count = 0;
    bool ok = true;
    SPROF_DECL
    for (int64_t it = 0; ok; ++it) {
      WUnit u;
      if (!wunit_at<PAIR>(P, it, rank, u)) break;
      int32_t e_lo, e_hi, m_last;
      wtile_range<FH, FUSED>(P, u.R0, e_lo, e_hi, m_last);
      const int32_t len = e_hi - e_lo;
      const int32_t box_x = (e_lo & ~(EPC - 1)) / (EPC / 2);  // in 8-byte units
      const int32_t nstages = P.NXS * P.NSUB;
      for (int32_t sidx = 0; sidx < nstages && ok; ++sidx, ++count, rr.advance(P.SR)) {
        const int32_t ch0 = sidx * P.GR;
        const uint32_t full = ptx::smem_u32(&bars->raw_full[rr.idx]);
        SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->raw_empty[rr.idx]), rr.phase ^ 1u, DEV_TIMEOUT_RAW_EMPTY, 64))
        if (!ok) break;
        const uint32_t dst0 = raw_sa + (uint32_t)rr.idx * P.raw_stage_bytes;
#ifdef IM2WIN_PROF
        if (P.skip & 4) {
          if (lane == 0) ptx::mbar_arrive(full);
          __syncwarp();
          continue;
        }
#endif
        if (P.box) {
          if (lane == 0) {
            ptx::mbar_arrive_expect_tx(full, P.raw_stage_bytes);
            const uint32_t box_bytes = (uint32_t)(P.GR * P.BXE) * ES;
            for (int32_t bx = 0; bx < P.NBX; ++bx)
              tma_load_2d(dst0 + (uint32_t)bx * box_bytes, &xmap, box_x + bx * (P.BXE / (EPC / 2)), u.img * P.C + ch0, full);
          }
        } else {
          const SrcT* src = nullptr;
          uint32_t dst = 0, bytes = 0;
          if (lane < P.GR) {
            const int64_t start = ((int64_t)u.img * P.C + ch0 + lane) * P.plane + e_lo;
            const int32_t skew = (int32_t)(start & (EPC - 1));
            const int64_t a0 = start - skew;
            int32_t nel = (skew + len + EPC - 1) & ~(EPC - 1);
            dst = dst0 + (uint32_t)(lane * P.BXE) * ES;
            if (a0 + nel > P.n_src) {  // the last 16-byte chunk would pass the end of the tensor
              const int32_t nbulk = (int32_t)((P.n_src - a0) & ~(int64_t)(EPC - 1));
              SrcT* d = reinterpret_cast<SrcT*>(smem + P.off_raw + (size_t)rr.idx * P.raw_stage_bytes) + (size_t)lane * P.BXE;
              for (int64_t e = a0 + nbulk; e < P.n_src; ++e) d[e - a0] = __ldg(xsrc + e);
              nel = nbulk;
            }
            src = xsrc + a0;
            bytes = (uint32_t)nel * ES;
          }
          const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
          if (lane == 0) ptx::mbar_arrive_expect_tx(full, total);
          __syncwarp();
          if (bytes) ptx::bulk_g2s(dst, src, bytes, full);
        }
        __syncwarp();
      }
    }
    SPROF_DUMP(0)
    // every copy issued must have landed before the CTA exits
    for (int64_t c = count > P.SR ? count - P.SR : 0; c < count; ++c)
      wait_bar(P, misc, ptx::smem_u32(&bars->raw_full[c % P.SR]), (uint32_t)(c / P.SR) & 1u, DEV_TIMEOUT_DRAIN);
  } else if (warp == 1 || (warp == 3 && P.two)) {
    // ================================================================ MMA ISSUER (one thread, or one each of warps 1 and 3)
    if (rank == 0) {
      const uint32_t which = warp == 1 ? 0u : 1u;
      const int nblk = P.G / (4 * NCH);
#define WRUN(MHv, NBv, TPv) do { if (!PAIR && P.two) wmma_role<FH, FW, BF16, MHv, NBv, TPv, PAIR, !PAIR>(P, bars, misc, tmem_base, x_sa, b_sa, which); \
                                else wmma_role<FH, FW, BF16, MHv, NBv, TPv, PAIR, false>(P, bars, misc, tmem_base, x_sa, b_sa, which); } while (0)
      if (P.TPS == 1) {
        if (P.MH == 1) { if (nblk == 1) WRUN(1, 1, 1); else WRUN(1, 2, 1); }
        else { if (nblk == 1) WRUN(2, 1, 1); else WRUN(2, 2, 1); }
      } else {
        if (P.MH == 1) { if (nblk == 1) WRUN(1, 1, FW); else WRUN(1, 2, FW); }
        else { if (nblk == 1) WRUN(2, 1, FW); else WRUN(2, 2, FW); }
      }
#undef WRUN
    }
    __syncwarp();
  } else if (warp == 2) {
    // ================================================================ FILTER PRODUCER
    if (lane == 0) {
      Ring br;
      int64_t count = 0;
      bool ok = true;
      SPROF_DECL
      const int32_t bke = BF16 ? 32 : 16;  // elements (channels) per 64-byte filter row
      const int32_t nblk = P.G / bke;
      asm volatile("griddepcontrol.wait;" ::: "memory");  // the filter copy is written by the kernel launched just before
      // Pair mode: this CTA fetches its half of every block's rows, and the bytes of both CTAs are counted on
      // the leader's barrier: the leader announces both halves with its one arrival, the other CTA only
      // issues its copies (its bytes may land before the announcement: the phase cannot complete before the
      // leader's arrival, and the other CTA cannot run a phase ahead, because it needs the stage's release).
      const uint32_t b_full_lead0 = remote ? mapa(ptx::smem_u32(&bars->b_full[0]), 0) : ptx::smem_u32(&bars->b_full[0]);
      for (int64_t it = 0; ok; ++it) {
        WUnit u;
        if (!wunit_at<PAIR>(P, it, rank, u)) break;
        if (P.bres && it > 0) break;  // resident filter: one unit's stages are the whole (single) filter tile
        const int32_t row0 = u.nt * P.NT + (int32_t)rank * P.NTB;
        for (int32_t xs = 0; xs < P.NXS && ok; ++xs) {
          for (int32_t t0 = 0; t0 < FH * FW && ok; t0 += P.TPS, ++count, br.advance(P.SB)) {
            if (!P.bres) {
              SPROF_W(0, ok = wait_bar(P, misc, ptx::smem_u32(&bars->b_empty[br.idx]), br.phase ^ 1u, DEV_TIMEOUT_B_EMPTY))
            }
            if (!ok) break;
            const uint32_t full = b_full_lead0 + (uint32_t)br.idx * 8u;
#ifdef IM2WIN_PROF
            if (P.skip & 2) { if (!remote) ptx::mbar_arrive(full); continue; }
#endif
            if (!remote) ptx::mbar_arrive_expect_tx(full, P.b_stage_bytes * kShare);
            uint32_t dst = b_sa + (uint32_t)br.idx * P.b_stage_bytes;
            for (int32_t dt = 0; dt < P.TPS; ++dt)
              for (int32_t blk = 0; blk < nblk; ++blk, dst += (uint32_t)P.NTB * 64u) {
                if (remote) tma_load_2d_pair(dst, &fmap, xs * P.G + blk * bke, (t0 + dt) * P.Kp + row0, full);
                else tma_load_2d(dst, &fmap, xs * P.G + blk * bke, (t0 + dt) * P.Kp + row0, full);
              }
          }
        }
      }
      SPROF_DUMP(7)
      // every copy issued must have landed before the CTA exits: the stage's release by the MMAs that read it
      // says so (in pair mode the bytes are counted on the leader's barrier, not here)
      if (P.bres) {
        for (int64_t c = 0; c < count; ++c) wait_bar(P, misc, ptx::smem_u32(&bars->b_full[c]), 0u, DEV_TIMEOUT_DRAIN);
      } else {
        for (int64_t c = count > P.SB ? count - P.SB : 0; c < count; ++c)
          wait_bar(P, misc, ptx::smem_u32(&bars->b_empty[c % P.SB]), (uint32_t)(c / P.SB) & 1u, DEV_TIMEOUT_DRAIN);
      }
    }
    __syncwarp();
  } else if (warp >= kTWarp0 && warp < kTWarp0 + kTW) {
    // ================================================================ INTERLEAVERS: staged channel rows -> X
    const int32_t tid = (warp - kTWarp0) * 32 + lane;
    const uint32_t lbo = (uint32_t)P.RA * 16u;
    const int32_t ncb = P.GR / NCH;  // channel blocks (chunks of X) per source stage
    Ring rr, xr;
    bool ok = true;
    SPROF_DECL
    const uint32_t x_full_lead0 = remote ? mapa(ptx::smem_u32(&bars->t_full[0]), 0) : ptx::smem_u32(&bars->t_full[0]);
    uint32_t hphase = 0;  // (epilogue help) phase of the single accumulator buffer's "full" barrier
    for (int64_t it = 0; ok; ++it) {
      WUnit u;
      if (!wunit_at<PAIR>(P, it, rank, u)) break;
      int32_t e_lo, e_hi, m_last;
      wtile_range<FH, FUSED>(P, u.R0, e_lo, e_hi, m_last);
      // this thread's X rows: x = tid + z*256 <-> input position e = R0 + x; where its value sits in a staged channel row
      int32_t sel[kXMax];   // source element relative to e_lo
      bool tv[kXMax];
#pragma unroll
      for (int z = 0; z < kXMax; ++z) {
        const int32_t x = tid + z * (kTW * 32);
        const int32_t e = u.R0 + x;
        tv[z] = false; sel[z] = 0;
        if (x < P.RX) {
          if (FUSED) {
            if (e < P.H * P.W) { tv[z] = true; sel[z] = e - e_lo; }
          } else {
            const int32_t h = e / P.W;
            if (h <= m_last) sel[z] = e * FH - e_lo;
            else if (h - m_last < FH) sel[z] = (e - (h - m_last) * P.W) * FH + (h - m_last) - e_lo;
            else sel[z] = -1;
            tv[z] = sel[z] >= 0;  // (rows outside the staged range feed only positions that are dropped)
            if (!tv[z]) sel[z] = 0;
          }
        }
      }
      // 16-byte phase of the staged ranges: per tile, plus (bulk copies of planes that are not a whole
      // number of chunks) per channel
      const int32_t sk0 = (int32_t)(((int64_t)u.img * P.C * P.plane + e_lo) & (EPC - 1));
      uint32_t soff[kXMax];
#pragma unroll
      for (int z = 0; z < kXMax; ++z) {
        const int32_t ei = sel[z] + (P.pm ? 0 : sk0);
        const int32_t bx = ei / P.BXE;
        soff[z] = (uint32_t)(bx * P.GR * P.BXE + (ei - bx * P.BXE)) * ES;
      }
      for (int32_t xs = 0; xs < P.NXS && ok; ++xs, xr.advance(2)) {
        const uint32_t x_stage = x_sa + (uint32_t)xr.idx * P.x_stage_bytes;
        for (int32_t sub = 0; sub < P.NSUB && ok; ++sub, rr.advance(P.SR)) {
          SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->raw_full[rr.idx]), rr.phase, DEV_TIMEOUT_RAW_FULL))
          if (!ok) break;
          if (sub == 0) {
            SPROF_W(1, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->t_empty[xr.idx]), xr.phase ^ 1u, DEV_TIMEOUT_A_EMPTY))
            if (!ok) break;
          }
#ifdef IM2WIN_PROF
          const long long cw0 = clock64();
#endif
          const uint32_t rs = raw_sa + (uint32_t)rr.idx * P.raw_stage_bytes;
          const int32_t ch0 = (xs * P.NSUB + sub) * P.GR;
          const uint32_t x_sub = x_stage + (uint32_t)(sub * ncb) * lbo;
#pragma unroll
          for (int z = 0; z < kXMax; ++z) {
#ifdef IM2WIN_PROF
            if (P.skip & 1) continue;
#endif
            if (tv[z]) {
              const uint32_t d0 = x_sub + (uint32_t)(tid + z * (kTW * 32)) * 16u;
              for (int32_t cb = 0; cb < ncb; ++cb) {
                uint32_t val[NCH];
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                  const int32_t ch = cb * NCH + c;
                  const int32_t sk = P.pm ? ((sk0 + (ch0 + ch) * P.pm) & (EPC - 1)) : 0;
                  const uint32_t a = rs + soff[z] + (uint32_t)(ch * P.BXE + sk) * ES;
                  val[c] = SRC16 ? lds_u16(a) : lds_u32(a);
                }
                const uint32_t d = d0 + (uint32_t)cb * lbo;
                if constexpr (!BF16) {
                  sts_v4(d, val[0], val[1], val[2], val[3]);
                } else if constexpr (SRC16) {
                  sts_v4(d, val[0] | (val[1] << 16), val[2] | (val[3] << 16), val[4] | (val[5] << 16), val[6] | (val[7] << 16));
                } else {
                  sts_v4(d, ptx::pack_bf16x2(__uint_as_float(val[0]), __uint_as_float(val[1])),
                         ptx::pack_bf16x2(__uint_as_float(val[2]), __uint_as_float(val[3])),
                         ptx::pack_bf16x2(__uint_as_float(val[4]), __uint_as_float(val[5])),
                         ptx::pack_bf16x2(__uint_as_float(val[6]), __uint_as_float(val[7])));
                }
              }
            }
          }
          const bool last = sub == P.NSUB - 1;
          if (last) ptx::fence_proxy_async_smem();  // this thread's X writes -> visible to the tensor core
          __syncwarp();
#ifdef IM2WIN_PROF
          pw[2] += clock64() - cw0;
#endif
          if (lane == 0) {
            ptx::mbar_arrive(ptx::smem_u32(&bars->raw_empty[rr.idx]));
            if (last) {
              if (remote) arrive_cluster(x_full_lead0 + (uint32_t)xr.idx * 8u);
              else ptx::mbar_arrive(x_full_lead0 + (uint32_t)xr.idx * 8u);
            }
          }
        }
      }
      // One accumulator buffer: the next unit's MMAs cannot start before this unit's results are stored, so
      // this warp stores the upper columns of its TMEM lane quarter meanwhile.
      if (ok && P.epi_split < P.NT) {
        const int32_t hh = (warp - kTWarp0) >> 2, q4 = warp & 3;
        ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_full[0]), hphase, DEV_TIMEOUT_ACC, 128);
        if (!ok) break;
        hphase ^= 1u;
        ptx::tc_fence_after();
        if (hh < P.MH) {
          const int32_t rho = u.R0 + hh * 128 + q4 * 32 + lane;
          const int32_t m = rho / P.W, q = rho - m * P.W;
          const bool valid = u.store && rho < P.RPI && q < P.Wo;
          const int32_t n0 = u.nt * P.NT;
          const int64_t HoWo = (int64_t)P.Ho * P.Wo;
          float* const orow = P.nhwc ? P.out + ((int64_t)u.img * HoWo + (int64_t)m * P.Wo + q) * P.K + n0
                                     : P.out + ((int64_t)u.img * P.K + n0) * HoWo + (int64_t)m * P.Wo + q;
          store_columns(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(hh * P.NT), orow, P.nhwc ? 1 : HoWo, P.epi_split, P.NT,
                        P.K - n0, valid, P.two != 0, P.nhwc && (P.K & 3) == 0);
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            const uint32_t ae = ptx::smem_u32(&bars->acc_empty[0]);
            if (remote) arrive_cluster(mapa(ae, 0));
            else ptx::mbar_arrive(ae);
          }
        }
      }
    }
    if (warp == kTWarp0) { SPROF_DUMP(2) }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + P.n_epi) {
    // ================================================================ EPILOGUE: TMEM -> NCHW
    const int32_t h0 = (warp - kEpiWarp0) >> 2, q4 = warp & 3;  // (kEpiWarp0 is a multiple of 4: warp & 3 = TMEM lane quarter)
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    Ring dr;
    bool ok = true;
    SPROF_DECL
    const int64_t eHoWo = (int64_t)P.Ho * P.Wo;
    const uint32_t acc_empty_lead0 = remote ? mapa(ptx::smem_u32(&bars->acc_empty[0]), 0) : ptx::smem_u32(&bars->acc_empty[0]);
    for (int64_t it = 0; ok; ++it, dr.advance(P.ND)) {
      WUnit u;
      if (!wunit_at<PAIR>(P, it, rank, u)) break;
      const int32_t n0 = u.nt * P.NT;
      SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_full[dr.idx]), dr.phase, DEV_TIMEOUT_ACC, 128))
      if (!ok) break;
      ptx::tc_fence_after();
      for (int32_t h = h0; h < P.MH; h += 2) {
        const int32_t rho = u.R0 + h * 128 + q4 * 32 + lane;
        const int32_t m = rho / P.W, q = rho - m * P.W;
        const bool valid = u.store && rho < P.RPI && q < P.Wo;
        float* const orow = P.nhwc ? P.out + ((int64_t)u.img * eHoWo + (int64_t)m * P.Wo + q) * P.K + n0
                                   : P.out + ((int64_t)u.img * P.K + n0) * eHoWo + (int64_t)m * P.Wo + q;
        const uint32_t d_tmem = tmem_base + lane_base + (uint32_t)((dr.idx * P.MH + h) * P.NT);
        store_columns(d_tmem, orow, P.nhwc ? 1 : eHoWo, 0, P.epi_split, P.K - n0, valid, P.two != 0, P.nhwc && (P.K & 3) == 0);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (remote) arrive_cluster(acc_empty_lead0 + (uint32_t)dr.idx * 8u);
        else ptx::mbar_arrive(acc_empty_lead0 + (uint32_t)dr.idx * 8u);
      }
    }
    if (warp == kEpiWarp0) { SPROF_DUMP(6) }
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();  // neither CTA leaves while the other may still signal its barriers
  if (warp == 1) {
    ptx::tc_fence_after();
    if constexpr (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(P.tmem_cols) : "memory");
    else ptx::tmem_dealloc(tmem_base, P.tmem_cols);
  }
}

// Tap-major copy of the filter for the TMA-streamed B operand:
//   F9[t][j][r] = F[j][r][u][v],  t = u*Fw + v   (j < K; rows K..Kp-1 are zero), fp32 or bf16 (nearest even).
// One CTA per (filter j, block of 128 channels): its 128*Fh*Fw values pass through shared memory, so that both
// the reads and the writes are contiguous, and every CTA is one load - store round trip (the convolution
// kernel's first MMA waits for this copy: its latency counts).
constexpr int kPrepCh = 128, kPrepTaps = 25;
template <bool BF16>
__global__ void __launch_bounds__(128) filter_tap_rows_kernel(const float* __restrict__ f, void* __restrict__ o, int32_t K,
                                                              int32_t Kp, int32_t C, int32_t taps) {
  // the convolution kernel that follows may start its prologue now (it waits for this grid's completion
  // before it reads the copy)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ float sm[kPrepCh * kPrepTaps];
  const int32_t j = (int32_t)blockIdx.x, tid = (int32_t)threadIdx.x;
  const int32_t c0 = (int32_t)blockIdx.y * kPrepCh;
  const int32_t nc = min(kPrepCh, C - c0);
  const float* fj = f + ((int64_t)j * C + c0) * taps;
  const int32_t n = nc * taps;
  if (j < K) {
    float v[kPrepTaps];
#pragma unroll
    for (int q = 0; q < kPrepTaps; ++q) {  // (all loads in flight before the first use)
      const int32_t i = tid + q * 128;
      v[q] = (q < taps && i < n) ? __ldg(fj + i) : 0.f;
    }
#pragma unroll
    for (int q = 0; q < kPrepTaps; ++q) {
      const int32_t i = tid + q * 128;
      if (q < taps && i < n) sm[i] = v[q];
    }
  } else {
    for (int32_t i = tid; i < n; i += 128) sm[i] = 0.f;
  }
  __syncthreads();
  if (tid < nc) {
    for (int32_t t = 0; t < taps; ++t) {
      const float x = sm[tid * taps + t];
      const int64_t oi = ((int64_t)t * Kp + j) * C + c0 + tid;
      if (BF16) static_cast<__nv_bfloat16*>(o)[oi] = __float2bfloat16_rn(x);
      else static_cast<float*>(o)[oi] = x;
    }
  }
}

// ---------------------------------------------------------------------------------------------- host side

struct WPlan {
  WParams P;
  size_t smem_bytes, scratch_bytes;
  int threads;
};

// Fills the launch parameters; IM2WIN_EUNSUPPORTED where the kernel does not apply.
template <int FH, int FW, bool BF16, int SRCK>
int make_wplan(const Geometry& g, WPlan* pl, int pair, int mh_fixed) {
  constexpr int NCH = BF16 ? 8 : 4;
  constexpr int64_t ES = SRCK == 2 ? 2 : 4;
  constexpr int64_t EPC = 16 / ES;
  static_assert(FH * FW <= kPrepTaps, "filter-copy kernel's shared buffer");
  WParams& P = pl->P;
  P = WParams{};
  if (g.s != 1) return IM2WIN_EUNSUPPORTED;
  const int gmin = 4 * NCH;  // one 64-byte filter block
  if (g.C % gmin != 0) return IM2WIN_EUNSUPPORTED;
  if (g.HoWo > (1 << 28) || (int64_t)g.H * g.W > (1 << 26)) return IM2WIN_EUNSUPPORTED;
  P.C = g.C; P.K = g.K; P.Ho = g.Ho; P.Wo = g.Wo; P.W = g.W; P.H = g.H;
  P.nhwc = g.out_nhwc;
  P.RPI = g.Ho * g.W;
  P.n_ntiles = (g.K + 255) / 256;
  P.NT = ((g.K + P.n_ntiles - 1) / P.n_ntiles + 15) / 16 * 16;
  P.Kp = P.n_ntiles * P.NT;
  if (pair && P.NT % 32 != 0) return IM2WIN_EUNSUPPORTED;  // (each CTA's half of the filter rows: a multiple of 16)
  P.pair = pair;
  // Two issuing threads where one is the bound: 64-column MMAs take the tensor pipe 54 cycles (their 128-row A
  // operand is fetched for only 64 columns) but one thread 64 or more to issue; measured: 64-filter layers gain
  // 10-20 %, wider tiles nothing.
  P.two = (!pair && (knobs().window_two == 1 || (knobs().window_two == 0 && P.NT <= 64))) ? 1 : 0;
  P.NTB = pair ? P.NT / 2 : P.NT;
  if (SRCK == 1) { P.plane = (int64_t)g.H * g.W; P.n_src = g.n_in; }
  else { P.plane = g.HoL; P.n_src = g.n_win; }
  P.pm = (int32_t)(P.plane % EPC);
  const int64_t cap = 227 * 1024 - 1024 - (1024 + 128 + 16) - (int64_t)((sizeof(SBars) + 15) / 16 * 16) - 64;
  P.MH = mh_fixed;
  if (P.MH < 1 || P.MH > 2 || P.MH * P.NT > 512) return IM2WIN_EUNSUPPORTED;
  P.RX = 128 * P.MH + (FH - 1) * g.W + FW - 1;
  if (P.RX > kXMax * kTW * 32) return IM2WIN_EUNSUPPORTED;
  P.RA = (P.RX + 7) / 8 * 8;
  P.TPI = (P.RPI + 128 * P.MH - 1) / (128 * P.MH);
  P.tiles = (int64_t)g.N * P.TPI;
  P.units = pair ? ((P.tiles + 1) / 2) * P.n_ntiles : P.tiles * P.n_ntiles;
  if (P.tiles * P.n_ntiles >= (1ll << 31) - 65536) return IM2WIN_EUNSUPPORTED;  // (the kernel's unit arithmetic is 32-bit)
  P.ND = 512 / (P.MH * P.NT) >= 2 ? 2 : 1;
  P.n_epi = 4 * (P.MH < 2 ? P.MH : 2);
  // one accumulator buffer: the interleaver warps (two sets of four, one per block) store the upper half of the
  // columns; with one block per tile only the first set could help, so the epilogue warps keep all columns
  P.epi_split = (P.ND == 1 && P.MH == 2 && P.NT >= 64 && !knobs().window_nohelp) ? (P.NT / 2 + 15) / 16 * 16 : P.NT;
  // source elements of one channel a tile needs at most, plus the 16-byte phase in front
  const int64_t len_max = SRCK == 1 ? P.RX : (int64_t)FH * (128 * P.MH + g.W);
  int64_t cp = len_max + 2 * EPC;
  const int64_t cp_align = 32 / ES;
  cp = (cp + cp_align - 1) / cp_align * cp_align;
  // The split of shared memory: filter blocks per X stage (16/32 or 32/64 channels), taps per filter stage
  // (one filter row, or one tap) and channels per source stage, tried in an order taken from measurements
  // (every combination, on six layers, both modes, three sources): a whole filter row per stage wherever two
  // such stages fit (one wait and one release of the issuing thread per Fw taps); two blocks per X stage for
  // the fused source, whose staged rows are a third of the im2win tensor's; sixteen channels per source stage,
  // eight where the fp32 im2win tensor's rows are long.  The first combination that leaves two stages for each
  // ring wins; what is left goes to the two rings by the latency each has to cover.
  const int64_t blk_bytes = (int64_t)P.NTB * 64;
  const double mma_cyc = P.NT / 2.0 > 54.0 ? P.NT / 2.0 : 54.0;
  const int forced_plan = knobs().window_plan;  // test build: nblk | taps-per-stage << 4 | channels per source stage << 8
  struct Try { int nblk, tps, gr; };
  const Try order_fused[] = {{2, FW, 16}, {2, FW, 8}, {2, 1, 32}, {2, 1, 16}, {1, FW, 32}, {1, FW, 16}, {1, 1, 16}, {1, 1, 8}, {1, 1, 4}};
  const Try order_win[] = {{1, FW, 16}, {1, FW, 8}, {2, 1, 8}, {1, 1, 8}, {1, 1, 4}, {1, 1, 16}};
  const Try order_win16[] = {{1, FW, 32}, {1, FW, 16}, {2, 1, 16}, {1, 1, 16}, {1, 1, 8}, {1, 1, 32}};
  const Try* order_tail = SRCK == 1 ? order_fused : (SRCK == 2 ? order_win16 : order_win);
  const int n_tail = SRCK == 1 ? 9 : 6;
  // In front of those, the measured exceptions: 256-wide filter tiles want one filter block per X stage (a stage of
  // two blocks x Fw taps x 256 rows is 96 KB, and two of them leave the other rings too little): fused with two
  // 128-row blocks {1,Fw,16} (the deep 3x3 layers in BF16 mode: 50 -> 43, 62 -> 56, 83 -> 74 us), with one block
  // (images under 128 positions) {2,Fw,32}; from the fp32 tensor eight or four channels per source stage for tiles
  // of 192 and more (TF32: 108 -> 98, 151 -> 134 us on the 384-filter layers).
  Try order_all[12];
  int n_order = 0;
  if (SRCK == 1) {
    if (P.NT >= 256) order_all[n_order++] = P.MH == 2 ? Try{1, FW, 16} : Try{2, FW, 32};
  } else if (SRCK == 0 && P.MH == 2) {  // (images of a single block keep the general order: measured)
    if (BF16) {
      if (P.NT >= 256 && FH == 3) order_all[n_order++] = Try{1, 1, 16};
      if (P.NT >= 192) order_all[n_order++] = Try{1, FW, 8};
    } else {
      if (P.NT >= 256 && FH == 3) order_all[n_order++] = Try{1, FW, 4};
      if (P.NT >= 192) order_all[n_order++] = Try{1, FW, 8};
    }
  }
  for (int t = 0; t < n_tail; ++t) order_all[n_order++] = order_tail[t];
  const Try* order = order_all;
  // (resident only where source stages of sixteen channels still fit: with smaller ones it was measured slower;
  // one filter block per X stage first: `resnet3x3` BF16 fused 71 -> 60 us)
  const Try order_res[] = {{1, FW, 32}, {1, FW, 16}, {2, FW, 32}, {2, FW, 16}};
  bool found = false;
  for (int pass = 0; pass < 2 && !found; ++pass) {  // first the resident filter, then the streamed one
    if (pass == 0 && (pair || P.n_ntiles != 1 || knobs().window_bres == 2)) continue;
    if (pass == 1 && knobs().window_bres == 1) break;  // (test build: resident or nothing)
    const Try* ord = pass == 0 ? order_res : order;
    const int n_ord = pass == 0 ? 4 : n_order;
    for (int t = 0; t < n_ord && !found; ++t) {
      int nblk = ord[t].nblk, tps = ord[t].tps, gr = ord[t].gr;
      if (forced_plan) {
        if (t > 0) break;
        nblk = forced_plan & 15; tps = (forced_plan >> 4) & 15; gr = forced_plan >> 8;
        if (nblk < 1 || nblk > 2 || (tps != 1 && tps != FW) || gr < NCH) return IM2WIN_EUNSUPPORTED;
      }
      const int G = nblk * gmin;
      if (g.C % G != 0 || G % gr != 0 || gr > 32 || gr < NCH) continue;
      const uint32_t x_stage_bytes = (uint32_t)((G / NCH) * P.RA * 16);
      const int64_t left = cap - 2 * (int64_t)x_stage_bytes;
      const int64_t b_stage_bytes = (int64_t)tps * nblk * blk_bytes;
      // boxes of at most 2 KB per channel row
      int64_t nbx = 1, bxe = cp;
      const bool box_ok = P.pm == 0 && gr >= 4 && encode_fn() != nullptr && (int64_t)g.N * g.C <= INT32_MAX && !knobs().no_box;
      if (box_ok) {
        nbx = (cp * ES + 2047) / 2048;
        bxe = (cp + nbx - 1) / nbx;
        bxe = (bxe + cp_align - 1) / cp_align * cp_align;
      }
      const int64_t raw_bytes = (int64_t)gr * nbx * bxe * ES;
      if (raw_bytes % 128 != 0 || bxe * ES > 65536) continue;
      // Resident filter: a single filter tile whose Fh*Fw*C/G stages all fit beside the X stages and two source
      // stages stays in shared memory for the whole kernel (no filter stream, no release traffic).
      const int64_t n_res = (int64_t)(g.C / G) * (FH * FW / tps);
      const bool try_res = pass == 0 && n_res <= kMaxB && n_res * b_stage_bytes + 2 * raw_bytes <= left;
      if (pass == 0 && !try_res) continue;
      if (try_res) {
        int64_t sr = 2;
        while (sr < kMaxRaw && n_res * b_stage_bytes + (sr + 1) * raw_bytes <= left) ++sr;
        P.G = G; P.NXS = g.C / G; P.x_stage_bytes = x_stage_bytes;
        P.TPS = tps; P.b_stage_bytes = (uint32_t)b_stage_bytes;
        P.GR = gr; P.NSUB = G / gr; P.box = box_ok ? 1 : 0;
        P.NBX = (int32_t)nbx; P.BXE = (int32_t)bxe; P.raw_stage_bytes = (uint32_t)raw_bytes;
        P.SB = (int32_t)n_res; P.SR = (int32_t)sr; P.bres = 1;
        found = true;
        break;
      }
      const int64_t min_b = 2;
      if (min_b * b_stage_bytes + 2 * raw_bytes > left) continue;
      const int nsub = G / gr;
      const double b_stage_cyc = (double)tps * nblk * 2 * P.MH * mma_cyc;
      const double raw_stage_cyc = (double)FH * FW * nblk * 2 * P.MH * mma_cyc / nsub;
      int64_t sb = min_b, sr = 2;
      while (true) {  // one more stage for the ring that covers less of the latency (about 2500 cycles), while it fits
        const bool can_b = sb < kMaxB && (sb + 1) * b_stage_bytes + sr * raw_bytes <= left;
        const bool can_r = sr < kMaxRaw && sb * b_stage_bytes + (sr + 1) * raw_bytes <= left;
        if (!can_b && !can_r) break;
        const double cover_b = (double)(sb - 1) * b_stage_cyc, cover_r = (double)(sr - 1) * raw_stage_cyc;
        if (can_b && (!can_r || cover_b <= cover_r)) ++sb;
        else ++sr;
      }
      P.G = G; P.NXS = g.C / G; P.x_stage_bytes = x_stage_bytes;
      P.TPS = tps; P.b_stage_bytes = (uint32_t)b_stage_bytes;
      P.GR = gr; P.NSUB = nsub; P.box = box_ok ? 1 : 0;
      P.NBX = (int32_t)nbx; P.BXE = (int32_t)bxe; P.raw_stage_bytes = (uint32_t)raw_bytes;
      P.SB = (int32_t)sb; P.SR = (int32_t)sr;
      found = true;
    }
  }
  if (!found) return IM2WIN_EUNSUPPORTED;
  uint32_t off = (uint32_t)(P.SB * P.b_stage_bytes);
  off = (off + 1023) / 1024 * 1024;
  P.off_x = off; off += 2 * P.x_stage_bytes;
  off = (off + 127) / 128 * 128;
  P.off_raw = off; off += (uint32_t)P.SR * P.raw_stage_bytes;
  off = (off + 15) / 16 * 16;
  P.off_bar = off; off += (uint32_t)((sizeof(SBars) + 15) / 16 * 16);
  P.off_misc = off; off += 64;
  pl->smem_bytes = off + 1024;
  if (pl->smem_bytes > 227 * 1024) return IM2WIN_EUNSUPPORTED;
  const int32_t cols = P.ND * P.MH * P.NT;
  P.tmem_cols = 32;
  while ((int32_t)P.tmem_cols < cols) P.tmem_cols *= 2;
  P.idesc = ptx::make_idesc(pair ? 256 : 128, P.NT, BF16 ? 1 : 2);
  pl->scratch_bytes = (size_t)FH * FW * P.Kp * (size_t)g.C * (BF16 ? 2 : 4);
  pl->threads = (kEpiWarp0 + P.n_epi) * 32;
  return IM2WIN_OK;
}

// Which variant a problem gets (knobs override).  CTA pairs (each CTA fetches half the filter rows) where they
// were measured faster than single CTAs: the 5x5 layers in BF16 mode with 256-wide filter tiles (25 taps make
// the filter stream the largest consumer of shared-memory bandwidth), with one block per tile so that two
// accumulator buffers remain; and 192-wide tiles in TF32 mode from the fused source and in BF16 mode from the
// bf16 tensor.  Elsewhere a pair's MMAs, which cost the issuing thread about twice as long, lose more than the
// halved filter traffic gains.
// Rows per tile: the number of 128-row blocks that gives the least estimated time: rounds of units over the
// SMs (or pairs) x (blocks per unit + the fixed part of a unit, measured as about two blocks); ties go to the
// taller tile.
template <int FH, int FW, bool BF16, int SRCK>
int choose_wplan(const Geometry& g, WPlan* best) {
  const int forced = knobs().window_mh & 255;
  const int nt = (((g.K + (g.K + 255) / 256 - 1) / ((g.K + 255) / 256)) + 15) / 16 * 16;
  int pair = 0;
  if (FH == 5) pair = BF16 && nt >= 192 && (int64_t)g.Ho * g.W >= 640;  // (faster on the 27x27-output 5x5 layer, slower on the 20x20 one)
  else if (nt >= 192 && nt < 256) pair = (SRCK == 1 && !BF16) || SRCK == 2;
  if (knobs().window_pair == 1) pair = 1;
  if (knobs().window_pair == 2) pair = 0;
  for (int attempt = 0; attempt < 2; ++attempt, pair = 1 - pair) {
    if (attempt == 1 && knobs().window_pair) break;  // (a forced variant that does not fit: unsupported)
    int64_t best_cost = -1;
    WPlan cand;
    const int64_t slots = pair ? sm_count() / 2 : sm_count();
    for (int mh = 2; mh >= 1; mh /= 2) {  // (four blocks per tile were measured too: never faster, and they leave the rings less room)
      if (forced && mh != forced) continue;
      if (!forced && pair && FH == 5 && mh != 1) continue;
      if (make_wplan<FH, FW, BF16, SRCK>(g, &cand, pair, mh) != IM2WIN_OK) continue;
      if (!forced && mh > 1 && (int64_t)g.Ho * g.W <= 128 * (mh / 2)) continue;  // the image fits fewer blocks
      // tiles of up to 128 filters keep two accumulator buffers (the epilogue overlaps the next unit); wider
      // ones gain more from the second block (each filter stage feeds two MMAs)
      if (!forced && cand.P.NT <= 128 && cand.P.ND < 2) continue;
      const int64_t rounds = (cand.P.units + slots - 1) / slots;
      const int64_t cost = rounds * (mh + 2);  // (a unit costs about two blocks' time beside its blocks: measured)
      if (best_cost < 0 || cost < best_cost) { best_cost = cost; *best = cand; }
    }
    if (best_cost >= 0) return IM2WIN_OK;
  }
  return IM2WIN_EUNSUPPORTED;
}

// Whether this kernel is expected to beat the strip-matrix and the persistent kernel: rules read off a
// measured table (B200, batch 128, every stride-1 3x3 / 5x5 layer of the benchmark lists, three source kinds,
// both modes).  Its strengths: the staged bytes and the interleaving work are a third of the strip-matrix
// kernel's, and it has no per-thread window loads (the persistent kernel's bound on deep layers in BF16 mode).
// In TF32 mode and for the fused source the 256-wide filter tiles on images of more than one block stay with
// the strip-matrix kernel's CTA pairs; TF32 layers of 64 filters from the fp32 im2win tensor stay with the
// persistent kernel (a 64-column MMA from shared memory takes 54 cycles, that kernel's from tensor memory 32,
// and the tensor's staged bytes are three times the input's), the same layers fused come here; and where the
// persistent kernel finishes in a single wave of tiles that span images (small images, one filter tile) that
// kernel stays.
template <int FH, int FW, bool BF16, int SRCK>
bool window_preferred(const Geometry& g, const WParams& P) {
  const int nsm = sm_count();
  if (P.units * 2 <= nsm) return false;  // under-filled launches: the persistent kernel's reduction slices
  if (FH == 5) return BF16 || (SRCK == 0 && P.RPI < 640);  // 5x5 layers: 25 taps of one staged tile (TF32: from the tensor, smaller images)
  const int64_t span_tiles = (g.Mtot + 127) / 128;
  if (P.n_ntiles == 1 && span_tiles <= nsm && P.NT > 128) return false;  // one wave of the persistent kernel
  if (!BF16) {
    if (SRCK == 1) return P.NT <= 64 || (g.C >= 128 && P.NT >= 128 && P.NT <= 192);
    return P.NT > 64 && P.NT <= 192;
  }
  if (SRCK == 2) return P.NT <= 192 || P.RPI >= 128;                   // bf16 im2win tensor
  if (SRCK == 1) return g.C >= 128 || P.NT <= 64;                      // fused
  return g.C >= 128;                                                    // fp32 im2win tensor
}

template <int FH, int FW, bool BF16, int SRCK, bool PAIR>
int launch_wkernel(const WParams& P, const WPlan& pl, const CUtensorMap& fmap, const CUtensorMap& xmap, cudaStream_t st) {
  auto kern = conv_tc_window_kernel<FH, FW, BF16, SRCK, PAIR>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes) != cudaSuccess) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3((unsigned)pl.threads);
  cfg.dynamicSmemBytes = pl.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  // programmatic dependent launch: the prologue and the first source copies overlap the filter-copy kernel
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int64_t grid;
  if (PAIR) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    cfg.gridDim = dim3((unsigned)(sm_count() / 2 * 2));
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg) != cudaSuccess || max_clusters < 1) {
      cudaGetLastError();
      return IM2WIN_EUNSUPPORTED;
    }
    int64_t pairs = sm_count() / 2;
    if (pairs > max_clusters) pairs = max_clusters;
    if (pairs > P.units) pairs = P.units;
    grid = 2 * pairs;
  } else {
    grid = P.units < sm_count() ? P.units : sm_count();
  }
  cfg.gridDim = dim3((unsigned)grid);
  if (cudaLaunchKernelEx(&cfg, kern, P, fmap, xmap) != cudaSuccess) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  return IM2WIN_OK;
}

template <int FH, int FW, bool BF16, int SRCK>
int launch_window(const void* src, const float* f, float* out, const Geometry& g, cudaStream_t st, Scratch scratch,
                  bool even_if_slower) {
  WPlan pl;
  int rc = choose_wplan<FH, FW, BF16, SRCK>(g, &pl);
  if (rc != IM2WIN_OK) return rc;
  WParams& P = pl.P;
  if (!even_if_slower && !knobs().force_window && !window_preferred<FH, FW, BF16, SRCK>(g, P)) return IM2WIN_EUNSUPPORTED;
  if (!scratch.ptr || scratch.bytes < pl.scratch_bytes || (reinterpret_cast<uintptr_t>(scratch.ptr) & 15u)) return IM2WIN_EUNSUPPORTED;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return IM2WIN_EUNSUPPORTED;
  P.src = src; P.out = out;
#ifdef IM2WIN_PROF
  P.prof = g_prof;
  P.skip = knobs().window_mh >> 8;   // (profiling build: ablation bits ride in the upper bits of the tile-height switch)
#endif
  P.status = device_status_word();
  if (!P.status) return IM2WIN_ECUDA;
  constexpr int64_t ES = SRCK == 2 ? 2 : 4;
  CUtensorMap fmap, xmap;
  memset(&fmap, 0, sizeof(fmap));
  memset(&xmap, 0, sizeof(xmap));
  {
    const cuuint64_t gdim[2] = {(cuuint64_t)g.C, (cuuint64_t)FH * FW * P.Kp};
    const cuuint64_t gstr[1] = {(cuuint64_t)g.C * (BF16 ? 2 : 4)};
    const cuuint32_t box[2] = {(cuuint32_t)(BF16 ? 32 : 16), (cuuint32_t)P.NTB};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&fmap, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, scratch.ptr, gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return IM2WIN_EUNSUPPORTED;
  }
  if (P.box) {
    // source planes as rows of 8-byte elements (the box then starts on any 16-byte boundary)
    const cuuint64_t gdim[2] = {(cuuint64_t)(P.plane * ES / 8), (cuuint64_t)g.N * g.C};
    const cuuint64_t gstr[1] = {(cuuint64_t)P.plane * ES};
    const cuuint32_t box[2] = {(cuuint32_t)(P.BXE * ES / 8), (cuuint32_t)P.GR};
    const cuuint32_t estr[2] = {1, 1};
    if ((P.plane * ES) % 16 != 0 || box[0] > 256 || box[1] > 256 ||
        enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_INT64, 2, const_cast<void*>(src), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      // bulk copies instead: one row of CP elements per channel
      P.box = 0;
      P.BXE = P.NBX * P.BXE;
      P.NBX = 1;
    }
  }
  const dim3 pgrid((unsigned)P.Kp, (unsigned)((g.C + kPrepCh - 1) / kPrepCh));
  if (BF16) filter_tap_rows_kernel<true><<<pgrid, 128, 0, st>>>(f, scratch.ptr, g.K, P.Kp, g.C, FH * FW);
  else filter_tap_rows_kernel<false><<<pgrid, 128, 0, st>>>(f, scratch.ptr, g.K, P.Kp, g.C, FH * FW);
  if (cudaGetLastError() != cudaSuccess) return IM2WIN_ECUDA;
  rc = P.pair ? launch_wkernel<FH, FW, BF16, SRCK, true>(P, pl, fmap, xmap, st) : launch_wkernel<FH, FW, BF16, SRCK, false>(P, pl, fmap, xmap, st);
  if (rc != IM2WIN_OK) return rc;
  note_kernel(KERNEL_WINDOW);
  {
    const int v[8] = {P.MH + 10 * P.pair + 100 * P.bres, P.G, P.TPS, P.GR, P.SB, P.SR, P.ND, P.box * 100 + P.NBX};
    note_plan(v, 8);
  }
  return IM2WIN_OK;
}

template <int FH, int FW>
int launch_window_fs(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st, Scratch scratch,
                     int src_kind, bool eis) {
  const bool bf16 = mode == IM2WIN_MODE_BF16;
  if (src_kind == 2) return bf16 ? launch_window<FH, FW, true, 2>(src, f, out, g, st, scratch, eis) : IM2WIN_EUNSUPPORTED;
  if (src_kind == 1)
    return bf16 ? launch_window<FH, FW, true, 1>(src, f, out, g, st, scratch, eis) : launch_window<FH, FW, false, 1>(src, f, out, g, st, scratch, eis);
  return bf16 ? launch_window<FH, FW, true, 0>(src, f, out, g, st, scratch, eis) : launch_window<FH, FW, false, 0>(src, f, out, g, st, scratch, eis);
}

template <int FH, int FW>
size_t wscratch_fs(const Geometry& g, int mode, int src_kind) {
  WPlan pl;
  const bool bf16 = mode == IM2WIN_MODE_BF16;
  int rc;
  if (src_kind == 2) rc = bf16 ? choose_wplan<FH, FW, true, 2>(g, &pl) : IM2WIN_EUNSUPPORTED;
  else if (src_kind == 1) rc = bf16 ? choose_wplan<FH, FW, true, 1>(g, &pl) : choose_wplan<FH, FW, false, 1>(g, &pl);
  else rc = bf16 ? choose_wplan<FH, FW, true, 0>(g, &pl) : choose_wplan<FH, FW, false, 0>(g, &pl);
  return rc == IM2WIN_OK ? (pl.scratch_bytes + 255) / 256 * 256 : 0;
}

}  // namespace

int launch_conv_tc_window(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                          Scratch scratch, int src_kind, bool out_bf16, bool even_if_slower) {
  if (out_bf16) return IM2WIN_EUNSUPPORTED;  // fp32 epilogue only
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16) return IM2WIN_EUNSUPPORTED;
  if (g.s != 1 || knobs().no_window) return IM2WIN_EUNSUPPORTED;
  if (g.Fh == 3 && g.Fw == 3) return launch_window_fs<3, 3>(src, f, out, g, mode, st, scratch, src_kind, even_if_slower);
  if (g.Fh == 5 && g.Fw == 5) return launch_window_fs<5, 5>(src, f, out, g, mode, st, scratch, src_kind, even_if_slower);
  return IM2WIN_EUNSUPPORTED;
}

size_t window_scratch_bytes(const Geometry& g, int mode, int src_kind) {
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16) return 0;
  if (g.s != 1) return 0;
  if (g.Fh == 3 && g.Fw == 3) return wscratch_fs<3, 3>(g, mode, src_kind);
  if (g.Fh == 5 && g.Fw == 5) return wscratch_fs<5, 5>(g, mode, src_kind);
  return 0;
}

}  // namespace im2win
