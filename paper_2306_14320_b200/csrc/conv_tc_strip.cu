// im2win-based convolution (Algorithm 2) on the sm_100a tensor cores: the STRIP-MATRIX kernel.
//
// What the im2win layout gives a tensor core.  For one (image, channel) the im2win tensor is a row-major
// matrix with Fh columns: row c = m*W + k holds the Fh input values of input column k under output row m
// (Algorithm 1).  The window of output (m, n) is Fw CONSECUTIVE rows of that matrix, rows m*W + n*s + v,
// v = 0..Fw-1, and neighbouring windows overlap in Fw-s of them (Section III-A).  So the convolution is
// Fw matrix products, one per filter column v, whose A operands are the SAME matrix T read from row
// offsets that differ by v:
//     O[(m,n), j] = sum_v  sum_{r,u}  T[m*W + n*s + v][(r,u)] * Fv[j][(r,u)],   Fv[j][(r,u)] = F[j][r][u][v].
// T is laid out in shared memory so that a row offset is a plain address offset of the MMA's matrix
// descriptor (no swizzle, 16-byte chunks stored chunk-major: chunk kc of row p at kc*LBO + p*16), hence
// every element of the im2win tensor is moved ONCE -- global -> shared by TMA, shared -> T by a
// transposing copy -- and the Fw/s-fold window expansion happens inside the tensor core's operand fetch.
// (Stride s > 1: the columns are split into s classes k mod s, one T matrix per class; tap v reads class
// v mod s at row offset v / s.)
//
// GEMM view per work unit: M = 128*MH consecutive rows p = m*WP + q of one image (WP = ceil(W/s); the
// rows with q >= Wo are computed and dropped), N = a tile of up to 256 filters, K = (r,u) per tap.
// Roles (one persistent CTA per SM, units t, t+grid, ...):
//   warp 0       source producer: one 2-D TMA box (or one bulk copy per channel) per group of GR channels
//   warp 1       MMA issuer (one thread): tcgen05.mma kind::tf32 / kind::f16, A and B from shared memory,
//                fp32 accumulators in TMEM, one fixed summation order (results are reproducible bit for bit)
//   warp 2       filter producer: TMA boxes (64-byte swizzle) from the tap-major filter copy Fv that a small
//                kernel writes into the caller's scratch at the start of the call (fp32, or bf16 in BF16 mode)
//   warps 4-11   transposers: staged source -> T (fp32 as is for TF32, cvt.rn.bf16x2 for BF16)
//   warps 12-19  epilogue (four per 128-row half): tcgen05.ld -> coalesced NCHW stores
// The source is the fp32 im2win tensor, the bf16 im2win tensor, or (fused) the untransformed input, whose
// rows m*s+u supply the same values.  Every wait is bounded (status word + common teardown on expiry).
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <cstring>
#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "strip_common.cuh"

namespace im2win {
namespace {

using namespace stripc;

struct SParams {
  const void* src;
  float* out;
  int32_t* status;
  int32_t C, K, Ho, Wo, W, WP;
  int32_t RPI;        // T rows per image: Ho * WP
  int32_t TPI;        // tiles per image
  int32_t MH;         // 128-row halves per tile
  int32_t RT;         // T rows per class a tile uses: 128*MH + (Fw-1)/s
  int32_t RA;         // T rows per class allocated (RT rounded up to 8)
  int32_t NJ;         // RT * s: (row, class) pairs = source columns per tile
  int32_t NT, n_ntiles, Kp;
  int32_t NTB;        // filter rows one CTA holds per block: NT, or NT/2 when two CTAs share an MMA
  int32_t pair;       // two CTAs (a cluster) work as one: tcgen05.mma.cta_group::2, M = 256, each CTA its own rows and half the filter tile
  int32_t nhwc;       // output layout N x Ho x Wo x K
  int64_t tiles;      // row tiles: N * TPI
  int32_t G, GR, NSUB, NTS;  // channels per T stage / per source stage, source stages per T stage, T stages per unit
  int32_t CBN;        // channel blocks (of NCH channels) per source stage
  int32_t NBLK, BB, NBS;     // filter blocks (2 K steps) per (T stage, tap); blocks per filter stage; filter stages per (T stage, tap)
  int32_t SR, SB, ND;
  int32_t epi_split;  // the epilogue warps store columns [0, epi_split); with one accumulator buffer the (then idle)
                      // transposer warps store [epi_split, NT); epi_split == NT: no help
  int32_t CP;         // elements per channel row of a source stage
  int32_t box;        // source stages come as one 2-D TMA box
  int32_t pm;         // plane length modulo the elements of a 16-byte chunk (bulk copies: per-channel phase)
  int64_t plane;      // source elements per (image, channel)
  int64_t n_src;
  int64_t units;
  uint32_t idesc, tmem_cols;
  uint32_t raw_stage_bytes, t_stage_bytes, b_stage_bytes;
  uint32_t off_t, off_raw, off_bar, off_misc;
#ifdef IM2WIN_PROF
  long long* prof;
#endif
};

// Work of iteration `it` of this CTA: filter tile, image, first T row of the row tile, and whether its
// results are stored.  Single-CTA mode: units t = blockIdx.x + it*grid, the filter tile fastest.  Pair
// mode: the pair (cluster) takes two consecutive row tiles of one filter tile, one per CTA; where the
// number of row tiles is odd the last pair's second CTA repeats the last tile without storing.
struct Unit {
  int32_t nt, img, R0;
  bool store;
};
template <bool PAIR>
__device__ __forceinline__ bool unit_at(const SParams& P, int64_t it, uint32_t rank, Unit& u) {
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
// Source elements [e_lo, e_hi) of a channel plane that the tile starting at T row R0 needs.
template <int FH, int S, bool FUSED>
__device__ __forceinline__ void tile_range(const SParams& P, int32_t R0, int32_t& e_lo, int32_t& e_hi) {
  const int32_t r_last = min(R0 + P.RT, P.RPI) - 1;
  const int32_t m0 = R0 / P.WP, q0 = R0 - m0 * P.WP;
  const int32_t m1 = r_last / P.WP, q1 = r_last - m1 * P.WP;
  const int32_t k1 = min(q1 * S + S - 1, P.W - 1);
  if (FUSED) {
    e_lo = m0 * S * P.W + q0 * S;
    e_hi = (m1 * S + FH - 1) * P.W + k1 + 1;
  } else {
    e_lo = (m0 * P.W + q0 * S) * FH;
    e_hi = (m1 * P.W + k1 + 1) * FH;
  }
}

// The MMA-issuing warp's whole life (all lanes run it, so that the descriptor arithmetic and the waits are
// warp-uniform work; lane 0 issues).  A filter stage holds the NBLK blocks of one (T stage, tap),
// so there is one wait and one release per NBLK*2*MH MMAs.
template <int FW, int S, bool BF16, int MH, int NBLK, bool PAIR>
__device__ __forceinline__ void mma_role(const SParams& P, SBars* bars, SMisc* misc, uint32_t tmem_base, uint32_t t_sa,
                                         uint32_t b_sa) {
  Ring tr, br, dr;
  bool ok = true;
  SPROF_DECL
  const uint64_t ad0 = ptx::smem_desc_k_chunkmajor(t_sa, (uint32_t)(S * P.RA) * 16u);
  const uint64_t bd0 = ptx::smem_desc_k_sw64(b_sa);
  const uint32_t a_lo0 = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32);
  const uint32_t b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
  const uint32_t t16 = P.t_stage_bytes >> 4, b16 = P.b_stage_bytes >> 4;
  const uint32_t blk16 = (uint32_t)P.NTB * 4u;         // one filter block (NTB rows x 64 bytes) in 16-byte units
  const uint32_t kstep16 = 2u * (uint32_t)(S * P.RA);  // one MMA K step (two chunks) of T in 16-byte units
  const uint32_t RA = (uint32_t)P.RA, NT = (uint32_t)P.NT, idesc = P.idesc;
  const uint32_t t_full0 = ptx::smem_u32(&bars->t_full[0]), t_empty0 = ptx::smem_u32(&bars->t_empty[0]);
  const uint32_t b_full0 = ptx::smem_u32(&bars->b_full[0]), b_empty0 = ptx::smem_u32(&bars->b_empty[0]);
  const int32_t lane = (int32_t)(threadIdx.x & 31);
  const uint32_t elect = lane == 0 ? 1u : 0u;
  for (int64_t it = 0; ok; ++it, dr.advance(P.ND)) {
    Unit u;
    if (!unit_at<PAIR>(P, it, 0, u)) break;
    SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_empty[dr.idx]), dr.phase ^ 1u, DEV_TIMEOUT_ACC))
    if (!ok) break;
    ptx::tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(dr.idx * MH) * NT;
    uint32_t accum = 0;
    for (int32_t ts = 0; ts < P.NTS && ok; ++ts, tr.advance(2)) {
      SPROF_W(1, ok = wait_bar_warp(P, misc, t_full0 + (uint32_t)tr.idx * 8u, tr.phase, DEV_TIMEOUT_A_FULL, 20))
      if (!ok) break;
      const uint32_t a_stage = a_lo0 + (uint32_t)tr.idx * t16;
#pragma unroll
      for (int v = 0; v < FW; ++v) {
        SPROF_W(2, ok = wait_bar_warp(P, misc, b_full0 + (uint32_t)br.idx * 8u, br.phase, DEV_TIMEOUT_B_FULL, 20))
        if (!ok) break;
        ptx::tc_fence_after();
        uint32_t a_k = a_stage + (uint32_t)(v % S) * RA + (uint32_t)(v / S);
        uint32_t b_k = b_lo0 + (uint32_t)br.idx * b16;
#pragma unroll
        for (int blk = 0; blk < NBLK; ++blk) {
#pragma unroll
          for (int k2 = 0; k2 < 2; ++k2) {
            mma_ss_e<BF16, PAIR>(d_tmem, a_k, a_hi, b_k + (uint32_t)k2 * 2u, b_hi, idesc, accum, elect);
            if (MH == 2) mma_ss_e<BF16, PAIR>(d_tmem + NT, a_k + 128u, a_hi, b_k + (uint32_t)k2 * 2u, b_hi, idesc, accum, elect);
            accum = 1;
            a_k += kstep16;
          }
          b_k += blk16;
        }
        mma_commit_e<PAIR>(b_empty0 + (uint32_t)br.idx * 8u, elect);
        br.advance(P.SB);
      }
      if (!ok) break;
      mma_commit_e<PAIR>(t_empty0 + (uint32_t)tr.idx * 8u, elect);
    }
    if (!ok) break;
    mma_commit_e<PAIR>(ptx::smem_u32(&bars->acc_full[dr.idx]), elect);
  }
  SPROF_DUMP(1)
}

// SRCK: 0 = fp32 im2win tensor, 1 = untransformed input (fused), 2 = bf16 im2win tensor (BF16 mode).
template <int FH, int FW, int S, bool BF16, int SRCK, bool PAIR>
__global__ void __launch_bounds__(640, 1)
conv_tc_strip_kernel(const SParams P, const __grid_constant__ CUtensorMap fmap, const __grid_constant__ CUtensorMap xmap) {
  constexpr bool FUSED = SRCK == 1;
  constexpr bool SRC16 = SRCK == 2;
  static_assert(!SRC16 || BF16, "a 16-bit source feeds the BF16 mode");
  constexpr uint32_t ES = SRC16 ? 2u : 4u;       // bytes per source element
  constexpr int32_t EPC = SRC16 ? 8 : 4;          // source elements per 16-byte chunk
  constexpr int NCH = BF16 ? 8 : 4;               // channels per transposer task = T elements per 16-byte chunk
  constexpr int GDIV = FH % 4 == 0 ? 1 : (FH % 2 == 0 ? 2 : 4);
  constexpr int NBLK = GDIV * FH / 4;             // filter blocks (two K steps each) per (T stage, tap)

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* const smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  SBars* const bars = reinterpret_cast<SBars*>(smem + P.off_bar);
  SMisc* const misc = reinterpret_cast<SMisc*>(smem + P.off_misc);
  const uint32_t b_sa = ptx::smem_u32(smem), t_sa = b_sa + P.off_t, raw_sa = b_sa + P.off_raw;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int32_t n_epi_warps = 4 * P.MH;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;  // pair mode: 0 = the leader, whose thread issues the MMAs of both
  constexpr uint32_t kShare = PAIR ? 2u : 1u;            // CTAs that arrive on the leader's "full"-side barriers

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
      ptx::mbar_init(ptx::smem_u32(&bars->t_empty[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[i]), (uint32_t)n_epi_warps * kShare * (P.epi_split < P.NT ? 2u : 1u));
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

  if (warp == 0) {
    // ================================================================ SOURCE PRODUCER
    using SrcT = typename std::conditional<SRC16, uint16_t, float>::type;
    const SrcT* const xsrc = reinterpret_cast<const SrcT*>(P.src);
    Ring rr;
    int64_t count = 0;
    bool ok = true;
    SPROF_DECL
    for (int64_t it = 0; ok; ++it) {
      Unit u;
      if (!unit_at<PAIR>(P, it, rank, u)) break;
      int32_t e_lo, e_hi;
      tile_range<FH, S, FUSED>(P, u.R0, e_lo, e_hi);
      const int32_t len = e_hi - e_lo;
      const int32_t box_x = (e_lo & ~(EPC - 1)) / (EPC / 2);  // in 8-byte units
      const int32_t nstages = P.NTS * P.NSUB;
      for (int32_t sidx = 0; sidx < nstages && ok; ++sidx, ++count, rr.advance(P.SR)) {
        const int32_t ch0 = sidx * P.GR;
        const uint32_t full = ptx::smem_u32(&bars->raw_full[rr.idx]);
        SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->raw_empty[rr.idx]), rr.phase ^ 1u, DEV_TIMEOUT_RAW_EMPTY, 64))
        if (!ok) break;
        const uint32_t dst0 = raw_sa + (uint32_t)rr.idx * P.raw_stage_bytes;
        if (P.box) {
          if (lane == 0) {
            ptx::mbar_arrive_expect_tx(full, P.raw_stage_bytes);
            tma_load_2d(dst0, &xmap, box_x, u.img * P.C + ch0, full);
          }
        } else {
          const SrcT* src = nullptr;
          uint32_t dst = 0, bytes = 0;
          if (lane < P.GR) {
            const int64_t start = ((int64_t)u.img * P.C + ch0 + lane) * P.plane + e_lo;
            const int32_t skew = (int32_t)(start & (EPC - 1));
            const int64_t a0 = start - skew;
            int32_t nel = (skew + len + EPC - 1) & ~(EPC - 1);
            dst = dst0 + (uint32_t)(lane * P.CP) * ES;
            if (a0 + nel > P.n_src) {  // the last 16-byte chunk would pass the end of the tensor
              const int32_t nbulk = (int32_t)((P.n_src - a0) & ~(int64_t)(EPC - 1));
              SrcT* d = reinterpret_cast<SrcT*>(smem + P.off_raw + (size_t)rr.idx * P.raw_stage_bytes) + (size_t)lane * P.CP;
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
  } else if (warp == 1) {
    // ================================================================ MMA ISSUER
    // One thread.  Its instruction stream is what bounds narrow filter tiles, so the loop over one
    // T stage is fully unrolled for the compile-time (taps, filter blocks, halves) and steps the
    // descriptors by additions of registers computed once.
    if (rank == 0) {
      if (P.MH == 1) mma_role<FW, S, BF16, 1, NBLK, PAIR>(P, bars, misc, tmem_base, t_sa, b_sa);
      else mma_role<FW, S, BF16, 2, NBLK, PAIR>(P, bars, misc, tmem_base, t_sa, b_sa);
    }
    __syncwarp();
  } else if (warp == 2) {
    // ================================================================ FILTER PRODUCER
    if (lane == 0) {
      Ring br;
      int64_t count = 0;
      bool ok = true;
      SPROF_DECL
      const int32_t bke = BF16 ? 32 : 16;  // elements per 64-byte filter row
      // Pair mode: this CTA fetches its half of every block's rows, and the bytes of both CTAs are counted
      // on the leader's barrier: the leader announces both halves with its one arrival (its own copies go
      // through the ordinary local form), the other CTA only issues its copies.  (Its bytes may land
      // before the announcement: the phase cannot complete before the leader's arrival, and the other
      // CTA cannot run a phase ahead, because it needs the stage's release, which follows the phase.)
      asm volatile("griddepcontrol.wait;" ::: "memory");  // the filter copy is written by the kernel launched just before
      const bool remote = PAIR && rank != 0;
      const uint32_t b_full_lead0 = remote ? mapa(ptx::smem_u32(&bars->b_full[0]), 0) : ptx::smem_u32(&bars->b_full[0]);
      for (int64_t it = 0; ok; ++it) {
        Unit u;
        if (!unit_at<PAIR>(P, it, rank, u)) break;
        const int32_t row0 = u.nt * P.NT + (int32_t)rank * P.NTB;
        for (int32_t ts = 0; ts < P.NTS && ok; ++ts) {
          for (int32_t v = 0; v < FW && ok; ++v, ++count, br.advance(P.SB)) {
            SPROF_W(0, ok = wait_bar(P, misc, ptx::smem_u32(&bars->b_empty[br.idx]), br.phase ^ 1u, DEV_TIMEOUT_B_EMPTY))
            if (!ok) break;
            const uint32_t full = b_full_lead0 + (uint32_t)br.idx * 8u;
            if (!remote) ptx::mbar_arrive_expect_tx(full, P.b_stage_bytes * kShare);
            for (int32_t blk = 0; blk < P.BB; ++blk) {
              const uint32_t dst = b_sa + (uint32_t)br.idx * P.b_stage_bytes + (uint32_t)blk * (uint32_t)P.NTB * 64u;
              if (remote) tma_load_2d_pair(dst, &fmap, (ts * P.NBLK + blk) * bke, v * P.Kp + row0, full);
              else tma_load_2d(dst, &fmap, (ts * P.NBLK + blk) * bke, v * P.Kp + row0, full);
            }
          }
        }
      }
      SPROF_DUMP(7)
      // every copy issued must have landed before the CTA exits: the stage's release by the MMAs that
      // read it says so (in pair mode the bytes are counted on the leader's barrier, not here)
      for (int64_t c = count > P.SB ? count - P.SB : 0; c < count; ++c)
        wait_bar(P, misc, ptx::smem_u32(&bars->b_empty[c % P.SB]), (uint32_t)(c / P.SB) & 1u, DEV_TIMEOUT_DRAIN);
    }
    __syncwarp();
  } else if (warp >= kTWarp0 && warp < kTWarp0 + kTW) {
    // ================================================================ TRANSPOSERS: staged source -> T
    const int32_t tid = (warp - kTWarp0) * 32 + lane;
    const int32_t ntasks = P.NJ * P.CBN;
    const uint32_t lbo = (uint32_t)(S * P.RA) * 16u;
    const uint32_t ustride = (FUSED ? (uint32_t)P.W : 1u) * ES;
    Ring rr, tr;
    bool ok = true;
    SPROF_DECL
    uint32_t hphase = 0;  // (epilogue help) phase of the single accumulator buffer's "full" barrier
    const bool remote = PAIR && rank != 0;
    const uint32_t t_full_lead0 = remote ? mapa(ptx::smem_u32(&bars->t_full[0]), 0) : ptx::smem_u32(&bars->t_full[0]);
    for (int64_t it = 0; ok; ++it) {
      Unit u;
      if (!unit_at<PAIR>(P, it, rank, u)) break;
      int32_t e_lo, e_hi;
      tile_range<FH, S, FUSED>(P, u.R0, e_lo, e_hi);
      // this thread's tasks: (source column j = (T row, class), channel block cb of the stage)
      uint32_t soff[kTMax], doff[kTMax];
      int32_t tcb[kTMax];
      bool tv[kTMax];
#pragma unroll
      for (int z = 0; z < kTMax; ++z) {
        const int32_t task = tid + z * (kTW * 32);
        tv[z] = false; soff[z] = 0; doff[z] = 0; tcb[z] = 0;
        if (task < ntasks) {
          const int32_t cb = task / P.NJ, j = task - cb * P.NJ;
          const int32_t p = j / S, cl = j - p * S;      // T row within the tile, class
          const int32_t rho = u.R0 + p;
          const int32_t m = rho / P.WP, q = rho - m * P.WP;
          const int32_t k = q * S + cl;
          if (rho < P.RPI && k < P.W) {
            tv[z] = true;
            tcb[z] = cb;
            const int32_t e = FUSED ? (m * S * P.W + k) : (m * P.W + k) * FH;
            soff[z] = (uint32_t)(e - e_lo + cb * NCH * P.CP) * ES;
            doff[z] = (uint32_t)(cl * P.RA + p) * 16u + (uint32_t)(cb * FH) * lbo;
          }
        }
      }
      // 16-byte phase of the staged ranges: per tile, plus (bulk copies of planes that are not a whole
      // number of chunks) per channel
      const int32_t sk0 = (int32_t)(((int64_t)u.img * P.C * P.plane + e_lo) & (EPC - 1));
      for (int32_t ts = 0; ts < P.NTS && ok; ++ts, tr.advance(2)) {
        const uint32_t t_stage = t_sa + (uint32_t)tr.idx * P.t_stage_bytes;
        for (int32_t sub = 0; sub < P.NSUB && ok; ++sub, rr.advance(P.SR)) {
          SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->raw_full[rr.idx]), rr.phase, DEV_TIMEOUT_RAW_FULL))
          if (!ok) break;
          if (sub == 0) {
            SPROF_W(1, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->t_empty[tr.idx]), tr.phase ^ 1u, DEV_TIMEOUT_A_EMPTY))
            if (!ok) break;
          }
#ifdef IM2WIN_PROF
          const long long cw0 = clock64();
#endif
          const uint32_t rs = raw_sa + (uint32_t)rr.idx * P.raw_stage_bytes;
          const int32_t ch0 = (ts * P.NSUB + sub) * P.GR;
          const uint32_t t_sub = t_stage + (uint32_t)(sub * P.CBN * FH) * lbo;
#pragma unroll
          for (int z = 0; z < kTMax; ++z) {
            if (tv[z]) {
              uint32_t val[NCH * FH];
#pragma unroll
              for (int c = 0; c < NCH; ++c) {
                const int32_t sk = P.pm ? ((sk0 + (ch0 + tcb[z] * NCH + c) * P.pm) & (EPC - 1)) : sk0;
                const uint32_t a = rs + soff[z] + (uint32_t)(c * P.CP + sk) * ES;
#pragma unroll
                for (int f = 0; f < FH; ++f) val[c * FH + f] = SRC16 ? lds_u16(a + (uint32_t)f * ustride) : lds_u32(a + (uint32_t)f * ustride);
              }
              const uint32_t d = t_sub + doff[z];
#pragma unroll
              for (int f = 0; f < FH; ++f) {
                if constexpr (!BF16) {
                  sts_v4(d + (uint32_t)f * lbo, val[4 * f], val[4 * f + 1], val[4 * f + 2], val[4 * f + 3]);
                } else if constexpr (SRC16) {
                  sts_v4(d + (uint32_t)f * lbo, val[8 * f] | (val[8 * f + 1] << 16), val[8 * f + 2] | (val[8 * f + 3] << 16),
                         val[8 * f + 4] | (val[8 * f + 5] << 16), val[8 * f + 6] | (val[8 * f + 7] << 16));
                } else {
                  sts_v4(d + (uint32_t)f * lbo,
                         ptx::pack_bf16x2(__uint_as_float(val[8 * f]), __uint_as_float(val[8 * f + 1])),
                         ptx::pack_bf16x2(__uint_as_float(val[8 * f + 2]), __uint_as_float(val[8 * f + 3])),
                         ptx::pack_bf16x2(__uint_as_float(val[8 * f + 4]), __uint_as_float(val[8 * f + 5])),
                         ptx::pack_bf16x2(__uint_as_float(val[8 * f + 6]), __uint_as_float(val[8 * f + 7])));
                }
              }
            }
          }
          const bool last = sub == P.NSUB - 1;
          if (last) ptx::fence_proxy_async_smem();  // this thread's T writes -> visible to the tensor core
          __syncwarp();
#ifdef IM2WIN_PROF
          pw[2] += clock64() - cw0;
#endif
          if (lane == 0) {
            ptx::mbar_arrive(ptx::smem_u32(&bars->raw_empty[rr.idx]));
            if (last) {
              if (remote) arrive_cluster(t_full_lead0 + (uint32_t)tr.idx * 8u);
              else ptx::mbar_arrive(t_full_lead0 + (uint32_t)tr.idx * 8u);
            }
          }
        }
      }
      // One accumulator buffer: nothing can be transposed for the next unit before this unit's MMAs are
      // done, so this warp stores the upper columns of its TMEM lane quarter meanwhile.
      if (ok && P.epi_split < P.NT) {
        const int32_t hh = (warp - kTWarp0) >> 2, q4 = warp & 3;
        ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_full[0]), hphase, DEV_TIMEOUT_ACC, 128);
        if (!ok) break;
        hphase ^= 1u;
        ptx::tc_fence_after();
        if (hh < P.MH) {
          const int32_t rho = u.R0 + hh * 128 + q4 * 32 + lane;
          const int32_t m = rho / P.WP, q = rho - m * P.WP;
          const bool valid = u.store && rho < P.RPI && q < P.Wo;
          const int32_t n0 = u.nt * P.NT;
          const int64_t HoWo = (int64_t)P.Ho * P.Wo;
          float* const orow = P.nhwc ? P.out + ((int64_t)u.img * HoWo + (int64_t)m * P.Wo + q) * P.K + n0
                                     : P.out + ((int64_t)u.img * P.K + n0) * HoWo + (int64_t)m * P.Wo + q;
          store_columns(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(hh * P.NT), orow, P.nhwc ? 1 : HoWo, P.epi_split, P.NT,
                        P.K - n0, valid, false, P.nhwc && (P.K & 3) == 0);
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
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + n_epi_warps) {
    // ================================================================ EPILOGUE: TMEM -> NCHW
    const int32_t h = (warp - kEpiWarp0) >> 2, q4 = warp & 3;  // (kEpiWarp0 is a multiple of 4: warp & 3 = TMEM lane quarter)
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    Ring dr;
    bool ok = true;
    SPROF_DECL
    const int32_t eK = P.K;
    const int64_t eHoWo = (int64_t)P.Ho * P.Wo;
    const bool remote = PAIR && rank != 0;
    const uint32_t acc_empty_lead0 = remote ? mapa(ptx::smem_u32(&bars->acc_empty[0]), 0) : ptx::smem_u32(&bars->acc_empty[0]);
    for (int64_t it = 0; ok; ++it, dr.advance(P.ND)) {
      Unit u;
      if (!unit_at<PAIR>(P, it, rank, u)) break;
      const int32_t rho = u.R0 + h * 128 + q4 * 32 + lane;
      const int32_t m = rho / P.WP, q = rho - m * P.WP;
      const bool valid = u.store && rho < P.RPI && q < P.Wo;
      const int32_t n0 = u.nt * P.NT;
      float* const orow = P.nhwc ? P.out + ((int64_t)u.img * eHoWo + (int64_t)m * P.Wo + q) * eK + n0
                                 : P.out + ((int64_t)u.img * P.K + n0) * eHoWo + (int64_t)m * P.Wo + q;
      SPROF_W(0, ok = wait_bar_warp(P, misc, ptx::smem_u32(&bars->acc_full[dr.idx]), dr.phase, DEV_TIMEOUT_ACC, 128))
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t d_tmem = tmem_base + lane_base + (uint32_t)((dr.idx * P.MH + h) * P.NT);
      store_columns(d_tmem, orow, P.nhwc ? 1 : eHoWo, 0, P.epi_split, eK - n0, valid, false, P.nhwc && (eK & 3) == 0);
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
//   Fv[v][j][r*Fh + u] = F[j][r][u][v]   (j < K; rows K..Kp-1 are zero), fp32 or bf16 (nearest even).
// One CTA per (filter j, block of 128 channels): its 128*Fh*Fw values pass through shared memory, so that both
// the reads and the writes are contiguous and every CTA is one load - store round trip (the convolution
// kernel's first MMA waits for this copy: its latency counts).
constexpr int kPrepCh = 128, kPrepFF = 9;
template <bool BF16>
__global__ void __launch_bounds__(128) filter_tap_major_kernel(const float* __restrict__ f, void* __restrict__ o, int32_t K,
                                                               int32_t Kp, int32_t C, int32_t FH, int32_t FW) {
  // the convolution kernel that follows may start its prologue now (it waits for this grid's completion
  // before it reads the copy)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ float sm[kPrepCh * kPrepFF];
  const int32_t j = (int32_t)blockIdx.x, tid = (int32_t)threadIdx.x;
  const int32_t c0 = (int32_t)blockIdx.y * kPrepCh;
  const int32_t nc = min(kPrepCh, C - c0);
  const int32_t ff = FH * FW, n = nc * ff;
  const float* fj = f + ((int64_t)j * C + c0) * ff;
  if (j < K) {
    float x[kPrepFF];
#pragma unroll
    for (int q = 0; q < kPrepFF; ++q) {  // (all loads in flight before the first use)
      const int32_t i = tid + q * 128;
      x[q] = (q < ff && i < n) ? __ldg(fj + i) : 0.f;
    }
#pragma unroll
    for (int q = 0; q < kPrepFF; ++q) {
      const int32_t i = tid + q * 128;
      if (q < ff && i < n) sm[i] = x[q];
    }
  } else {
    for (int32_t i = tid; i < n; i += 128) sm[i] = 0.f;
  }
  __syncthreads();
  const int32_t row = C * FH, nku = nc * FH;
  for (int32_t v = 0; v < FW; ++v) {
    const int64_t obase = ((int64_t)v * Kp + j) * row + (int64_t)c0 * FH;
    for (int32_t ku = tid; ku < nku; ku += 128) {
      const float y = sm[ku * FW + v];  // (r*Fh + u)*Fw + v = ku*Fw + v
      if (BF16) static_cast<__nv_bfloat16*>(o)[obase + ku] = __float2bfloat16_rn(y);
      else static_cast<float*>(o)[obase + ku] = y;
    }
  }
}

// ---------------------------------------------------------------------------------------------- host side

struct Plan {
  SParams P;
  size_t smem_bytes, scratch_bytes;
  int threads;
};

// Fills the launch parameters for (FH, FW, S, BF16, SRCK); IM2WIN_EUNSUPPORTED where the kernel does not apply.
template <int FH, int FW, int S, bool BF16, int SRCK>
int make_plan(const Geometry& g, Plan* pl, int pair, int mh_fixed) {
  constexpr int NCH = BF16 ? 8 : 4;
  constexpr int64_t ES = SRCK == 2 ? 2 : 4;
  constexpr int64_t EPC = 16 / ES;
  constexpr int SH = (FW - 1) / S;
  constexpr int GDIV = FH % 4 == 0 ? 1 : (FH % 2 == 0 ? 2 : 4);  // channel blocks per T stage: (G/NCH)*FH chunks = whole filter blocks of 4
  SParams& P = pl->P;
  P = SParams{};
  P.G = NCH * GDIV;
  if (g.C % P.G != 0) return IM2WIN_EUNSUPPORTED;
  if (g.HoWo > (1 << 28) || (int64_t)g.H * g.W > (1 << 28)) return IM2WIN_EUNSUPPORTED;
  P.C = g.C; P.K = g.K; P.Ho = g.Ho; P.Wo = g.Wo; P.W = g.W;
  P.nhwc = g.out_nhwc;
  P.WP = (g.W + S - 1) / S;
  P.RPI = g.Ho * P.WP;
  P.n_ntiles = (g.K + 255) / 256;
  P.NT = ((g.K + P.n_ntiles - 1) / P.n_ntiles + 15) / 16 * 16;
  P.Kp = P.n_ntiles * P.NT;
  P.pair = pair;
  P.NTB = pair ? P.NT / 2 : P.NT;
  P.NTS = g.C / P.G;
  P.NBLK = GDIV * FH / 4;
  if (SRCK == 1) { P.plane = (int64_t)g.H * g.W; P.n_src = g.n_in; }
  else { P.plane = g.HoL; P.n_src = g.n_win; }
  P.pm = (int32_t)(P.plane % EPC);
  // dynamic shared memory for the three areas: the limit less the base alignment (1024), the round-ups
  // between the areas (1024 + 128 + 16), the barriers and the small state block
  const int64_t cap = 227 * 1024 - 1024 - (1024 + 128 + 16) - (int64_t)((sizeof(SBars) + 15) / 16 * 16) - 64;
  P.MH = mh_fixed;
  if (P.MH * P.NT > 512) return IM2WIN_EUNSUPPORTED;
  P.TPI = (P.RPI + 128 * P.MH - 1) / (128 * P.MH);
  P.tiles = (int64_t)g.N * P.TPI;
  P.units = pair ? ((P.tiles + 1) / 2) * P.n_ntiles : P.tiles * P.n_ntiles;
  if (P.tiles * P.n_ntiles >= (1ll << 31) - 65536) return IM2WIN_EUNSUPPORTED;  // (the kernel's unit arithmetic is 32-bit)
  P.RT = 128 * P.MH + SH;
  P.RA = (P.RT + 7) / 8 * 8;
  P.NJ = P.RT * S;
  if ((int64_t)S * P.RA > 16383) return IM2WIN_EUNSUPPORTED;
  // elements of one channel a tile needs at most, plus the 16-byte phase in front
  const int64_t len_max = SRCK == 1 ? ((int64_t)((P.RT - 1) / P.WP + 1) * S + FH) * g.W : (int64_t)FH * P.NJ;
  int64_t cp = len_max + 2 * EPC;
  const int64_t cp_align = 32 / ES;  // a row is a whole number of 32 bytes: a stage of >= 4 rows a whole number of 128
  cp = (cp + cp_align - 1) / cp_align * cp_align;
  if (cp * ES > 65536) return IM2WIN_EUNSUPPORTED;
  P.CP = (int32_t)cp;
  P.t_stage_bytes = (uint32_t)(GDIV * FH * S * P.RA * 16);
  const int64_t blk_bytes = (int64_t)P.NTB * 64;
  const int64_t fixed = 2 * (int64_t)P.t_stage_bytes;
  P.ND = 512 / (P.MH * P.NT) >= 2 ? 2 : 1;
  P.BB = P.NBLK;  // a filter stage = the blocks of one (T stage, tap): one wait and one release per NBLK*2*MH MMAs
  P.NBS = 1;
  P.b_stage_bytes = (uint32_t)(P.BB * blk_bytes);
  // Channel blocks per source stage: as many as keep a stage's (column, block) tasks within about two
  // rounds of the 256 transposer threads, fewer if the rings do not fit otherwise.  What is left beside
  // the two T stages goes to the two rings stage by stage, in proportion to what each needs in flight.
  int64_t sb = 0, sr = 0;
  const int64_t left = cap - fixed;
  for (int cbn = GDIV; cbn >= 1; cbn /= 2) {
    if (GDIV % cbn != 0 || (int64_t)P.NJ * cbn > 2 * kTW * 32 + 32) {
      if (cbn > 1) continue;
    }
    if ((int64_t)P.NJ * cbn > (int64_t)kTMax * kTW * 32) return IM2WIN_EUNSUPPORTED;
    const int64_t raw_bytes = (int64_t)cbn * NCH * cp * ES;
    if (cbn * NCH > 32 || raw_bytes % 128 != 0) continue;
    if (2 * (int64_t)P.b_stage_bytes + 2 * raw_bytes > left) continue;
    P.CBN = cbn;
    P.GR = cbn * NCH;
    P.raw_stage_bytes = (uint32_t)raw_bytes;
    // stages each ring wants: the bytes it must keep in flight to cover the memory latency (about 2500
    // cycles under load) at its consumption rate, plus the stage being consumed
    const double mma_cyc = P.NT / 2.0 > 50.0 ? P.NT / 2.0 : 50.0;
    const double b_stage_cyc = (double)P.NBLK * 2 * P.MH * mma_cyc;
    const double raw_stage_cyc = b_stage_cyc * FW * cbn / GDIV;
    const int64_t want_b = (int64_t)(2500.0 / b_stage_cyc + 0.999) + 1, want_r = (int64_t)(2500.0 / raw_stage_cyc + 0.999) + 1;
    sb = 2; sr = 2;
    while (true) {  // one more stage for the ring that is further below what it wants, while it fits
      const bool can_b = sb < kMaxB && (sb + 1) * P.b_stage_bytes + sr * raw_bytes <= left;
      const bool can_r = sr < kMaxRaw && sb * P.b_stage_bytes + (sr + 1) * raw_bytes <= left;
      if (!can_b && !can_r) break;
      const double fill_b = (double)sb / (double)want_b, fill_r = (double)sr / (double)want_r;
      if (can_b && (!can_r || fill_b <= fill_r)) ++sb;
      else ++sr;
    }
    break;
  }
  if (!sb) return IM2WIN_EUNSUPPORTED;
  P.NSUB = P.G / P.GR;
  P.box = (P.pm == 0 && cp * ES <= 2048 && P.GR >= 4 && encode_fn() != nullptr && (int64_t)g.N * g.C <= INT32_MAX &&
           !knobs().no_box) ? 1 : 0;
  P.SB = (int32_t)sb; P.SR = (int32_t)sr;
  uint32_t off = (uint32_t)(P.SB * P.b_stage_bytes);
  off = (off + 1023) / 1024 * 1024;
  P.off_t = off; off += 2 * P.t_stage_bytes;
  off = (off + 127) / 128 * 128;
  P.off_raw = off; off += (uint32_t)P.SR * P.raw_stage_bytes;
  off = (off + 15) / 16 * 16;
  P.off_bar = off; off += (uint32_t)((sizeof(SBars) + 15) / 16 * 16);
  P.off_misc = off; off += 64;
  pl->smem_bytes = off + 1024;
  if (pl->smem_bytes > 227 * 1024) return IM2WIN_EUNSUPPORTED;
  // one accumulator buffer: the transposer warps (two sets of four, one per half) store the upper half of
  // the columns; with one half per tile only the first set helps, so the epilogue warps keep all columns
  P.epi_split = (P.ND == 1 && P.MH == 2 && P.NT >= 64) ? (P.NT / 2 + 15) / 16 * 16 : P.NT;
  const int32_t cols = P.ND * P.MH * P.NT;
  P.tmem_cols = 32;
  while ((int32_t)P.tmem_cols < cols) P.tmem_cols *= 2;
  P.idesc = ptx::make_idesc(pair ? 256 : 128, P.NT, BF16 ? 1 : 2);
  pl->scratch_bytes = (size_t)FW * P.Kp * ((size_t)g.C * FH) * (BF16 ? 2 : 4);
  pl->threads = (kEpiWarp0 + 4 * P.MH) * 32;
  return IM2WIN_OK;
}

// Which variant of the kernel a problem gets (knobs override; rules from measurements on B200, batch 128):
//  * filter tiles of 192 columns or more run as CTA pairs (each CTA fetches half the filter rows: a single
//    CTA streaming a wide tile is bound by shared-memory bandwidth -- operand fetch of the MMAs plus the
//    TMA writes of the filter stages -- and by the filter stream's L2 rate); narrower tiles run on single
//    CTAs (a pair's MMAs cost the issuing thread about twice as long, which short MMAs cannot hide);
//  * two 128-row halves per tile (each filter stage feeds two MMAs, half the filter bytes per output) for
//    pairs when an image has more than 128 T rows, and for single CTAs whose units would otherwise be
//    short (few channels); one half otherwise: it keeps two accumulator buffers, so that the epilogue
//    overlaps the next unit.
template <int FH, int FW, int S, bool BF16, int SRCK>
int choose_plan(const Geometry& g, Plan* best) {
  const int nt = (((g.K + (g.K + 255) / 256 - 1) / ((g.K + 255) / 256)) + 15) / 16 * 16;
  const int wp = (g.W + S - 1) / S;
  int pair = nt >= 192 ? 1 : 0;
  int mh;
  if (pair) mh = ((int64_t)g.Ho * wp > 128) ? 2 : 1;
  else mh = ((int64_t)g.C * FH * FW / 8 < 100) ? 2 : 1;
  if (knobs().strip_pair == 1) pair = 1;
  if (knobs().strip_pair == 2) pair = 0;
  if (knobs().strip_mh) mh = knobs().strip_mh;
  // the preferred variant, then the others (a variant may not fit shared or tensor memory)
  const int order[4][2] = {{pair, mh}, {pair, 3 - mh}, {1 - pair, mh}, {1 - pair, 3 - mh}};
  for (const auto& o : order) {
    if (knobs().strip_pair == 1 && !o[0]) continue;
    if (knobs().strip_pair == 2 && o[0]) continue;
    if (knobs().strip_mh && knobs().strip_mh != o[1]) continue;
    if (make_plan<FH, FW, S, BF16, SRCK>(g, best, o[0], o[1]) == IM2WIN_OK) return IM2WIN_OK;
  }
  return IM2WIN_EUNSUPPORTED;
}

// Whether the strip-matrix kernel is expected to beat the persistent kernel (conv_tc_persistent.cu) on
// this problem.  Measured on B200 (batch 128, the 3x3 layers of the benchmark lists): per wave of
// 128-row passes it takes about 0.8 (TF32) / 0.75 (BF16) of the persistent kernel's time where the
// filter tile is 96 or wider (narrower MMAs are bound by its single issuing thread, where the persistent
// kernel's three win) and the stride is 1 (with two column classes its T stages leave the rings too
// little shared memory).  The persistent kernel's tiles may span images, this kernel's do not, so the
// comparison is between the two kernels' waves: small images whose tiles just fill one wave there stay
// there.  In BF16 mode a filter small enough to stay resident in the persistent kernel's shared memory
// also stays there.  Launches that fill less than half the SMs stay there too (reduction slices).
template <int FH, int FW, int S, bool BF16, int SRCK>
bool strip_preferred(const Geometry& g, const SParams& P) {
  if (S != 1 || P.NT < 96) return false;
  if (BF16 && (int64_t)g.K * g.Kg * 2 <= 160 * 1024) return false;
  const int nsm = sm_count();
  const int64_t slots = P.pair ? nsm / 2 : nsm;
  const double strip_passes = (double)((P.units + slots - 1) / slots) * P.MH;
  const int64_t tpi = (g.HoWo + 127) / 128;
  const bool pim = tpi * 128 * 100 <= g.HoWo * 107;
  const int64_t tiles = pim ? (int64_t)g.N * tpi : (g.Mtot + 127) / 128;
  // an under-filled launch: the persistent kernel cuts the reduction into slices there and wins
  // (measured at batch 1 and 32 on the deepest layers)
  if (tiles * P.n_ntiles * 2 <= nsm) return false;
  const double persistent_passes = (double)((tiles * P.n_ntiles + nsm - 1) / nsm);
  // (BF16: a tie goes to this kernel where the source is the input itself or the bf16 tensor, a third or half of the
  // fp32 tensor's staged bytes: sweep layer 7 fused 88 -> 77 us)
  if (BF16) return SRCK != 0 ? strip_passes * 0.75 <= persistent_passes : strip_passes * 0.75 < persistent_passes;
  return strip_passes * 0.8 <= persistent_passes;
}

template <int FH, int FW, int S, bool BF16, int SRCK, bool PAIR>
int launch_kernel(const SParams& P, const Plan& pl, const CUtensorMap& fmap, const CUtensorMap& xmap, cudaStream_t st) {
  auto kern = conv_tc_strip_kernel<FH, FW, S, BF16, SRCK, PAIR>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes) != cudaSuccess) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3((unsigned)pl.threads);
  cfg.dynamicSmemBytes = pl.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  // programmatic dependent launch: the prologue (barriers, TMEM, first source copies) overlaps the
  // filter-copy kernel launched just before; the filter producer waits for that kernel (griddepcontrol.wait)
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
  note_kernel(KERNEL_STRIP);
  return IM2WIN_OK;
}

template <int FH, int FW, int S, bool BF16, int SRCK>
int launch_strip(const void* src, const float* f, float* out, const Geometry& g, cudaStream_t st, Scratch scratch,
                 bool even_if_slower) {
  Plan pl;
  int rc = choose_plan<FH, FW, S, BF16, SRCK>(g, &pl);
  if (rc != IM2WIN_OK) return rc;
  SParams& P = pl.P;
  if (!even_if_slower && !knobs().force_strip && !strip_preferred<FH, FW, S, BF16, SRCK>(g, P)) return IM2WIN_EUNSUPPORTED;
  if (!scratch.ptr || scratch.bytes < pl.scratch_bytes || (reinterpret_cast<uintptr_t>(scratch.ptr) & 15u)) return IM2WIN_EUNSUPPORTED;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return IM2WIN_EUNSUPPORTED;
  P.src = src; P.out = out;
#ifdef IM2WIN_PROF
  P.prof = g_prof;
#endif
  P.status = device_status_word();
  if (!P.status) return IM2WIN_ECUDA;
  constexpr int64_t ES = SRCK == 2 ? 2 : 4;
  CUtensorMap fmap, xmap;
  memset(&fmap, 0, sizeof(fmap));
  memset(&xmap, 0, sizeof(xmap));
  {
    const int64_t row = (int64_t)g.C * FH;
    const cuuint64_t gdim[2] = {(cuuint64_t)row, (cuuint64_t)FW * P.Kp};
    const cuuint64_t gstr[1] = {(cuuint64_t)row * (BF16 ? 2 : 4)};
    const cuuint32_t box[2] = {BF16 ? 32u : 16u, (cuuint32_t)P.NTB};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&fmap, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, scratch.ptr, gdim, gstr, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return IM2WIN_EUNSUPPORTED;
  }
  if (P.box) {
    const cuuint64_t gdim[2] = {(cuuint64_t)(P.plane * ES / 8), (cuuint64_t)g.N * g.C};
    const cuuint64_t gstr[1] = {(cuuint64_t)P.plane * ES};
    const cuuint32_t box[2] = {(cuuint32_t)(P.CP * ES / 8), (cuuint32_t)P.GR};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(src), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      P.box = 0;  // bulk copies then
  }
  {
    static_assert(FH * FW <= kPrepFF, "filter-copy kernel's shared buffer");
    const dim3 pg((unsigned)P.Kp, (unsigned)((g.C + kPrepCh - 1) / kPrepCh));
    filter_tap_major_kernel<BF16><<<pg, 128, 0, st>>>(f, scratch.ptr, g.K, P.Kp, g.C, FH, FW);
  }
  return P.pair ? launch_kernel<FH, FW, S, BF16, SRCK, true>(P, pl, fmap, xmap, st)
                : launch_kernel<FH, FW, S, BF16, SRCK, false>(P, pl, fmap, xmap, st);
}

template <int FH, int FW, int S>
int launch_strip_fs(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                    Scratch scratch, int src_kind, bool slow_ok) {
  const bool bf16 = mode == IM2WIN_MODE_BF16;
  if (src_kind == 2) return bf16 ? launch_strip<FH, FW, S, true, 2>(src, f, out, g, st, scratch, slow_ok) : IM2WIN_EUNSUPPORTED;
  if (src_kind == 1) return bf16 ? launch_strip<FH, FW, S, true, 1>(src, f, out, g, st, scratch, slow_ok)
                                 : launch_strip<FH, FW, S, false, 1>(src, f, out, g, st, scratch, slow_ok);
  return bf16 ? launch_strip<FH, FW, S, true, 0>(src, f, out, g, st, scratch, slow_ok)
              : launch_strip<FH, FW, S, false, 0>(src, f, out, g, st, scratch, slow_ok);
}

template <int FH, int FW, int S>
size_t scratch_fs(const Geometry& g, int mode, int src_kind) {
  Plan pl;
  const bool bf16 = mode == IM2WIN_MODE_BF16;
  int rc;
  if (src_kind == 2) rc = bf16 ? choose_plan<FH, FW, S, true, 2>(g, &pl) : IM2WIN_EUNSUPPORTED;
  else if (src_kind == 1) rc = bf16 ? choose_plan<FH, FW, S, true, 1>(g, &pl) : choose_plan<FH, FW, S, false, 1>(g, &pl);
  else rc = bf16 ? choose_plan<FH, FW, S, true, 0>(g, &pl) : choose_plan<FH, FW, S, false, 0>(g, &pl);
  return rc == IM2WIN_OK ? (pl.scratch_bytes + 255) / 256 * 256 : 0;
}

}  // namespace

int launch_conv_tc_strip(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                         Scratch scratch, int src_kind, bool out_bf16, bool even_if_slower) {
  if (out_bf16) return IM2WIN_EUNSUPPORTED;  // fp32 epilogue only
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16) return IM2WIN_EUNSUPPORTED;
  if (g.Fh == 3 && g.Fw == 3 && g.s == 1) return launch_strip_fs<3, 3, 1>(src, f, out, g, mode, st, scratch, src_kind, even_if_slower);
  if (g.Fh == 3 && g.Fw == 3 && g.s == 2) return launch_strip_fs<3, 3, 2>(src, f, out, g, mode, st, scratch, src_kind, even_if_slower);
  return IM2WIN_EUNSUPPORTED;
}

size_t strip_scratch_bytes(const Geometry& g, int mode, int src_kind) {
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16) return 0;
  if (g.Fh == 3 && g.Fw == 3 && g.s == 1) return scratch_fs<3, 3, 1>(g, mode, src_kind);
  if (g.Fh == 3 && g.Fw == 3 && g.s == 2) return scratch_fs<3, 3, 2>(g, mode, src_kind);
  return 0;
}

}  // namespace im2win
