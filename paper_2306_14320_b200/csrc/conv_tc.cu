// im2win-based convolution (Algorithm 2) on the sm_100a tensor cores: generic kernel (any Fh, Fw, C, K).
// The persistent kernel specialised on the filter size is preferred when one applies; this one takes
// every other shape.
//
// The contraction  O[i][j][m][n] = sum_{r,u,v} Ihat[i][r][m][(n*s+v)*Fh+u] * F[j][r][u][v]  is run as a
// GEMM with M = output positions (i,m,n flattened), N = filters j, K = (r,u,v):
//
//   * One CTA owns a tile of up to 128 consecutive output positions and up to 256 filters.
//   * PRODUCER warp: for each group of CB channels it bulk-copies (TMA, cp.async.bulk) the part of
//     the im2win strips the tile's windows touch -- one contiguous range per (image, channel),
//     because consecutive strips of a plane are adjacent in memory -- into a shared-memory ring.
//   * REPACK warps (thread = output position = TMEM lane): the Fh*Fw floats of a window are
//     contiguous in its strip; each thread reads its own window from the staged range and writes
//     it to TENSOR MEMORY with tcgen05.st as row p of the A operand (converted to BF16 pairs in
//     BF16 mode).  Windows of neighbouring positions overlap in the strip, so the staged bytes
//     are about s/Fw of the operand bytes; the expansion never touches shared or global memory.
//   * FILTER warps build the B operand tiles (K-major, 128-byte swizzle) in shared memory straight
//     from the filter's native K,C,Fh,Fw order (no repacked copy of the filter exists).
//   * MMA thread: tcgen05.mma (A from TMEM, B from shared memory, fp32 accumulator in TMEM),
//     kind::tf32 or kind::f16(BF16); tcgen05.commit releases stages through mbarriers.
//   * EPILOGUE (the repack warps again): tcgen05.ld the accumulator, lane = position, and store
//     NCHW: for a fixed filter the 32 lanes of a warp write 32 consecutive floats.
//
// Every wait is bounded; on expiry the kernel records a code in the status word, unwinds through
// the common teardown (copies drained, TMEM freed) and returns.
#include "common.cuh"
#include "ptx_sm100.cuh"

namespace im2win {

namespace {

constexpr int kThreads = 384;       // 12 warps: 0 producer, 1 MMA, 4-7 repack/epilogue, 2,3,8-11 filter
constexpr int kFilterThreads = 192;
constexpr int kSegMax = 8;          // images a tile may span
constexpr int kMaxStages = 8;
constexpr uint32_t kSpinLimit = 1u << 22;

struct Seg {
  int64_t start0;  // element index in Ihat of the first needed float, channel 0
  int64_t virt_a;  // m_a*L + n_a*sFh of the segment's first position
  int32_t len;     // floats needed from start0 on
  int32_t dst_off; // float offset of this segment inside a channel slot
};

struct ConvParams {
  const float* xhat;
  const float* f;
  float* out;
  int32_t* status;
  int32_t C, K, Ho, Wo, L, FF, Fh, Fw, sFh;
  int64_t HoL, HoWo, Kg, Mtot, n_win;
  int32_t nhwc;        // output layout N x Ho x Wo x K
  int32_t TP;          // positions per tile (128 unless images are tiny)
  int32_t NT;          // filters per tile (multiple of 16, <= 256)
  int32_t n_ntiles;
  int32_t CB;          // channels per group
  int32_t KCG;         // CB*FF real reduction elements per group
  int32_t KCGP;        // padded to the MMA K step
  int32_t NG;          // groups = ceil(C / CB)
  int32_t a_cols;      // TMEM columns per A slot
  int32_t SA, SB, SR;  // ring depths: A slots (TMEM), B stages (smem), raw strip stages (smem)
  int32_t chan_pitch;  // floats per channel slot in a raw stage
  int32_t kstep;       // reduction elements per MMA: 8 (TF32) or 16 (BF16)
  int32_t kchunk;      // reduction elements per B stage: 32 or 64 (one 128-byte swizzle row)
  int32_t nsteps;      // NG*KCGP/kstep
  int32_t nchunks;     // ceil(nsteps/4)
  int32_t tmem_cols;
  int32_t bf16;
  uint32_t idesc;
  uint32_t off_raw, off_tab, off_seg, off_bar, off_misc;  // shared-memory offsets in bytes
};

struct Bars {
  uint64_t raw_full[kMaxStages], raw_empty[kMaxStages];
  uint64_t a_full[kMaxStages], a_empty[kMaxStages];
  uint64_t b_full[kMaxStages], b_empty[kMaxStages];
  uint64_t acc_full;
};

struct Misc {
  uint32_t tmem_base;
  int32_t abort;
  int32_t nseg;
  int32_t pad;
  int64_t i_first;
};

__device__ __forceinline__ void record(const ConvParams& P, Misc* misc, int32_t code) {
  atomicCAS(P.status, 0, code);
  atomicExch(&misc->abort, 1);
}

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait (about a second, or kSpinLimit polls); false = gave up (status recorded) or another
// role already aborted.
__device__ __forceinline__ bool wait_bar(const ConvParams& P, Misc* misc, uint64_t* bar, uint32_t parity,
                                         int32_t code) {
  const uint32_t b = ptx::smem_u32(bar);
  uint64_t t0 = 0;
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (ptx::mbar_try_wait(b, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*reinterpret_cast<volatile int32_t*>(&misc->abort)) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 1000000000ull) break;
    }
  }
  record(P, misc, code);
  return false;
}

// The same for a whole warp: every lane polls, the outcome is made uniform so that the
// warp-collective tcgen05 instructions that follow run converged.
__device__ __forceinline__ bool wait_bar_warp(const ConvParams& P, Misc* misc, uint64_t* bar, uint32_t parity,
                                              int32_t code) {
  return __all_sync(0xffffffffu, wait_bar(P, misc, bar, parity, code));
}

__global__ void __launch_bounds__(kThreads, 1) conv_tc_kernel(const __grid_constant__ ConvParams P) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // the swizzled operand tiles need a 1024-byte aligned base; the launch reserves the slack
  uint8_t* const smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* const b_stages = smem;  // SB stages of NT*128 bytes, each 1024-byte aligned
  float* const raw = reinterpret_cast<float*>(smem + P.off_raw);
  int32_t* const tab = reinterpret_cast<int32_t*>(smem + P.off_tab);
  Seg* const segs = reinterpret_cast<Seg*>(smem + P.off_seg);
  Bars* const bars = reinterpret_cast<Bars*>(smem + P.off_bar);
  Misc* const misc = reinterpret_cast<Misc*>(smem + P.off_misc);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t tile_m = blockIdx.x / P.n_ntiles;
  const int32_t ntile = (int32_t)(blockIdx.x - tile_m * P.n_ntiles);
  const int32_t n0 = ntile * P.NT;
  const int64_t P0 = tile_m * P.TP;
  const int64_t Pend = min(P0 + P.TP, P.Mtot) - 1;  // last valid position of the tile
  const int32_t raw_stage_floats = P.CB * P.chan_pitch;

  // ------------------------------------------------------------------ prologue
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&bars->raw_full[i]), 32);
      ptx::mbar_init(ptx::smem_u32(&bars->raw_empty[i]), 128);
      ptx::mbar_init(ptx::smem_u32(&bars->a_full[i]), 128);
      ptx::mbar_init(ptx::smem_u32(&bars->a_empty[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->b_full[i]), kFilterThreads);
      ptx::mbar_init(ptx::smem_u32(&bars->b_empty[i]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&bars->acc_full), 1);
    ptx::fence_mbar_init();
    misc->abort = 0;
    // segments: one per image the tile touches
    const int64_t i_first = P0 / P.HoWo, i_last = Pend / P.HoWo;
    misc->i_first = i_first;
    const int32_t nseg = (int32_t)(i_last - i_first + 1);
    misc->nseg = nseg;
    int32_t off = 0;
    for (int32_t g = 0; g < nseg && g < kSegMax; ++g) {
      const int64_t i = i_first + g;
      const int64_t qa = max(P0 - i * P.HoWo, (int64_t)0);
      const int64_t qb = min(Pend - i * P.HoWo, P.HoWo - 1);
      const int64_t m_a = qa / P.Wo, n_a = qa - m_a * P.Wo;
      const int64_t m_b = qb / P.Wo, n_b = qb - m_b * P.Wo;
      Seg s;
      s.virt_a = m_a * P.L + n_a * P.sFh;
      s.start0 = (i * P.C * P.Ho) * (int64_t)P.L + s.virt_a;
      s.len = (int32_t)((m_b * P.L + n_b * P.sFh) - s.virt_a) + P.FF;
      s.dst_off = off;
      off += (s.len + 3 + 3) & ~3;
      segs[g] = s;
    }
    if (nseg > kSegMax || off > P.chan_pitch) record(P, misc, DEV_RANGE);
  }
  // offset table: local reduction index -> (channel within group) << 20 | offset inside the window
  for (int32_t kl = threadIdx.x; kl < P.KCGP; kl += kThreads) {
    int32_t e = -1;
    if (kl < P.KCG) {
      const int32_t rl = kl / P.FF, w = kl - rl * P.FF;
      const int32_t u = w / P.Fw, v = w - u * P.Fw;
      e = (rl << 20) | (v * P.Fh + u);
    }
    tab[kl] = e;
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), (uint32_t)P.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  const uint32_t tmem_a0 = tmem_base + (uint32_t)P.NT;  // A slots follow the accumulator columns
  const int32_t nseg = misc->nseg;
  const bool bad = *reinterpret_cast<volatile int32_t*>(&misc->abort) != 0;

  if (!bad) {
    if (warp == 0) {
      // ================================================================ PRODUCER: strips -> smem
      const int32_t npairs = P.CB * nseg;
      int32_t issued = 0;
      for (int32_t g = 0; g < P.NG; ++g, ++issued) {
        const int32_t sr = g % P.SR;
        const uint32_t ph = (uint32_t)(g / P.SR) & 1u;
        if (!wait_bar(P, misc, &bars->raw_empty[sr], ph ^ 1u, DEV_TIMEOUT_RAW_EMPTY)) break;
        const uint32_t full = ptx::smem_u32(&bars->raw_full[sr]);
        float* stage = raw + (size_t)sr * raw_stage_floats;
        for (int32_t idx = lane; idx < npairs; idx += 32) {
          const int32_t rl = idx / nseg, sg = idx - rl * nseg;
          const int32_t r = g * P.CB + rl;
          if (r >= P.C) continue;
          const Seg s = segs[sg];
          const int64_t start = s.start0 + (int64_t)r * P.HoL;
          const int32_t skew = (int32_t)(start & 3);
          const int64_t a0 = start - skew;
          int32_t nfl = (skew + s.len + 3) & ~3;
          float* dst = stage + rl * P.chan_pitch + s.dst_off;
          if (a0 + nfl > P.n_win) {  // last chunk would run past the tensor: finish with plain loads
            const int32_t nbulk = (int32_t)((P.n_win - a0) & ~(int64_t)3);
            for (int64_t t = a0 + nbulk; t < P.n_win; ++t) dst[t - a0] = __ldg(P.xhat + t);
            nfl = nbulk;
          }
          if (nfl > 0) {
            ptx::mbar_expect_tx(full, (uint32_t)nfl * 4u);
            ptx::bulk_g2s(ptx::smem_u32(dst), P.xhat + a0, (uint32_t)nfl * 4u, full);
          }
        }
        ptx::mbar_arrive(full);
      }
      // teardown duty: every copy this warp issued must have landed before the CTA may exit
      for (int32_t g = max(issued - P.SR, 0); g < issued; ++g)
        wait_bar(P, misc, &bars->raw_full[g % P.SR], (uint32_t)(g / P.SR) & 1u, DEV_TIMEOUT_DRAIN);
    } else if (warp == 1) {
      // ================================================================ MMA ISSUER
      if (lane == 0) {
        const int32_t spg = P.KCGP / P.kstep;  // steps per group
        bool ok = true;
        for (int32_t ks = 0; ks < P.nsteps && ok; ++ks) {
          const int32_t g = ks / spg, kin = ks - g * spg;
          const int32_t c = ks >> 2, cin = ks & 3;
          const int32_t sa = g % P.SA, sb = c % P.SB;
          if (kin == 0) {
            ok = wait_bar(P, misc, &bars->a_full[sa], (uint32_t)(g / P.SA) & 1u, DEV_TIMEOUT_A_FULL);
            if (!ok) break;
            ptx::tc_fence_after();
          }
          if (cin == 0) {
            ok = wait_bar(P, misc, &bars->b_full[sb], (uint32_t)(c / P.SB) & 1u, DEV_TIMEOUT_B_FULL);
            if (!ok) break;
            ptx::tc_fence_after();
          }
          const uint32_t a_addr = tmem_a0 + (uint32_t)(sa * P.a_cols + kin * 8);
          const uint64_t b_desc =
              ptx::smem_desc_k_sw128(ptx::smem_u32(b_stages + (size_t)sb * P.NT * 128)) + (uint64_t)(cin * 2);
          if (P.bf16) ptx::mma_ts_f16(tmem_base, a_addr, b_desc, P.idesc, ks > 0);
          else        ptx::mma_ts_tf32(tmem_base, a_addr, b_desc, P.idesc, ks > 0);
          if (cin == 3 || ks == P.nsteps - 1) ptx::mma_commit(ptx::smem_u32(&bars->b_empty[sb]));
          if (kin == spg - 1) ptx::mma_commit(ptx::smem_u32(&bars->a_empty[sa]));
        }
        ptx::mma_commit(ptx::smem_u32(&bars->acc_full));
      }
      __syncwarp();
    } else if (warp >= 4 && warp < 8) {
      // ================================================================ REPACK + EPILOGUE
      const int32_t q4 = warp - 4;                       // TMEM lane quarter of this warp
      const int32_t p = q4 * 32 + lane;                  // row of the tile = TMEM lane
      const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
      const int64_t pos = P0 + p;
      const bool valid = p < P.TP && pos <= Pend;
      int32_t base_off = 0, skew0 = 0;
      int64_t out_off = 0;
      if (valid) {
        const int64_t i = pos / P.HoWo, q = pos - i * P.HoWo;
        const int64_t m = q / P.Wo, n = q - m * P.Wo;
        const Seg s = segs[(int32_t)(i - misc->i_first)];
        base_off = s.dst_off + (int32_t)((m * P.L + n * P.sFh) - s.virt_a);
        skew0 = (int32_t)(s.start0 & 3);
        out_off = P.nhwc ? (i * P.HoWo + q) * P.K + n0 : (i * P.K + n0) * P.HoWo + q;
      }
      const int32_t skew_step = (int32_t)(P.HoL & 3);
      bool ok = true;
      for (int32_t g = 0; g < P.NG && ok; ++g) {
        const int32_t sa = g % P.SA, sr = g % P.SR;
        ok = wait_bar_warp(P, misc, &bars->a_empty[sa], ((uint32_t)(g / P.SA) & 1u) ^ 1u, DEV_TIMEOUT_A_EMPTY);
        if (!ok) break;
        ptx::tc_fence_after();
        ok = wait_bar_warp(P, misc, &bars->raw_full[sr], (uint32_t)(g / P.SR) & 1u, DEV_TIMEOUT_RAW_FULL);
        if (!ok) break;
        const float* stage = raw + (size_t)sr * raw_stage_floats + base_off;
        const int32_t r0 = g * P.CB;
        auto fetch = [&](int32_t kl) -> float {
          const int32_t e = tab[kl];
          if (e < 0 || !valid) return 0.f;
          const int32_t rl = e >> 20, r = r0 + rl;
          if (r >= P.C) return 0.f;
          const int32_t skew = (skew0 + r * skew_step) & 3;
          return stage[rl * P.chan_pitch + skew + (e & 0xFFFFF)];
        };
        const uint32_t a_slot = tmem_a0 + lane_base + (uint32_t)(sa * P.a_cols);
        for (int32_t c8 = 0; c8 < P.a_cols; c8 += 8) {
          uint32_t v[8];
          if (P.bf16) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              v[e] = ptx::pack_bf16x2(fetch(2 * (c8 + e)), fetch(2 * (c8 + e) + 1));
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = __float_as_uint(fetch(c8 + e));
          }
          ptx::tmem_st_x8(a_slot + (uint32_t)c8, v);
        }
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        ptx::mbar_arrive(ptx::smem_u32(&bars->a_full[sa]));
        ptx::mbar_arrive(ptx::smem_u32(&bars->raw_empty[sr]));
      }
      // ---- epilogue: accumulator (lane = position, column = filter) -> NCHW
      if (ok) ok = wait_bar_warp(P, misc, &bars->acc_full, 0u, DEV_TIMEOUT_ACC);
      if (ok) {
        ptx::tc_fence_after();
        float* orow = P.out + out_off;
        for (int32_t c0 = 0; c0 < P.NT; c0 += 16) {
          uint32_t v[16];
          ptx::tmem_ld_x16(tmem_base + lane_base + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (n0 + c0 + e < P.K) orow[P.nhwc ? (int64_t)(c0 + e) : (int64_t)(c0 + e) * P.HoWo] = __uint_as_float(v[e]);
          }
        }
      }
    } else {
      // ================================================================ FILTER tiles -> smem (B operand)
      const int32_t bl = (warp < 4 ? warp - 2 : warp - 6) * 32 + lane;  // 0..191
      const int32_t epp = P.bf16 ? 8 : 4;                               // elements per 16-byte piece
      const bool dense = (P.KCG == P.KCGP);                             // padded index == real index
      const bool vec_ok = dense && (P.Kg & 3) == 0;
      bool ok = true;
      for (int32_t c = 0; c < P.nchunks && ok; ++c) {
        const int32_t sb = c % P.SB;
        ok = wait_bar(P, misc, &bars->b_empty[sb], ((uint32_t)(c / P.SB) & 1u) ^ 1u, DEV_TIMEOUT_B_EMPTY);
        if (!ok) break;
        uint8_t* stage = b_stages + (size_t)sb * P.NT * 128;
        for (int32_t idx = bl; idx < P.NT * 8; idx += kFilterThreads) {
          const int32_t j = idx >> 3, q = idx & 7;
          const int64_t kp0 = (int64_t)c * P.kchunk + (int64_t)q * epp;  // padded reduction index
          const bool row_ok = n0 + j < P.K;
          const float* frow = P.f + (int64_t)(n0 + j) * P.Kg;
          float x[8];
          if (row_ok && vec_ok && kp0 + epp <= P.Kg) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(frow + kp0));
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
            if (epp == 8) {
              const float4 b = __ldg(reinterpret_cast<const float4*>(frow + kp0 + 4));
              x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              x[e] = 0.f;
              if (e < epp && row_ok) {
                const int64_t kp = kp0 + e;
                const int64_t g = kp / P.KCGP;
                const int32_t kl = (int32_t)(kp - g * P.KCGP);
                const int64_t k = g * P.KCG + kl;
                if (kl < P.KCG && k < P.Kg) x[e] = __ldg(frow + k);
              }
            }
          }
          uint4 piece;
          if (P.bf16) {
            piece.x = ptx::pack_bf16x2(x[0], x[1]); piece.y = ptx::pack_bf16x2(x[2], x[3]);
            piece.z = ptx::pack_bf16x2(x[4], x[5]); piece.w = ptx::pack_bf16x2(x[6], x[7]);
          } else {
            piece.x = __float_as_uint(x[0]); piece.y = __float_as_uint(x[1]);
            piece.z = __float_as_uint(x[2]); piece.w = __float_as_uint(x[3]);
          }
          *reinterpret_cast<uint4*>(stage + (j >> 3) * 1024 + (j & 7) * 128 + ((q ^ (j & 7)) << 4)) = piece;
        }
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(ptx::smem_u32(&bars->b_full[sb]));
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    // on the abort path MMAs may still be in flight: give them a bounded chance to finish
    if (*reinterpret_cast<volatile int32_t*>(&misc->abort) && lane == 0 && !bad) {
      const uint32_t b = ptx::smem_u32(&bars->acc_full);
      for (uint32_t it = 0; it < kSpinLimit && !ptx::mbar_try_wait(b, 0u); ++it) {}
    }
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
  }
}

int32_t round_up(int32_t x, int32_t m) { return (x + m - 1) / m * m; }

}  // namespace

int launch_conv_tc_generic(const float* xhat, const float* f, float* out, const Geometry& g, int mode,
                   cudaStream_t st) {
  ConvParams P{};
  P.xhat = xhat; P.f = f; P.out = out;
  P.status = device_status_word();
  if (!P.status) return IM2WIN_ECUDA;
  P.C = g.C; P.K = g.K; P.Ho = g.Ho; P.Wo = g.Wo; P.L = g.L; P.FF = g.FF; P.Fh = g.Fh; P.Fw = g.Fw;
  P.sFh = g.sFh; P.HoL = g.HoL; P.HoWo = g.HoWo; P.Kg = g.Kg; P.Mtot = g.Mtot; P.n_win = g.n_win;
  P.nhwc = g.out_nhwc;
  P.bf16 = (mode == IM2WIN_MODE_BF16);
  P.kstep = P.bf16 ? 16 : 8;
  P.kchunk = P.bf16 ? 64 : 32;

  // positions per tile: at most kSegMax images may be touched
  int64_t tp = 128;
  if ((kSegMax - 1) * g.HoWo + 1 < tp) tp = (kSegMax - 1) * g.HoWo + 1;
  P.TP = (int32_t)tp;
  // filters per tile
  P.n_ntiles = (g.K + 255) / 256;
  P.NT = round_up((g.K + P.n_ntiles - 1) / P.n_ntiles, 16);

  // worst-case floats one channel contributes to a tile (see the segment construction in the kernel)
  const int64_t rowwrap = (int64_t)g.L - (int64_t)(g.Wo - 1) * g.sFh;
  const int64_t wraps = (tp + g.Wo - 2) / g.Wo;
  int64_t nseg_max = (tp - 1) / g.HoWo + 2;
  if (nseg_max > kSegMax) nseg_max = kSegMax;
  int64_t pitch = (tp - 1) * g.sFh + wraps * (rowwrap > g.sFh ? rowwrap - g.sFh : 0) + nseg_max * (g.FF + 6) + 4;
  pitch = (pitch + 3) & ~(int64_t)3;

  // channel group / ring depths: search the largest CB (<= 8) whose columns and bytes fit
  const int64_t smem_cap = 227 * 1024 - 2048;
  bool found = false;
  for (int sa = 2; sa >= 1 && !found; --sa) {
    double best_eff = -1.0;
    for (int cb = (g.C < 8 ? g.C : 8); cb >= 1; --cb) {
      const int64_t kcg = (int64_t)cb * g.FF;
      const int64_t kcgp = (kcg + P.kstep - 1) / P.kstep * P.kstep;
      const int64_t a_cols = P.bf16 ? kcgp / 2 : kcgp;
      if (a_cols * sa + P.NT > 512) continue;
      if (a_cols > 160 && cb > 1) continue;  // keep groups short so the rings turn over
      const int64_t raw_bytes = (int64_t)cb * pitch * 4;
      int sr = 3, sb = 4;
      auto total = [&](int sr_, int sb_) {
        return (int64_t)sb_ * P.NT * 128 + (int64_t)sr_ * raw_bytes + kcgp * 4 + 4096;
      };
      while (total(sr, sb) > smem_cap && sb > 2) --sb;
      while (total(sr, sb) > smem_cap && sr > 1) --sr;
      if (total(sr, sb) > smem_cap) continue;
      const double eff = (double)kcg / (double)kcgp;
      if (eff > best_eff + 1e-9) {
        best_eff = eff;
        P.CB = cb; P.KCG = (int32_t)kcg; P.KCGP = (int32_t)kcgp; P.a_cols = (int32_t)a_cols;
        P.SA = sa; P.SR = sr; P.SB = sb;
        found = true;
      }
    }
  }
  if (!found || pitch > INT32_MAX / 64) return IM2WIN_EUNSUPPORTED;
  P.chan_pitch = (int32_t)pitch;
  P.NG = (g.C + P.CB - 1) / P.CB;
  P.nsteps = P.NG * (P.KCGP / P.kstep);
  P.nchunks = (P.nsteps + 3) / 4;
  int32_t cols = P.NT + P.SA * P.a_cols;
  P.tmem_cols = 32;
  while (P.tmem_cols < cols) P.tmem_cols *= 2;
  P.idesc = ptx::make_idesc(128, P.NT, P.bf16 ? 1 : 2);

  uint32_t off = (uint32_t)P.SB * P.NT * 128;
  P.off_raw = off;  off += (uint32_t)P.SR * P.CB * P.chan_pitch * 4;
  P.off_tab = off;  off += (uint32_t)round_up(P.KCGP * 4, 16);
  P.off_seg = off;  off += (uint32_t)(kSegMax * sizeof(Seg));
  P.off_bar = off;  off += (uint32_t)round_up((int32_t)sizeof(Bars), 16);
  P.off_misc = off; off += 64;
  const size_t smem_bytes = off + 1024;  // slack for the in-kernel 1024-byte alignment

  const int64_t tiles_m = (g.Mtot + P.TP - 1) / P.TP;
  const int64_t nblocks = tiles_m * P.n_ntiles;
  if (nblocks > INT32_MAX) return IM2WIN_EUNSUPPORTED;
  cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem_bytes);
  if (e != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  conv_tc_kernel<<<(unsigned)nblocks, kThreads, smem_bytes, st>>>(P);
  note_kernel(KERNEL_GENERIC);
  return cuda_status(cudaGetLastError());
}

}  // namespace im2win
