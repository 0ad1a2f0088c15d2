// Internal declarations shared by the translation units of libim2win (device library only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "im2win.h"

namespace im2win {

// Sizes derived once on the host and handed to every kernel by value.
struct Geometry {
  int32_t N, C, H, W, K, Fh, Fw, s;
  int32_t Ho, Wo;
  int32_t L;        // strip length W*Fh (floats)
  int32_t FF;       // Fh*Fw, the contiguous run one window occupies in a strip
  int32_t sFh;      // s*Fh, distance between consecutive windows in a strip
  int64_t HoL;      // Ho*L, one (image, channel) plane of the im2win tensor
  int64_t HoWo;     // one (image, filter) plane of the output
  int64_t Kg;       // C*Fh*Fw, the reduction length
  int64_t Mtot;     // N*Ho*Wo, number of output positions
  int64_t n_in, n_win, n_col, n_out, n_flt;  // element counts
};

// Fills g from shape; returns IM2WIN_OK or IM2WIN_EINVAL (bad sizes / 64-bit overflow).
int make_geometry(const im2win_shape* shape, Geometry* g);

// Device status word (one per loaded library).  Codes written by kernels:
enum : int32_t {
  DEV_OK = 0,
  DEV_TIMEOUT_RAW_FULL = 101,   // repack warps waiting for a staged strip
  DEV_TIMEOUT_RAW_EMPTY = 102,  // producer waiting for a free strip stage
  DEV_TIMEOUT_A_FULL = 103,     // MMA thread waiting for window columns in TMEM
  DEV_TIMEOUT_A_EMPTY = 104,    // repack warps waiting for a free TMEM slot
  DEV_TIMEOUT_B_FULL = 105,     // MMA thread waiting for a filter tile
  DEV_TIMEOUT_B_EMPTY = 106,    // filter loaders waiting for a free stage
  DEV_TIMEOUT_ACC = 107,        // epilogue waiting for the accumulator
  DEV_TIMEOUT_DRAIN = 108,      // teardown waiting for copies in flight
  DEV_TIMEOUT_COPY = 109,       // transform waiting for the bulk copy of its input range
  DEV_RANGE = 201               // an internal index check failed
};
int32_t* device_status_word();  // device address of the status word (nullptr if no device)

// Launchers (all asynchronous on `st`; return a cudaError_t-derived im2win status).
int launch_transform(const float* in, float* out, const Geometry& g, cudaStream_t st);
int launch_transform_bf16(const float* in, uint16_t* out, const Geometry& g, cudaStream_t st);
int launch_conv_fp32(const float* xhat, const float* f, float* out, const Geometry& g, cudaStream_t st);
// Tensor-core convolution: the persistent specialised kernel when one applies (it returns
// IM2WIN_EUNSUPPORTED otherwise), else the generic kernel.
int launch_conv_tc_persistent(const void* src, const float* f, float* out, const Geometry& g, int mode,
                              cudaStream_t st, bool may_alloc, bool fused = false, bool src_bf16 = false, bool out_bf16 = false);
int launch_conv_tc_generic(const float* xhat, const float* f, float* out, const Geometry& g, int mode,
                           cudaStream_t st);
// may_alloc = false keeps the call free of any (even stream-ordered) device allocation.
int launch_conv_tc(const float* xhat, const float* f, float* out, const Geometry& g, int mode,
                   cudaStream_t st, bool may_alloc = true);

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? IM2WIN_OK : IM2WIN_ECUDA; }

}  // namespace im2win
