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
  int32_t out_nhwc;  // the fp32 output is written N x Ho x Wo x K (im2win_conv_nhwc) instead of N x K x Ho x Wo
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
// Device memory from the caller's workspace (beyond the im2win tensor) that a tensor-core convolution
// may use for a re-laid-out copy of the filter; ptr may be null / bytes 0 (kernels that need such a
// copy then return IM2WIN_EUNSUPPORTED and the dispatcher moves on).  The library allocates nothing.
struct Scratch {
  void* ptr = nullptr;
  size_t bytes = 0;
};
// Tensor-core convolution kernels.  Each returns IM2WIN_EUNSUPPORTED when it does not apply (shape,
// scratch) before anything is enqueued; launch_conv_tc tries them in order of expected speed.
// src_kind: 0 = fp32 im2win tensor, 1 = untransformed input consumed fused, 2 = bf16 im2win tensor.
// (even_if_slower: take the problem wherever the kernel is implemented, not only where it is expected to
// be the fastest -- for sources no other kernel accepts)
int launch_conv_tc_strip(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                         Scratch scratch, int src_kind, bool out_bf16, bool even_if_slower = false);
int launch_conv_tc_persistent(const void* src, const float* f, float* out, const Geometry& g, int mode,
                              cudaStream_t st, Scratch scratch, bool fused = false, bool src_bf16 = false,
                              bool out_bf16 = false);
int launch_conv_tc_generic(const float* xhat, const float* f, float* out, const Geometry& g, int mode,
                           cudaStream_t st);
int launch_conv_tc(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                   Scratch scratch, int src_kind, bool out_bf16);
// Scratch bytes with which every kernel above is available for this problem (0 if none wants any).
size_t strip_scratch_bytes(const Geometry& g, int mode, int src_kind);
// The window-offset kernel (conv_tc_window.cu; stride 1, 3x3 and 5x5): same source kinds and scratch rules.
int launch_conv_tc_window(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                          Scratch scratch, int src_kind, bool out_bf16, bool even_if_slower = false);
size_t window_scratch_bytes(const Geometry& g, int mode, int src_kind);
size_t persistent_scratch_bytes(const Geometry& g, int mode);
size_t conv_scratch_bytes(const Geometry& g, int mode, int src_kind);
// Shared body of im2win_conv / im2win_conv_bf16out / im2win_conv_static (argument checks, workspace
// split into the im2win tensor and the filter scratch, transform, dispatch).
int conv_impl(const void* src, int src_kind, const float* filter, const im2win_shape* shape, int mode, void* out,
              bool out16, void* workspace, size_t workspace_bytes, void* cuda_stream, bool out_nhwc = false);

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? IM2WIN_OK : IM2WIN_ECUDA; }

// Diagnostic switches of the launchers.  The product library answers knobs() with the constant
// defaults below and reads no environment; only the test build of api.cu (-DIM2WIN_TEST_KNOBS,
// linked into libim2win_test.so) keeps a mutable copy and exports im2win_debug_set_option(name, value)
// to set a field by name, which is how the parity tests force each kernel configuration.
struct Knobs {
  int force_generic = 0;     // every tensor-core convolution through the generic kernel
  int no_strip = 0;          // never use the strip-matrix kernel (conv_tc_strip.cu)
  int force_strip = 0;       // use the strip-matrix kernel wherever it is implemented, not only where its cost model picks it
  int no_box = 0;            // persistent kernel: strips by bulk copies instead of 2-D TMA boxes
  int no_pim = 0;            // persistent kernel: tiles may span images
  int bslice = 0;            // persistent kernel: force the slice-resident filter mode
  int no_bslice = 0;         // persistent kernel: never use it
  int splitk = -1;           // persistent kernel: force this many reduction slices (-1: cost model)
  int force_stream = 0;      // persistent kernel: stream the filter although it would fit
  int nsets = 0;             // persistent kernel: 2 or 3 repack sets (0: own choice)
  int no_l2ahead = 0;        // persistent kernel: no L2 prefetch of the next tile's boxes
  int no_btma = 0;           // persistent kernel: resident filter built by threads, not fetched by TMA
  int ntiles = 0;            // persistent kernel: number of filter tiles (0: own choice)
  int transform_budget_kb = 0;  // transform tile kernel: shared-memory budget per CTA in KB (0: own choice)
  int transform_gather = 0;  // transform: the staged-gather kernel instead of the tile kernel
  int test_skip_copy = 0;    // transform tile kernel, single-CTA problems: announce the input copy, never issue it
  int strip_mh = 0;          // strip-matrix kernel: 128-row halves per tile (0: own choice)
  int strip_pair = 0;        // strip-matrix kernel: 1 = CTA pairs (cta_group::2) forced, 2 = single CTAs forced, 0 = own choice
  int force_window = 0;      // use the window-offset kernel (conv_tc_window.cu) wherever it is implemented
  int no_window = 0;         // never use it
  int window_mh = 0;         // window-offset kernel: 128-row blocks per tile (0: own choice)
  int window_plan = 0;       // window-offset kernel: forced split of shared memory (0: own choice)
  int window_pair = 0;       // window-offset kernel: 1 = CTA pairs forced, 2 = single CTAs forced, 0 = own choice
  int window_bres = 0;       // window-offset kernel: 1 = resident filter or nothing, 2 = never resident, 0 = own choice
  int window_nohelp = 0;     // window-offset kernel: the interleaver warps never help the epilogue
  int window_two = 0;        // window-offset kernel: 1 = two MMA-issuing threads forced, 2 = one forced, 0 = own choice
};
const Knobs& knobs();

// Which convolution kernel the last launch on this host thread's library image used (a diagnostic the
// test build exposes as im2win_debug_last_kernel; the product library only writes it).
enum : int { KERNEL_NONE = 0, KERNEL_STRIP = 1, KERNEL_PERSISTENT = 2, KERNEL_GENERIC = 3, KERNEL_FP32 = 4, KERNEL_WINDOW = 5 };
void note_kernel(int which);
// The launch plan of the last strip-matrix / window-offset launch (same diagnostic): up to eight integers.
void note_plan(const int* v, int n);

// Streaming multiprocessors of the current device (cached per device).
int sm_count();

}  // namespace im2win
