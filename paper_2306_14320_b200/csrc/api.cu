// C-ABI entry points: argument checks, size queries and dispatch to the kernels.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace im2win {

namespace {

__device__ int32_t g_status_word = 0;

bool mul_ok(int64_t a, int64_t b, int64_t* out) {
  if (a < 0 || b < 0) return false;
  if (a != 0 && b > INT64_MAX / a) return false;
  *out = a * b;
  return true;
}

bool prod(int64_t* out, std::initializer_list<int64_t> v) {
  int64_t p = 1;
  for (int64_t x : v)
    if (!mul_ok(p, x, &p)) return false;
  // keep byte counts (x4) and float offsets comfortably inside int64 / size_t
  if (p > (INT64_MAX >> 4)) return false;
  *out = p;
  return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool overlap(const void* a, int64_t abytes, const void* b, int64_t bbytes) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + (uintptr_t)bbytes && b0 < a0 + (uintptr_t)abytes;
}

}  // namespace

int make_geometry(const im2win_shape* sh, Geometry* g) {
  if (!sh || !g) return IM2WIN_EINVAL;
  if (sh->N < 1 || sh->C < 1 || sh->H < 1 || sh->W < 1 || sh->K < 1 || sh->Fh < 1 || sh->Fw < 1 ||
      sh->stride < 1)
    return IM2WIN_EINVAL;
  if (sh->Fh > sh->H || sh->Fw > sh->W) return IM2WIN_EINVAL;
  g->N = sh->N; g->C = sh->C; g->H = sh->H; g->W = sh->W;
  g->K = sh->K; g->Fh = sh->Fh; g->Fw = sh->Fw; g->s = sh->stride;
  g->out_nhwc = 0;
  g->Ho = (sh->H - sh->Fh) / sh->stride + 1;
  g->Wo = (sh->W - sh->Fw) / sh->stride + 1;
  int64_t L, FF, sFh;
  if (!prod(&L, {sh->W, sh->Fh}) || !prod(&FF, {sh->Fh, sh->Fw}) || !prod(&sFh, {sh->stride, sh->Fh}))
    return IM2WIN_EINVAL;
  if (L > INT32_MAX / 4 || FF > INT32_MAX / 4 || sFh > INT32_MAX / 4) return IM2WIN_EINVAL;
  g->L = (int32_t)L; g->FF = (int32_t)FF; g->sFh = (int32_t)sFh;
  if (!prod(&g->HoL, {g->Ho, L}) || !prod(&g->HoWo, {g->Ho, g->Wo}) || !prod(&g->Kg, {sh->C, FF}) ||
      !prod(&g->Mtot, {sh->N, g->HoWo}) || !prod(&g->n_in, {sh->N, sh->C, sh->H, sh->W}) ||
      !prod(&g->n_win, {sh->N, sh->C, g->HoL}) || !prod(&g->n_col, {sh->N, sh->C, FF, g->HoWo}) ||
      !prod(&g->n_out, {sh->N, sh->K, g->HoWo}) || !prod(&g->n_flt, {sh->K, g->Kg}))
    return IM2WIN_EINVAL;
  return IM2WIN_OK;
}

int launch_conv_tc(const void* src, const float* f, float* out, const Geometry& g, int mode, cudaStream_t st,
                   Scratch scratch, int src_kind, bool out_bf16) {
  // src_kind: 0 = fp32 im2win tensor, 1 = untransformed input consumed fused, 2 = bf16 im2win tensor.
  // Order: the window-offset and the strip-matrix kernel where each is implemented and expected to win, else
  // the persistent specialised kernel, else (fp32 im2win tensor and fp32 output only) the generic kernel.
  int rc = IM2WIN_EUNSUPPORTED;
  if (!knobs().force_generic) {
    rc = launch_conv_tc_window(src, f, out, g, mode, st, scratch, src_kind, out_bf16);
    if (rc != IM2WIN_EUNSUPPORTED) return rc;
    if (!knobs().no_strip) rc = launch_conv_tc_strip(src, f, out, g, mode, st, scratch, src_kind, out_bf16);
    if (rc != IM2WIN_EUNSUPPORTED) return rc;
    rc = launch_conv_tc_persistent(src, f, out, g, mode, st, scratch, src_kind == 1, src_kind == 2, out_bf16);
    if (rc != IM2WIN_EUNSUPPORTED) return rc;
    // sources the generic kernel does not read (bf16 im2win tensor, fused): the strip-matrix or the
    // window-offset kernel wherever one applies
    if (src_kind != 0 && !knobs().no_strip) {
      rc = launch_conv_tc_strip(src, f, out, g, mode, st, scratch, src_kind, out_bf16, /*even_if_slower=*/true);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
    if (src_kind != 0) {
      rc = launch_conv_tc_window(src, f, out, g, mode, st, scratch, src_kind, out_bf16, /*even_if_slower=*/true);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
  }
  if (src_kind != 0 || out_bf16) return IM2WIN_EUNSUPPORTED;
  return launch_conv_tc_generic(static_cast<const float*>(src), f, out, g, mode, st);
}

size_t conv_scratch_bytes(const Geometry& g, int mode, int src_kind) {
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16) return 0;
  const size_t a = strip_scratch_bytes(g, mode, src_kind), b = persistent_scratch_bytes(g, mode);
  const size_t c = knobs().no_window ? 0 : window_scratch_bytes(g, mode, src_kind);
  return a > b ? (a > c ? a : c) : (b > c ? b : c);
}

#ifdef IM2WIN_TEST_KNOBS
static Knobs g_knobs;
const Knobs& knobs() { return g_knobs; }
#else
const Knobs& knobs() {
  static const Knobs defaults;
  return defaults;
}
#endif

static std::atomic<int> g_last_kernel{KERNEL_NONE};
void note_kernel(int which) { g_last_kernel.store(which, std::memory_order_relaxed); }
static std::atomic<int> g_last_plan[8];
void note_plan(const int* v, int n) {
  for (int i = 0; i < 8; ++i) g_last_plan[i].store(i < n ? v[i] : 0, std::memory_order_relaxed);
}

int sm_count() {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cached[kMaxDev];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { cudaGetLastError(); return 148; }
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 148;
  }
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

int32_t* device_status_word() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return static_cast<int32_t*>(p);
}

}  // namespace im2win

using namespace im2win;

extern "C" {

int im2win_out_dims(const im2win_shape* shape, int32_t* Ho, int32_t* Wo) {
  Geometry g;
  if (!Ho || !Wo) return IM2WIN_EINVAL;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  *Ho = g.Ho;
  *Wo = g.Wo;
  return IM2WIN_OK;
}

int im2win_workspace_bytes(const im2win_shape* shape, size_t* bytes) {
  Geometry g;
  if (!bytes) return IM2WIN_EINVAL;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  *bytes = (size_t)g.n_win * sizeof(float);
  return IM2WIN_OK;
}

int im2win_im2col_bytes(const im2win_shape* shape, size_t* bytes) {
  Geometry g;
  if (!bytes) return IM2WIN_EINVAL;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  *bytes = (size_t)g.n_col * sizeof(float);
  return IM2WIN_OK;
}

int im2win_transform(const float* in_nchw, const im2win_shape* shape, float* out_im2win,
                     void* cuda_stream) {
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!in_nchw || !out_im2win) return IM2WIN_EINVAL;
  if (!aligned16(in_nchw) || !aligned16(out_im2win)) return IM2WIN_EALIGN;
  if (overlap(in_nchw, g.n_in * 4, out_im2win, g.n_win * 4)) return IM2WIN_EOVERLAP;
  return launch_transform(in_nchw, out_im2win, g, static_cast<cudaStream_t>(cuda_stream));
}

int im2win_workspace_bytes_bf16(const im2win_shape* shape, size_t* bytes) {
  Geometry g;
  const int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!bytes) return IM2WIN_EINVAL;
  *bytes = (size_t)g.n_win * 2;
  return IM2WIN_OK;
}

int im2win_transform_bf16(const float* in_nchw, const im2win_shape* shape, uint16_t* out_im2win_bf16,
                          void* cuda_stream) {
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!in_nchw || !out_im2win_bf16) return IM2WIN_EINVAL;
  if (!aligned16(in_nchw) || !aligned16(out_im2win_bf16)) return IM2WIN_EALIGN;
  if (overlap(in_nchw, g.n_in * 4, out_im2win_bf16, g.n_win * 2)) return IM2WIN_EOVERLAP;
  return launch_transform_bf16(in_nchw, out_im2win_bf16, g, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

namespace im2win {

// Shared body of im2win_conv (fp32 output), im2win_conv_bf16out (out16: `out` holds 16-bit words;
// tensor-core modes, kernels with a bf16 epilogue) and im2win_conv_static.
int conv_impl(const void* src, int src_kind, const float* filter, const im2win_shape* shape, int mode, void* out,
              bool out16, void* workspace, size_t workspace_bytes, void* cuda_stream, bool out_nhwc) {
  float* const out_nchw = static_cast<float*>(out);
  const int64_t out_es = out16 ? 2 : 4;
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (out_nhwc && out16) return IM2WIN_EINVAL;
  g.out_nhwc = out_nhwc ? 1 : 0;
  if (!src || !filter || !out_nchw) return IM2WIN_EINVAL;
  if (src_kind != IM2WIN_SRC_NCHW && src_kind != IM2WIN_SRC_IM2WIN && src_kind != IM2WIN_SRC_NCHW_FUSED &&
      src_kind != IM2WIN_SRC_IM2WIN_BF16)
    return IM2WIN_EINVAL;
  if (src_kind == IM2WIN_SRC_IM2WIN_BF16 && mode != IM2WIN_MODE_BF16) return IM2WIN_EINVAL;
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16 && mode != IM2WIN_MODE_FP32)
    return IM2WIN_EINVAL;
  if (out16 && mode == IM2WIN_MODE_FP32) return IM2WIN_EINVAL;
  if (!aligned16(src) || !aligned16(filter) || !aligned16(out_nchw)) return IM2WIN_EALIGN;
  const int64_t src_bytes = src_kind == IM2WIN_SRC_IM2WIN_BF16 ? g.n_win * 2
                                                                : (src_kind == IM2WIN_SRC_IM2WIN ? g.n_win : g.n_in) * 4;
  if (overlap(out_nchw, g.n_out * out_es, src, src_bytes) || overlap(out_nchw, g.n_out * out_es, filter, g.n_flt * 4))
    return IM2WIN_EOVERLAP;
  // The workspace: first the im2win tensor (src_kind NCHW, or the fallback of NCHW_FUSED), then, from the
  // next 256-byte boundary, whatever is left as scratch for a re-laid-out copy of the filter.
  uint8_t* const ws = static_cast<uint8_t*>(workspace);
  const size_t ws_bytes = ws ? workspace_bytes : 0;
  const size_t win_bytes = (size_t)g.n_win * 4;
  if (src_kind == IM2WIN_SRC_NCHW && ws_bytes < win_bytes) return IM2WIN_EWORKSPACE;
  if (ws_bytes) {
    if (!aligned16(ws)) return IM2WIN_EALIGN;
    if (ws_bytes > (size_t)INT64_MAX || overlap(ws, (int64_t)ws_bytes, src, src_bytes) ||
        overlap(ws, (int64_t)ws_bytes, out_nchw, g.n_out * out_es) || overlap(ws, (int64_t)ws_bytes, filter, g.n_flt * 4))
      return IM2WIN_EOVERLAP;
  }
  auto scratch_from = [&](size_t offset) {
    Scratch sc;
    offset = (offset + 255) / 256 * 256;
    if (ws_bytes > offset) { sc.ptr = ws + offset; sc.bytes = ws_bytes - offset; }
    return sc;
  };
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (src_kind == IM2WIN_SRC_IM2WIN_BF16) {  // (no generic-kernel fallback for this storage variant)
    if (knobs().force_generic) return IM2WIN_EUNSUPPORTED;
    return launch_conv_tc(src, filter, out_nchw, g, mode, st, scratch_from(0), 2, out16);
  }
  const float* xhat = static_cast<const float*>(src);
  if (src_kind == IM2WIN_SRC_NCHW_FUSED) {
    if (mode != IM2WIN_MODE_FP32 && !knobs().force_generic) {
      rc = launch_conv_tc_window(xhat, filter, out_nchw, g, mode, st, scratch_from(0), 1, out16);
      if (rc == IM2WIN_EUNSUPPORTED && !knobs().no_strip)
        rc = launch_conv_tc_strip(xhat, filter, out_nchw, g, mode, st, scratch_from(0), 1, out16);
      if (rc == IM2WIN_EUNSUPPORTED)
        rc = launch_conv_tc_persistent(xhat, filter, out_nchw, g, mode, st, scratch_from(0), /*fused=*/true,
                                       /*src_bf16=*/false, out16);
      if (rc == IM2WIN_EUNSUPPORTED && !knobs().no_strip)
        rc = launch_conv_tc_strip(xhat, filter, out_nchw, g, mode, st, scratch_from(0), 1, out16, /*even_if_slower=*/true);
      if (rc == IM2WIN_EUNSUPPORTED)
        rc = launch_conv_tc_window(xhat, filter, out_nchw, g, mode, st, scratch_from(0), 1, out16, /*even_if_slower=*/true);
      if (rc != IM2WIN_EUNSUPPORTED) return rc;
    }
    // no fused kernel for this shape or mode: the unfused path, if the caller supplied a workspace
    if (ws_bytes < win_bytes) return IM2WIN_EUNSUPPORTED;
    src_kind = IM2WIN_SRC_NCHW;
  }
  Scratch scratch = scratch_from(0);
  if (src_kind == IM2WIN_SRC_NCHW) {
    rc = launch_transform(static_cast<const float*>(src), reinterpret_cast<float*>(ws), g, st);
    if (rc != IM2WIN_OK) return rc;
    xhat = reinterpret_cast<const float*>(ws);
    scratch = scratch_from(win_bytes);
  }
  if (mode == IM2WIN_MODE_FP32) return launch_conv_fp32(xhat, filter, out_nchw, g, st);
  return launch_conv_tc(xhat, filter, out_nchw, g, mode, st, scratch, 0, out16);
}

}  // namespace im2win

extern "C" {

int im2win_conv_workspace_bytes(const im2win_shape* shape, int src_kind, int mode, size_t* bytes) {
  Geometry g;
  const int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!bytes) return IM2WIN_EINVAL;
  if (src_kind != IM2WIN_SRC_NCHW && src_kind != IM2WIN_SRC_IM2WIN && src_kind != IM2WIN_SRC_NCHW_FUSED &&
      src_kind != IM2WIN_SRC_IM2WIN_BF16)
    return IM2WIN_EINVAL;
  if (mode != IM2WIN_MODE_TF32 && mode != IM2WIN_MODE_BF16 && mode != IM2WIN_MODE_FP32) return IM2WIN_EINVAL;
  const size_t win = src_kind == IM2WIN_SRC_NCHW ? ((size_t)g.n_win * 4 + 255) / 256 * 256 : 0;
  const int kind = src_kind == IM2WIN_SRC_NCHW_FUSED ? 1 : (src_kind == IM2WIN_SRC_IM2WIN_BF16 ? 2 : 0);
  const size_t extra = conv_scratch_bytes(g, mode, kind);
  *bytes = extra ? win + extra : (src_kind == IM2WIN_SRC_NCHW ? (size_t)g.n_win * 4 : 0);
  return IM2WIN_OK;
}

int im2win_conv(const void* src, int src_kind, const float* filter, const im2win_shape* shape,
                int mode, float* out_nchw, void* workspace, size_t workspace_bytes,
                void* cuda_stream) {
  return conv_impl(src, src_kind, filter, shape, mode, out_nchw, false, workspace, workspace_bytes, cuda_stream);
}

int im2win_conv_nhwc(const void* src, int src_kind, const float* filter, const im2win_shape* shape,
                     int mode, float* out_nhwc, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return conv_impl(src, src_kind, filter, shape, mode, out_nhwc, false, workspace, workspace_bytes, cuda_stream, true);
}

int im2win_conv_bf16out(const void* src, int src_kind, const float* filter, const im2win_shape* shape,
                        int mode, uint16_t* out_nchw_bf16, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  return conv_impl(src, src_kind, filter, shape, mode, out_nchw_bf16, true, workspace, workspace_bytes, cuda_stream);
}

int im2win_last_device_status(void* cuda_stream, int32_t* status) {
  if (!status) return IM2WIN_EINVAL;
  int32_t* word = device_status_word();
  if (!word) return IM2WIN_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return IM2WIN_ECUDA;
  int32_t v = 0;
  if (cudaMemcpy(&v, word, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return IM2WIN_ECUDA;
  if (v != 0 && cudaMemset(word, 0, sizeof(v)) != cudaSuccess) return IM2WIN_ECUDA;
  *status = v;
  // an expired bounded wait (codes 101..199) is reported as such; the raw code stays in *status
  return (v >= 100 && v < 200) ? IM2WIN_ETIMEOUT : IM2WIN_OK;
}

#ifdef IM2WIN_TEST_KNOBS
// Test build only: which convolution kernel the last call launched (KERNEL_* of common.cuh).
int im2win_debug_last_kernel(void) { return g_last_kernel.load(std::memory_order_relaxed); }

// Test build only (libim2win_test.so): set one diagnostic switch by name.  Returns IM2WIN_EINVAL for
// an unknown name.
void im2win_debug_last_plan(int* out8) {
  for (int i = 0; i < 8; ++i) out8[i] = im2win::g_last_plan[i].load(std::memory_order_relaxed);
}
int im2win_debug_set_option(const char* name, int value) {
  if (!name) return IM2WIN_EINVAL;
  struct Entry { const char* name; int Knobs::*field; };
  static const Entry table[] = {
      {"force_generic", &Knobs::force_generic}, {"no_strip", &Knobs::no_strip}, {"force_strip", &Knobs::force_strip},
      {"no_box", &Knobs::no_box}, {"no_pim", &Knobs::no_pim}, {"bslice", &Knobs::bslice},
      {"no_bslice", &Knobs::no_bslice}, {"splitk", &Knobs::splitk}, {"force_stream", &Knobs::force_stream},
      {"nsets", &Knobs::nsets}, {"no_l2ahead", &Knobs::no_l2ahead}, {"no_btma", &Knobs::no_btma},
      {"ntiles", &Knobs::ntiles}, {"transform_gather", &Knobs::transform_gather},
      {"test_skip_copy", &Knobs::test_skip_copy}, {"strip_mh", &Knobs::strip_mh}, {"strip_pair", &Knobs::strip_pair},
      {"force_window", &Knobs::force_window}, {"no_window", &Knobs::no_window}, {"window_mh", &Knobs::window_mh},
      {"window_plan", &Knobs::window_plan}, {"window_pair", &Knobs::window_pair}, {"window_two", &Knobs::window_two}, {"window_nohelp", &Knobs::window_nohelp}, {"window_bres", &Knobs::window_bres}, {"transform_budget_kb", &Knobs::transform_budget_kb}};
  for (const Entry& e : table)
    if (strcmp(e.name, name) == 0) { g_knobs.*(e.field) = value; return IM2WIN_OK; }
  return IM2WIN_EINVAL;
}
#endif

const char* im2win_strerror(int status) {
  switch (status) {
    case IM2WIN_OK: return "ok";
    case IM2WIN_EINVAL: return "invalid argument (null pointer, size < 1, filter larger than input, unknown enum or size overflow)";
    case IM2WIN_EALIGN: return "device pointer is not 16-byte aligned";
    case IM2WIN_EWORKSPACE: return "workspace missing or smaller than im2win_workspace_bytes";
    case IM2WIN_EOVERLAP: return "output range overlaps an input or workspace range";
    case IM2WIN_ECUDA: return "CUDA runtime call or kernel launch failed (no device, or see cudaGetLastError)";
    case IM2WIN_ETIMEOUT: return "a bounded device-side wait expired";
    case IM2WIN_EUNSUPPORTED: return "shape outside what the tensor-core kernels implement";
    case IM2WIN_ESCRATCH: return "the problem's im2win tensor is larger than the library's built-in scratch buffer";
    default: return "unknown im2win status";
  }
}

// ---------------------------------------------------------------------------------------------
// Host-buffer convenience path: the batch is cut into chunks of images that flow through three
// streams (host->device copy, kernels, device->host copy), so that the two copy directions and the
// compute overlap; images are independent, so a chunk is a complete problem of its own.

namespace {
constexpr int kHostChunks = 8;
struct HostCtx {
  cudaStream_t s_in = nullptr, s_cmp = nullptr, s_out = nullptr;
  cudaEvent_t ev_in[kHostChunks + 1] = {}, ev_cmp[kHostChunks] = {};
  float *d_in = nullptr, *d_f = nullptr, *d_out = nullptr, *d_ws = nullptr;
  size_t b_in = 0, b_f = 0, b_out = 0, b_ws = 0;
  bool ready = false;
} g_host;

int grow(float** p, size_t* have, size_t need) {
  if (*have >= need) return IM2WIN_OK;
  if (*p) cudaFree(*p);
  *p = nullptr;
  *have = 0;
  if (cudaMalloc(reinterpret_cast<void**>(p), need) != cudaSuccess) {
    cudaGetLastError();
    return IM2WIN_ECUDA;
  }
  *have = need;
  return IM2WIN_OK;
}

int host_ctx_init() {
  if (g_host.ready) return IM2WIN_OK;
  for (cudaStream_t* st : {&g_host.s_in, &g_host.s_cmp, &g_host.s_out})
    if (cudaStreamCreateWithFlags(st, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  for (cudaEvent_t& e : g_host.ev_in)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  for (cudaEvent_t& e : g_host.ev_cmp)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return IM2WIN_ECUDA; }
  g_host.ready = true;
  return IM2WIN_OK;
}
}  // namespace

int im2win_conv_host(const float* in_host, const float* filter_host, const im2win_shape* shape,
                     int mode, float* out_host) {
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != IM2WIN_OK) return rc;
  if (!in_host || !filter_host || !out_host) return IM2WIN_EINVAL;
  if ((rc = host_ctx_init()) != IM2WIN_OK) return rc;
  const int64_t in_img = g.n_in / g.N, out_img = g.n_out / g.N, win_img = g.n_win / g.N;
  // images per chunk: about an eighth of the batch, and such that every chunk starts on a
  // 16-byte boundary of the device input and output buffers (the kernels require aligned bases)
  auto need = [](int64_t img_floats) { return img_floats % 4 == 0 ? 1 : (img_floats % 2 == 0 ? 2 : 4); };
  const int mult = need(in_img) > need(out_img) ? need(in_img) : need(out_img);
  int per = (g.N + kHostChunks - 1) / kHostChunks;
  per = (per + mult - 1) / mult * mult;
  const int nchunks = (g.N + per - 1) / per;
  if ((rc = grow(&g_host.d_in, &g_host.b_in, (size_t)g.n_in * 4)) != IM2WIN_OK) return rc;
  if ((rc = grow(&g_host.d_f, &g_host.b_f, (size_t)g.n_flt * 4)) != IM2WIN_OK) return rc;
  if ((rc = grow(&g_host.d_out, &g_host.b_out, (size_t)g.n_out * 4)) != IM2WIN_OK) return rc;
  // workspace for one chunk: the im2win tensor (only the shapes without a fused kernel use it) and
  // behind it the scratch the tensor-core kernels may want for a copy of the filter
  size_t ws_need = ((size_t)win_img * per * 4 + 255) / 256 * 256;
  {
    im2win_shape shc = *shape;
    shc.N = per;
    Geometry gc;
    if (make_geometry(&shc, &gc) == IM2WIN_OK) {
      const size_t a = conv_scratch_bytes(gc, mode, 0), b = conv_scratch_bytes(gc, mode, 1);
      ws_need += a > b ? a : b;
    }
  }
  if ((rc = grow(&g_host.d_ws, &g_host.b_ws, ws_need)) != IM2WIN_OK) return rc;
  if (cudaMemcpyAsync(g_host.d_f, filter_host, (size_t)g.n_flt * 4, cudaMemcpyHostToDevice, g_host.s_in) != cudaSuccess ||
      cudaEventRecord(g_host.ev_in[kHostChunks], g_host.s_in) != cudaSuccess ||
      cudaStreamWaitEvent(g_host.s_cmp, g_host.ev_in[kHostChunks], 0) != cudaSuccess)
    return IM2WIN_ECUDA;
  for (int c = 0; c < nchunks; ++c) {
    const int i0 = c * per, n = (i0 + per <= g.N ? per : g.N - i0);
    if (n <= 0) break;
    im2win_shape sh = *shape;
    sh.N = n;
    const float* hin = in_host + (int64_t)i0 * in_img;
    float* din = g_host.d_in + (int64_t)i0 * in_img;
    float* dout = g_host.d_out + (int64_t)i0 * out_img;
    if (cudaMemcpyAsync(din, hin, (size_t)n * in_img * 4, cudaMemcpyHostToDevice, g_host.s_in) != cudaSuccess ||
        cudaEventRecord(g_host.ev_in[c], g_host.s_in) != cudaSuccess ||
        cudaStreamWaitEvent(g_host.s_cmp, g_host.ev_in[c], 0) != cudaSuccess)
      return IM2WIN_ECUDA;
    // fused where a specialisation exists (the workspace then stays untouched), else transform + convolution
    rc = im2win_conv(din, IM2WIN_SRC_NCHW_FUSED, g_host.d_f, &sh, mode, dout, g_host.d_ws, g_host.b_ws, g_host.s_cmp);
    if (rc != IM2WIN_OK) return rc;
    if (cudaEventRecord(g_host.ev_cmp[c], g_host.s_cmp) != cudaSuccess ||
        cudaStreamWaitEvent(g_host.s_out, g_host.ev_cmp[c], 0) != cudaSuccess ||
        cudaMemcpyAsync(out_host + (int64_t)i0 * out_img, dout, (size_t)n * out_img * 4, cudaMemcpyDeviceToHost,
                        g_host.s_out) != cudaSuccess)
      return IM2WIN_ECUDA;
  }
  if (cudaStreamSynchronize(g_host.s_out) != cudaSuccess) return IM2WIN_ECUDA;
  return IM2WIN_OK;
}

int im2win_host_release(void) {
  if (g_host.ready) {
    cudaStreamSynchronize(g_host.s_in);
    cudaStreamSynchronize(g_host.s_cmp);
    cudaStreamSynchronize(g_host.s_out);
  }
  for (float** p : {&g_host.d_in, &g_host.d_f, &g_host.d_out, &g_host.d_ws})
    if (*p) { cudaFree(*p); *p = nullptr; }
  g_host.b_in = g_host.b_f = g_host.b_out = g_host.b_ws = 0;
  if (g_host.ready) {
    for (cudaEvent_t& e : g_host.ev_in) cudaEventDestroy(e);
    for (cudaEvent_t& e : g_host.ev_cmp) cudaEventDestroy(e);
    cudaStreamDestroy(g_host.s_in);
    cudaStreamDestroy(g_host.s_cmp);
    cudaStreamDestroy(g_host.s_out);
    g_host = HostCtx{};
  }
  return IM2WIN_OK;
}

}  // extern "C"
