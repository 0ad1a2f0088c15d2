/*
 * im2win on NVIDIA B200 (sm_100a): the im2win data transformation and the
 * im2win-based convolution, behind a plain C ABI.
 *
 * Notation follows the paper: input I[N][C][H][W], filter F[K][C][Fh][Fw],
 * output O[N][K][Ho][Wo], one stride s for both directions, no padding, no
 * dilation, no groups, no bias, no filter flip (Section II-A, Eq. 1).  All
 * tensors are dense, row-major and flat in memory (Section I) in fp32.
 * The im2win tensor is Ihat[N][C][Ho][W*Fh] (Section III-A, Algorithm 1).
 *
 * Unless a function says HOST, data pointers are DEVICE pointers owned by the
 * caller; the library never frees or keeps them.  Shapes are passed by pointer
 * to a plain struct in host memory that is read before the call returns.
 * Device work is enqueued on the CUDA stream given as `cuda_stream`
 * (a cudaStream_t cast to void*; NULL = the default stream) and the call
 * returns without synchronising.  Every function returns IM2WIN_OK (0) or a
 * negative im2win_status.  Argument errors (EINVAL, EALIGN, EWORKSPACE,
 * EOVERLAP, ESCRATCH) are found before anything is launched; EUNSUPPORTED
 * and ECUDA from im2win_conv with src_kind NCHW can come after the transform
 * has been enqueued (the workspace then holds the im2win tensor).
 * The library allocates no device memory in any call on device pointers
 * (im2win_conv_host, which works on host buffers, owns its device buffers).
 * There is no CPU fallback: without a CUDA device the launching calls return
 * IM2WIN_ECUDA.
 */
#ifndef IM2WIN_H
#define IM2WIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t N, C, H, W;  /* input  I[N][C][H][W]                      */
  int32_t K, Fh, Fw;   /* filter F[K][C][Fh][Fw]                    */
  int32_t stride;      /* s >= 1, the same in both directions       */
} im2win_shape;

/* What `src` of im2win_conv points to. */
enum { IM2WIN_SRC_NCHW = 0,   /* the untransformed input I; the call runs the transform first   */
       IM2WIN_SRC_IM2WIN = 1, /* an im2win tensor Ihat produced earlier by im2win_transform      */
       IM2WIN_SRC_NCHW_FUSED = 2, /* the untransformed input I; each tile's window rows are built
                                    on the fly in shared memory, no im2win tensor reaches memory   */
       IM2WIN_SRC_IM2WIN_BF16 = 3 /* an im2win tensor stored as bf16 by im2win_transform_bf16
                                    (a storage variant of this build, not in the paper)            */ };

/* Arithmetic of the contraction.  Products are accumulated in fp32 in every mode. */
enum { IM2WIN_MODE_TF32 = 0,  /* tensor cores, operands read as TF32 (low 13 mantissa bits unused) */
       IM2WIN_MODE_BF16 = 1,  /* tensor cores, operands rounded to BF16 (nearest-even) on the fly  */
       IM2WIN_MODE_FP32 = 2   /* plain fp32 FMA on the CUDA cores: a slow exact-arithmetic check    */ };

typedef enum {
  IM2WIN_OK = 0,
  IM2WIN_EINVAL = -1,       /* null pointer, size < 1, Fh > H, Fw > W, unknown enum, size overflow */
  IM2WIN_EALIGN = -2,       /* a device base pointer is not 16-byte aligned                        */
  IM2WIN_EWORKSPACE = -3,   /* workspace missing or smaller than im2win_workspace_bytes            */
  IM2WIN_EOVERLAP = -4,     /* an output range overlaps an input or workspace range                */
  IM2WIN_ECUDA = -5,        /* a CUDA runtime call or kernel launch failed                         */
  IM2WIN_ETIMEOUT = -6,     /* a bounded device-side wait expired (see im2win_last_device_status)  */
  IM2WIN_EUNSUPPORTED = -7, /* shape outside what the kernels implement (see im2win_conv)          */
  IM2WIN_ESCRATCH = -8      /* problem needs more scratch than im2win_conv_static's built-in buffer */
} im2win_status;

/* Output sizes, Ho = floor((H-Fh)/s)+1 and Wo = floor((W-Fw)/s)+1
 * (Algorithm 1, first line; Table I fixes the division as floor). */
int im2win_out_dims(const im2win_shape* shape, int32_t* Ho, int32_t* Wo);

/* Bytes of the im2win tensor, 4*N*C*Ho*Fh*W (the element count Section III-A gives for it: batch x
 * channels x filter height x input width x output height).  This is the least workspace im2win_conv
 * needs when it is given the untransformed input, and the size of im2win_transform's output.  The same
 * tight size is used when Fh <= s, where Algorithm 1 allocates the (larger or equal) input size. */
int im2win_workspace_bytes(const im2win_shape* shape, size_t* bytes);

/* Workspace with which im2win_conv can pick its fastest kernel for (shape, src_kind, mode) (no
 * counterpart in the paper): the im2win tensor where src_kind is NCHW (as above, rounded up to 256
 * bytes), plus room for a re-laid-out copy of the filter that some tensor-core kernels stream by TMA
 * (tap-major orders for the strip-matrix and window-offset kernels; bf16 for BF16 mode).  That copy is at
 * most about 1.4 x the filter's own 4*K*C*Fh*Fw bytes, i.e. a few MB against an im2win tensor of tens to hundreds
 * of MB.  A smaller workspace is legal (down to im2win_workspace_bytes, or none for the other source
 * kinds): kernels that need no copy are used instead, some of them slower. */
int im2win_conv_workspace_bytes(const im2win_shape* shape, int src_kind, int mode, size_t* bytes);

/* Bytes an im2col matrix for the whole batch would take, 4*N*C*Fh*Fw*Ho*Wo (Section III-A).
 * Reporting only: the library never builds one. */
int im2win_im2col_bytes(const im2win_shape* shape, size_t* bytes);

/* Algorithm 1:  Ihat[i][r][m][k*Fh+u] = I[i][r][m*s+u][k]  for every k in [0, W).
 * in_nchw:    device, N*C*H*W floats, read only.
 * out_im2win: device, N*C*Ho*W*Fh floats, every element is written; bit-exact copy of the inputs.
 * Both bases 16-byte aligned (EALIGN); the ranges must not overlap (EOVERLAP). */
int im2win_transform(const float* in_nchw, const im2win_shape* shape, float* out_im2win,
                     void* cuda_stream);

/* Storage variant of Algorithm 1 (no counterpart in the paper, which stores fp32 only):
 *   Ihat16[i][r][m][k*Fh+u] = bf16(I[i][r][m*s+u][k]),  round to nearest even,
 * i.e. the same tensor at 2 bytes per element, for IM2WIN_MODE_BF16 convolutions, whose operands
 * are rounded to bf16 anyway: it halves what the transform writes and what the convolution reads.
 * in_nchw:         device, N*C*H*W floats, read only.
 * out_im2win_bf16: device, N*C*Ho*W*Fh 16-bit words (im2win_workspace_bytes_bf16), all written.
 * Both bases 16-byte aligned (EALIGN); the ranges must not overlap (EOVERLAP). */
int im2win_workspace_bytes_bf16(const im2win_shape* shape, size_t* bytes);  /* 2*N*C*Ho*Fh*W */
int im2win_transform_bf16(const float* in_nchw, const im2win_shape* shape, uint16_t* out_im2win_bf16,
                          void* cuda_stream);

/* Algorithm 2 (the im2win-based convolution; its result is Eq. 1):
 *   O[i][j][m][n] = sum_{r,u,v} Ihat[i][r][m][(n*s+v)*Fh+u] * F[j][r][u][v].
 * (Algorithm 2 prints the strip offset as n*s*Wf+v*Hf+u, which equals the above for Hf==Wf and
 * is the form consistent with Algorithm 1 otherwise.)
 * src:       device.  src_kind NCHW: the input I (N*C*H*W floats); the call first runs the
 *            transform into `workspace`, which then holds Ihat and may be reused by the caller.
 *            src_kind IM2WIN: an im2win tensor; `workspace` may be NULL, or give scratch (see below).
 *            src_kind NCHW_FUSED: the input I; the tensor-core kernel stages the input rows a tile
 *            needs and reads the windows from them, so nothing of size Ihat is written (workspace
 *            0 bytes).  Same result as the other two kinds.  Shapes without a fused specialisation
 *            (the specialised filter sizes are 3x3, 5x5, 7x7, 11x11 and, with channel counts that are
 *            multiples of 16, 1x1, 1x3, 3x1, 1x7, 7x1, 2x2, 4x4, 3x5, 5x3) fall back to transform + convolution if a
 *            sufficient `workspace` is given, else EUNSUPPORTED; IM2WIN_MODE_FP32 always takes that
 *            fallback.
 *            src_kind IM2WIN_BF16: a bf16 im2win tensor from im2win_transform_bf16; mode must be
 *            IM2WIN_MODE_BF16 (EINVAL otherwise); `workspace` optional scratch.  The MMA operands
 *            are the same bf16 values as from an fp32 im2win tensor.  Implemented where a
 *            tensor-core kernel with a 16-bit source applies (3x3 layers of the strip-matrix kernel
 *            and stride-1 3x3 / 5x5 layers of the window-offset kernel, both with scratch;
 *            filter-size specialisations whose images have roughly a thousand output positions or
 *            more); EUNSUPPORTED otherwise.
 * filter:    device, K*C*Fh*Fw floats, native K,C,Fh,Fw order (the caller repacks nothing; kernels
 *            that want another order or bf16 write their copy into the workspace's scratch part).
 * mode:      IM2WIN_MODE_*.
 * out_nchw:  device, N*K*Ho*Wo floats, every element is written.  In the tensor-core modes the
 *            order in which the fp32 partial sums over channel groups are added is not fixed
 *            (several threads issue the MMAs of a tile; small batches and long reductions onto
 *            few filters add partial sums of reduction slices into the zeroed output), so two
 *            calls on the same data agree within fp32 rounding, and bit for bit where every
 *            product and partial sum is exactly representable.
 * workspace: device, 16-byte aligned, caller-owned; at least im2win_workspace_bytes(shape) bytes when
 *            src_kind is NCHW (EWORKSPACE otherwise), optional for the other kinds.  Bytes beyond
 *            the im2win tensor (from the next 256-byte boundary) serve as scratch for the filter copy;
 *            im2win_conv_workspace_bytes gives the size with which the fastest kernels apply.  The
 *            whole range must not overlap src, filter or out (EOVERLAP); its contents after the
 *            call are the im2win tensor (NCHW) followed by unspecified scratch.
 * Limits of the tensor-core modes (EUNSUPPORTED beyond them): Fh*Fw <= 1024; one output row's
 * worth of staged strips must fit in shared memory (W*Fh up to a few thousand floats).
 * IM2WIN_MODE_FP32 has no such limits. */
int im2win_conv(const void* src, int src_kind, const float* filter_kcfhfw,
                const im2win_shape* shape, int mode, float* out_nchw,
                void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Output-layout variant of im2win_conv (no counterpart in the paper, whose outputs are NCHW): the
 * same fp32 result written channels-last, out_nhwc[i][m][n][j] = O(i, j, m, n) of Eq. 1, so that a
 * position's K filter outputs are contiguous (the accumulator row of a tensor-core tile as it is).
 * out_nhwc: device, N*Ho*Wo*K floats, every element is written; 16-byte aligned.
 * Everything else as im2win_conv: all source kinds, all three modes and every shape (each kernel
 * has the layout as an epilogue option; the reduction slices of under-filled launches, which add
 * into an NCHW output, are not used). */
int im2win_conv_nhwc(const void* src, int src_kind, const float* filter_kcfhfw,
                     const im2win_shape* shape, int mode, float* out_nhwc,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Output-storage variant of im2win_conv (no counterpart in the paper, whose outputs are fp32):
 * the same result rounded to bf16 (nearest even) from the fp32 accumulators, NCHW, 2 bytes per
 * element: half the output footprint and half the bytes written.
 * out_nchw_bf16: device, N*K*Ho*Wo 16-bit words, every element is written; 16-byte aligned.
 * Everything else as im2win_conv.  Tensor-core modes only (IM2WIN_MODE_FP32: EINVAL), and only
 * square filters with a specialisation: 3x3, 5x5, 7x7, 11x11 (EUNSUPPORTED otherwise: the generic
 * kernel and the pointwise / factorised families have no bf16 epilogue). */
int im2win_conv_bf16out(const void* src, int src_kind, const float* filter_kcfhfw,
                        const im2win_shape* shape, int mode, uint16_t* out_nchw_bf16,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* HOST-buffer convenience for callers without device memory of their own: copies the input and
 * the filter from host memory, runs transform + convolution on an internal stream and copies the
 * result back; returns after the result is in out_host.  Device buffers are owned by the library,
 * grown on demand and kept for the next call (released by im2win_host_release).  Not reentrant.
 * in_host: N*C*H*W floats; filter_host: K*C*Fh*Fw floats; out_host: N*K*Ho*Wo floats (pinned
 * memory makes the copies faster, pageable memory is accepted). */
int im2win_conv_host(const float* in_host, const float* filter_host, const im2win_shape* shape,
                     int mode, float* out_host);
int im2win_host_release(void);

/* No counterpart in the paper: an entry point for callers that cannot allocate device memory.
 * Who that is: a process whose GPU memory belongs whole to some other allocator (a serving
 * arena, a framework pool sized to the device), or code under a no-allocation-after-start-up rule
 * (hard-real-time loops, safety-reviewed code).  im2win_conv needs a caller-supplied workspace for
 * the im2win tensor; this variant keeps that tensor in a buffer built into the library image
 * (IM2WIN_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library, held until
 * the process exits) and itself calls no cudaMalloc, cudaFree or other allocating routine; a filter
 * copy that a tensor-core kernel wants goes into the same buffer behind the im2win tensor when there
 * is room, else a kernel that needs none is used.
 * Computes exactly what im2win_conv(in_nchw, IM2WIN_SRC_NCHW, ...) computes, on `cuda_stream`,
 * asynchronously.  in_nchw / filter_kcfhfw / out_nchw: device pointers as for im2win_conv.
 * Errors: IM2WIN_ESCRATCH when im2win_workspace_bytes(shape) exceeds the built-in buffer (nothing
 * is launched); otherwise as im2win_conv.
 * The first call on a device looks up the buffer's device address (a one-time set-up step, done
 * with that device current); make that first call outside any stream capture.
 * All calls on a device share the one buffer: two calls whose kernels can overlap on the GPU
 * (different streams without an ordering between them) race on it and give wrong results.  The
 * buffer keeps the previous call's contents; nothing in it needs clearing, because each call
 * overwrites every element it later reads.  The cached address is an atomic per device, so first calls
 * from several host threads are safe; the buffer itself is not. */
#define IM2WIN_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
int im2win_conv_static(const float* in_nchw, const float* filter_kcfhfw, const im2win_shape* shape,
                       int mode, float* out_nchw, void* cuda_stream);
/* Kernels never trap.  A bounded wait that expires, or an internal range check that fails,
 * records a code in a device-side status word and the kernel exits early (its output is then
 * undefined).  This call synchronises `cuda_stream`, stores the word in *status (0 = clean) and
 * clears it.  Returns IM2WIN_OK when the word was clean (or holds a range-check code, 201),
 * IM2WIN_ETIMEOUT when it names an expired wait (101..109; the code says which wait). */
int im2win_last_device_status(void* cuda_stream, int32_t* status);

/* English text for a status code; never NULL. */
const char* im2win_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif
