/*
 * vd_ops.h - test and measurement interface of libvd.so.
 *
 * Not part of the decoder's boundary (that is vd.h: create, decode, destroy and their helpers).
 * What is declared here exists for the per-kernel and per-layer parity tests and for the
 * benchmark: plan introspection, per-step device timing, a way to stop a decode after a given
 * step, and the fused operators of the chain of Section IV-B.1 (Eq. 9) as single calls on
 * caller-provided device tensors.  The same general rules as in vd.h apply.
 */
#ifndef VD_OPS_H_
#define VD_OPS_H_

#include "vd.h"

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------------------------------
 * Plan introspection and measurement (used by the benchmark and the per-layer parity tests).
 * ---------------------------------------------------------------------------------------- */
typedef enum {
    VD_STEP_INGEST = 0,     /* latents NCHW -> internal NHWC (+ optional extrapolation) */
    VD_STEP_GN_STATS = 1,   /* GroupNorm statistics -> per-(n,c) scale/shift */
    VD_STEP_CONV = 2,       /* 3x3 / 1x1 convolution with fused prologue/epilogue */
    VD_STEP_ATTENTION = 3   /* softmax(q k^T / sqrt(C)) v */
} vd_step_kind;

typedef struct {
    char name[64];              /* e.g. "up1.res0.conv1" */
    int32_t kind;               /* vd_step_kind */
    int32_t impl;               /* 0 = FFMA kernel, 1 = tcgen05 tensor-core kernel */
    int32_t launches;           /* kernel launches this step issues per decode */
    int32_t c_in, c_out, ksize, upsample;
    int32_t out_h, out_w;       /* resolution of the step's output */
    int32_t out_channels;       /* channels of the output tensor */
    int32_t out_dtype;          /* vd_dtype of the output tensor */
    int32_t out_nchw;           /* 1 if the output is NCHW (the frames), else NHWC */
    int64_t out_offset;         /* byte offset of the output in the workspace, -1 if it is `frames` */
    double flops_per_frame;     /* 2*taps*Cin*Cout*P for a conv, 4*T*T*C for attention, 0 otherwise */
    double bytes_per_frame;     /* algorithmic HBM bytes as stored (inputs once, output once, residual once) */
    double weight_bytes;        /* parameter bytes read once per launch (shared by the batch) */
    int32_t c_in2;              /* > 0: a 1x1 shortcut on a second input of c_in2 channels is fused in */
    int32_t has_residual;       /* 1: an fp32 residual tensor is added in the epilogue */
    int32_t phase_collapsed;    /* 1: an upsampling conv run as four 2x2 convolutions of the source (flops_per_frame
                                   still counts the layer's own 9 taps; the kernel executes 4/9 of them) */
    int32_t out_u8;             /* 1: the output is the display-packed uint8 NHWC frame (VD_FLAG_OUT_U8) */
    int32_t stats_fused;        /* 1: a convolution whose epilogue also produces the statistics (scale, shift) of the
                                   GroupNorm that follows; that GroupNorm has no step of its own then */
    int32_t reserved;
    int64_t out_pending_offset; /* >= 0: byte offset in the workspace of an fp32 vector [out_channels]; the step's stored
                                   output lacks this per-channel constant (a bias left out of the epilogue and accounted
                                   for by the steps that read the tensor): layer output = stored + pending[c].  -1: none */
} vd_step_info;

VD_API vd_status vd_num_steps(vd_handle h, int32_t* n);
VD_API vd_status vd_get_step(vd_handle h, int32_t index, vd_step_info* info);

/* Runs one decode with a CUDA event recorded around every step, waits for it, and writes the
 * device time of each step in milliseconds to ms[0..n_steps).  Creates and destroys events:
 * a measurement call, not for the serving path. */
VD_API vd_status vd_profile(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream,
                            float* ms, int32_t n_steps);

/* Test hooks of the device-timeout path (vd_get_status / VD_ERR_DEVICE_TIMEOUT):
 *   vd_debug_status_offset  byte offset of the status word (four uint32: code, block, detail, 0)
 *                           in the workspace, so a test can plant a code there from the host;
 *   vd_debug_wait_probe     launches a one-block kernel that runs the library's bounded mbarrier
 *                           wait into its limit on purpose: it waits `limit_cycles` SM clocks
 *                           (1e3..2e9) on a barrier nothing arrives on, gives up, records code
 *                           0xC0DE0003 in the status word and returns normally.  The kernel
 *                           neither traps nor spins without bound; the context stays usable. */
VD_API vd_status vd_debug_status_offset(vd_handle h, int64_t* offset);
VD_API vd_status vd_debug_wait_probe(vd_handle h, int64_t limit_cycles, void* cuda_stream);

/* Debug (handles created with VD_FLAG_CANARY): synchronises the device and verifies the guard pattern behind
 * every workspace region; VD_ERR_WORKSPACE (with the guard's index and offset in vd_last_error) if a kernel
 * wrote outside its buffer.  *n_guards (may be NULL) receives the number of guards (0 without the flag). */
VD_API vd_status vd_debug_check_canaries(vd_handle h, int32_t* n_guards);

/* Debug: makes vd_decode stop after step `index` (so that step's output can be read from the
 * workspace at out_offset); -1 restores the full decode. */
VD_API vd_status vd_debug_stop_after(vd_handle h, int32_t index);

/* ------------------------------------------------------------------------------------------
 * Operator-level entry points: the fused building blocks of the chain of Section IV-B.1,
 * callable on caller-provided device tensors (internal NHWC layout).  Used by per-kernel tests.
 * ---------------------------------------------------------------------------------------- */
typedef enum { VD_IMPL_AUTO = 0, VD_IMPL_SIMT = 1, VD_IMPL_TC = 2 } vd_impl;

typedef struct {
    uint32_t struct_size;
    int32_t batch;
    int32_t in_h, in_w;         /* resolution of the input tensor */
    int32_t c_in, c_out;
    int32_t ksize;              /* 1 or 3 (zero padding ksize/2, stride 1) */
    int32_t upsample;           /* 1: nearest-2x upsample folded into the addressing; output is 2*in_h x 2*in_w.
                                   2: the same result phase-collapsed (four 2x2 convolutions of the source with
                                   pre-summed weights; tensor-core kernel only, 3x3, c_out % 128 == 0, no residual) */
    int32_t silu;               /* 1: SiLU after the scale/shift prologue */
    int32_t in_dtype;           /* vd_dtype of x */
    int32_t out_dtype;          /* vd_dtype of y */
    int32_t out_nchw;           /* 1: y is NCHW, else NHWC */
    int32_t bf16_operands;      /* 1: round the (transformed) operand to bf16 before the product */
    int32_t impl;               /* vd_impl */
} vd_conv_desc;

/* Bytes of the packed form of a [c_out,c_in,k,k] weight for the implementation `impl` resolves to. */
VD_API vd_status vd_conv_packed_weight_bytes(const vd_conv_desc* d, size_t* bytes);
/* Repacks a device [c_out,c_in,k,k] weight of dtype `w_dtype` into `packed` (device). */
VD_API vd_status vd_conv_pack_weight(const vd_conv_desc* d, const void* w_oihw, int32_t w_dtype, void* packed,
                                     void* cuda_stream);
/* y = conv(pad0(up2x?(act(x*scale + shift)))) + bias (+ residual):
 *   x        device NHWC [batch,in_h,in_w,c_in], in_dtype
 *   scale, shift   device fp32 [batch,c_in] or both NULL (no prologue); act = SiLU if d->silu
 *   bias     device fp32 [c_out] or NULL;  residual  device fp32 NHWC like y, or NULL
 *   y        device, out_dtype, NHWC (or NCHW if out_nchw) at the output resolution */
VD_API vd_status vd_op_conv2d(const vd_conv_desc* d, const void* x, const void* w_packed, const float* bias,
                              const float* scale, const float* shift, const float* residual, void* y,
                              void* cuda_stream);

/* vd_op_conv2d and, from the same launch, the statistics of GroupNorm(y) folded with the affine parameters
 * (Section IV-B.1: the normalisation's reduction is taken while the tile is on chip):
 *   out_scale[n,c] = gamma[c]*rstd[n,g], out_shift[n,c] = beta[c] - mean[n,g]*out_scale[n,c]   (device fp32 [batch,c_out]),
 * mean and biased variance of the fp32 values before they are rounded to y's dtype.  Tensor-core kernel only:
 * c_out % 128 == 0, bf16 NHWC output, no residual, no upsampling of kind 2, groups <= 32 holding 4, 8 or 16 channels
 * each; anything else returns VD_ERR_UNSUPPORTED.  `scratch`: device memory of vd_conv_stats_scratch_bytes bytes
 * (the per-group sums, then an arrival counter; the call clears both itself).  Totals of a tile are turned into
 * 64-bit fixed point (2^-20 for sums, 2^-16 for sums of squares) and all further additions are integer
 * additions: results are bitwise reproducible and do not depend on the batch. */
VD_API size_t vd_conv_stats_scratch_bytes(int32_t batch, int32_t groups);
VD_API vd_status vd_op_conv2d_stats(const vd_conv_desc* d, const void* x, const void* w_packed, const float* bias,
                                    const float* scale, const float* shift, void* y, int32_t groups, float eps,
                                    const float* gamma, const float* beta, float* out_scale, float* out_shift,
                                    void* scratch, void* cuda_stream);

/* GroupNorm statistics of x (device NHWC [batch,h,w,c], dtype `dtype`) folded with the affine
 * parameters: scale[n,c] = gamma[c]*rstd[n,g], shift[n,c] = beta[c] - mean[n,g]*scale[n,c]
 * (biased variance, eps inside the root).  `offset` (device fp32 [c], or NULL): the statistics are those
 * of x[..,c] + offset[c] and shift takes scale*offset in, so that scale*x + shift is GroupNorm(x + offset):
 * the decoder leaves a convolution's bias out of its epilogue and lets the next normalisation account for it.  `scratch` is device memory of
 * vd_gn_scratch_bytes(batch, groups) bytes (chunk records, then one arrival counter per sample,
 * which the call clears itself).  scale/shift are device fp32 [batch,c].  c <= 1024, c/groups a
 * multiple of 4.  One kernel launch; results are bitwise reproducible and do not depend on batch. */
VD_API size_t vd_gn_scratch_bytes(int32_t batch, int32_t groups);
VD_API vd_status vd_op_gn_stats(const void* x, int32_t dtype, int32_t batch, int32_t h, int32_t w, int32_t c,
                                int32_t groups, float eps, const float* gamma, const float* beta, const float* offset,
                                float* scale, float* shift, void* scratch, void* cuda_stream);

/* The same operator for callers that cannot hand over (or allocate) a scratch buffer.  The paper
 * has no counterpart of this entry point; it exists for hosts where device allocation is not an
 * option at call time: frame loops that must not hit the allocator's implicit synchronisation,
 * plug-ins living inside another application's memory budget, code running in a host callback.
 * The chunk records and the arrival counters live in a 148 KiB array built into the library (held
 * by every GPU that loads it until the process exits).  Limits and rules:
 *   - batch * groups <= 64, else VD_ERR_UNSUPPORTED (use vd_op_gn_stats);
 *   - no cudaMalloc/cudaFree or any allocating routine is called;
 *   - the first call on a device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture;
 *   - all calls on a device share the array: calls whose kernels may overlap on the GPU race.
 *     The records need no clearing between calls (each call writes every record it later
 *     reads); the arrival counters are cleared by an asynchronous memset at the start of a call. */
VD_API vd_status vd_op_gn_stats_static(const void* x, int32_t dtype, int32_t batch, int32_t h, int32_t w,
                                       int32_t c, int32_t groups, float eps, const float* gamma,
                                       const float* beta, float* scale, float* shift, void* cuda_stream);

/* o[t,:] = sum_u softmax_u(scale * q[t,:].k[u,:]) v[u,:] for each batch item; q, k, v, o are
 * device rows of `dtype` with `ld` elements between consecutive tokens (so q, k, v may be
 * slices of one [tokens, 3C] tensor); tokens >= 1.  The tensor-core kernel needs bf16, 512
 * channels, 16-byte aligned pointers, ld multiples of 8, and `scratch`: device memory of
 * vd_attention_scratch_bytes bytes (it holds V transposed); the FFMA kernel ignores scratch. */
VD_API size_t vd_attention_scratch_bytes(int32_t batch, int32_t tokens, int32_t channels);
VD_API vd_status vd_op_attention(const void* q, const void* k, const void* v, void* o, int32_t dtype,
                                 int32_t batch, int32_t tokens, int32_t channels, int32_t ld_qkv, int32_t ld_o,
                                 float scale, int32_t impl, void* scratch, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* VD_OPS_H_ */
