/*
 * vd — frame decoder for a generative game engine: world-model latents in, RGB frames out.
 *
 * C ABI of libvd.so (CUDA, sm_100a only; there is no CPU or other-GPU fallback).
 *
 * The decoder is the convolutional VAE decoder that the paper's pipeline calls once per
 * displayed frame (Algorithm 1, "VAE decode" step; Algorithm 2, both branches) and whose
 * operator chain Upsample -> Conv2d -> GroupNorm -> SiLU it fuses to cut HBM round trips
 * (Section IV-B.1, Eq. 8 and Eq. 9).  Layer lists ("layouts") are those of the benchmark
 * configurations:
 *   VD_ARCH_SDVAE  conv_in 4->512; mid = ResNet(512), single-head attention(512), ResNet(512);
 *                  levels 512,512,256,128 with 3 ResNet blocks each (1x1 shortcut where the
 *                  width changes) and nearest-2x upsample + conv3x3 after the first three;
 *                  GroupNorm, SiLU, conv_out 128->3.  Output is 8x the latent size.
 *   VD_ARCH_TINY   conv_in 4->64; ResNet(64); 3 x [nearest-2x upsample, conv3x3, ResNet] with
 *                  widths 64->64->32->32; GroupNorm, SiLU, conv_out 32->3.
 *
 * General rules
 *   - Every pointer named "device" is CUDA device memory on the current device, owned and
 *     allocated by the caller; the library never allocates device memory.
 *   - Every entry point returns a vd_status; nothing throws or aborts across the ABI.
 *     Arguments are validated on the host before anything is launched.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef VD_H_
#define VD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define VD_API __attribute__((visibility("default")))
#else
#define VD_API
#endif

typedef struct vd_handle_s* vd_handle;

typedef enum {
    VD_OK = 0,
    VD_ERR_INVALID_ARG = -1,    /* NULL/misaligned pointer, bad size, unknown enum, missing weight */
    VD_ERR_UNSUPPORTED = -2,    /* valid request this build cannot run (e.g. device is not sm_100) */
    VD_ERR_WORKSPACE = -3,      /* workspace smaller than vd_query_workspace reports */
    VD_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed; see vd_last_error */
    VD_ERR_DEVICE_TIMEOUT = -5  /* a bounded wait inside a kernel expired (latched status word) */
} vd_status;

typedef enum { VD_F32 = 0, VD_BF16 = 1 } vd_dtype;
typedef enum { VD_ARCH_TINY = 0, VD_ARCH_SDVAE = 1 } vd_arch;

/* vd_config.flags */
#define VD_FLAG_FORCE_SIMT 0x1u   /* run every layer on the plain FFMA kernels (cross-check path) */

typedef struct {
    uint32_t struct_size;       /* sizeof(vd_config), for versioning */
    int32_t arch;               /* vd_arch */
    int32_t dtype;              /* vd_dtype of latents, frames and weights.  VD_BF16: bf16 operands and
                                   intra-block tensors, fp32 accumulation, fp32 residual stream.
                                   VD_F32: fp32 throughout (FFMA kernels). */
    int32_t latent_channels;    /* 4 */
    int32_t out_channels;       /* 3 */
    int32_t latent_h, latent_w; /* frames are 8*latent_h x 8*latent_w */
    int32_t max_batch;          /* largest `batch` vd_decode will be given */
    int32_t norm_groups;        /* 32 (SDVAE) / 8 (TINY) in the benchmark configurations */
    float norm_eps;             /* 1e-6 */
    uint32_t flags;
} vd_config;

/* One parameter tensor in the caller's (PyTorch-canonical) layout: convolution weights
 * [Cout,Cin,kh,kw], attention projections [out,in], GroupNorm scale/shift and biases [C].
 * Names: conv_in, mid.res{0,1}, mid.attn.{norm,q,k,v,o}, up{i}.res{j}.{norm1,conv1,norm2,
 * conv2,shortcut}, up{i}.upconv, norm_out, conv_out, each with ".weight" and ".bias". */
typedef struct {
    const char* name;
    const void* dptr;           /* device, contiguous */
    int32_t dtype;              /* must equal vd_config.dtype */
    int32_t ndim;
    int64_t shape[4];
} vd_tensor;

/* Bytes of workspace a handle for `cfg` needs (repacked weights, activations for max_batch
 * frames, GroupNorm statistics).  Host-only; touches no device. */
VD_API vd_status vd_query_workspace(const vd_config* cfg, size_t* bytes);

/* Builds a decoder: validates `cfg` and the weight list (every tensor of the layout must be
 * present with the right shape and dtype), repacks the weights into `workspace` and builds the
 * launch plan.  `workspace` is device memory, 256-byte aligned, at least vd_query_workspace
 * bytes, and must outlive the handle.  The call synchronises `cuda_stream` before returning, so
 * the weight tensors may be freed afterwards.  On failure *out is NULL. */
VD_API vd_status vd_create(const vd_config* cfg, const vd_tensor* weights, int32_t n_weights,
                           void* workspace, size_t workspace_bytes, void* cuda_stream, vd_handle* out);

/* Decodes `batch` latents into frames (Algorithm 1, VAE decode step: I_t = Decode(z_t)).
 *   latents  device, [batch, latent_channels, latent_h, latent_w], NCHW, cfg.dtype
 *   frames   device, [batch, out_channels, 8*latent_h, 8*latent_w], NCHW, cfg.dtype; raw conv_out
 *            values (no clamp)
 * Asynchronous on `cuda_stream`: enqueues kernels only, no allocation, no host synchronisation.
 * 1 <= batch <= cfg.max_batch.  Calls on one handle must not overlap (one workspace). */
VD_API vd_status vd_decode(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream);

/* Latent extrapolation fused in front of the decoder (Algorithm 2, hit branch; Eq. 10):
 * z = z_prev + lambda * v_prev is formed on the fly and decoded; if z_out / v_out are non-NULL
 * they receive z and the new motion vector z - z_prev (device, same shape/dtype as latents). */
VD_API vd_status vd_decode_extrapolated(vd_handle h, const void* z_prev, const void* v_prev, float lambda,
                                        void* z_out, void* v_out, void* frames, int32_t batch,
                                        void* cuda_stream);

/* Same as vd_decode with HOST buffers (pinned memory recommended): copies the latents to the
 * device, decodes, copies the frames back and waits for the stream.  Staging areas for
 * max_batch frames are part of the workspace. */
VD_API vd_status vd_decode_host(vd_handle h, const void* latents_host, void* frames_host, int32_t batch,
                                void* cuda_stream);

/* Reads the device status word (call after the stream has been synchronised): VD_OK, or
 * VD_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded wait.  Synchronises the device copy. */
VD_API vd_status vd_get_status(vd_handle h);

/* Last error text of this handle (or of the last failed vd_create/vd_query_workspace when h is
 * NULL).  The string is owned by the library and valid until the next call on the handle. */
VD_API const char* vd_last_error(vd_handle h);

VD_API vd_status vd_destroy(vd_handle h);

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
    int32_t reserved[2];
} vd_step_info;

VD_API vd_status vd_num_steps(vd_handle h, int32_t* n);
VD_API vd_status vd_get_step(vd_handle h, int32_t index, vd_step_info* info);

/* Runs one decode with a CUDA event recorded around every step, waits for it, and writes the
 * device time of each step in milliseconds to ms[0..n_steps).  Creates and destroys events:
 * a measurement call, not for the serving path. */
VD_API vd_status vd_profile(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream,
                            float* ms, int32_t n_steps);

/* Debug: when `device_buffer` is non-NULL (160*4*2048*8 bytes, zeroed by the caller), every
 * tensor-core convolution launched afterwards records per-CTA role timelines into it (records
 * are code << 48 | SM clock; roles: 0 operand producer, 1 MMA issue, 2 epilogue); NULL turns
 * tracing off.  For kernel timing studies only. */
VD_API vd_status vd_debug_conv_trace(void* device_buffer, size_t bytes);

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
    int32_t upsample;           /* 1: nearest-2x upsample folded in; output is 2*in_h x 2*in_w */
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

/* GroupNorm statistics of x (device NHWC [batch,h,w,c], dtype `dtype`) folded with the affine
 * parameters: scale[n,c] = gamma[c]*rstd[n,g], shift[n,c] = beta[c] - mean[n,g]*scale[n,c]
 * (biased variance, eps inside the root).  `scratch` is device memory of
 * vd_gn_scratch_bytes(batch, groups) bytes (chunk records, then one arrival counter per sample,
 * which the call clears itself).  scale/shift are device fp32 [batch,c].  c <= 1024, c/groups a
 * multiple of 4.  One kernel launch; results are bitwise reproducible and do not depend on batch. */
VD_API size_t vd_gn_scratch_bytes(int32_t batch, int32_t groups);
VD_API vd_status vd_op_gn_stats(const void* x, int32_t dtype, int32_t batch, int32_t h, int32_t w, int32_t c,
                                int32_t groups, float eps, const float* gamma, const float* beta,
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
#endif /* VD_H_ */
