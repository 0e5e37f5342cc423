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
#define VD_FLAG_OUT_U8 0x4u       /* frames leave display-packed for transport (output side of Algorithm 1's decode
                                     step, Q_out.push(I_t); the frame copy is Table II's "Data Transport" row): NHWC
                                     uint8 [batch, 8*latent_h, 8*latent_w, out_channels], q = round(clamp(x*0.5+0.5,
                                     0, 1)*255), computed in fp32 as rint(clamp(fma(x, 127.5, 127.5), 0, 255)) with ties
                                     to even, in the last convolution's epilogue (a quarter / half of the bytes to copy) */
#define VD_FLAG_CANARY 0x8u       /* debugging: every workspace region is followed by a 256-byte guard pattern that
                                     vd_debug_check_canaries (vd_ops.h) verifies; costs a little workspace, no time */
#define VD_FLAG_UPSAMPLE_9TAP 0x2u /* upsampling convolutions as 9 taps on the 2x grid (upsampling folded into the
                                     addressing) instead of the default phase-collapsed form: per output parity a
                                     2x2 convolution of the source with pre-summed weights, 4/9 of the products,
                                     weights summed in fp32 and rounded once to bf16 */

#define VD_FLAG_FUSED_STATS 0x10u  /* where the tensor-core convolution that produces a normalised tensor can, its
                                     epilogue adds the per-group sums while the tile is in registers and the last CTA
                                     to finish writes scale and shift: no second read of the tensor (Section IV-B.1).
                                     Default off: every GroupNorm takes its statistics in a pass of its own, which is
                                     faster on B200 (the epilogue warps are the pace-setters of the narrow layers and
                                     the sums double their instruction count; measured 3.77 against 3.70 ms per
                                     720x480 frame). */

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
 * frames, GroupNorm statistics).  Host-only; touches no device.  The paper's decoder is one
 * worker of the VAE stage (Algorithm 1, "Initialize ... VAE Workers"); sizing its memory ahead of
 * time is what lets the decode step itself run without allocation. */
VD_API vd_status vd_query_workspace(const vd_config* cfg, size_t* bytes);

/* Builds one VAE worker of Algorithm 1 (the object whose decode step maps a latent z_t to the
 * frame I_t): validates `cfg` and the weight list (every tensor of the layout must be
 * present with the right shape and dtype), repacks the weights into `workspace` and builds the
 * launch plan.  `workspace` is device memory, 256-byte aligned, at least vd_query_workspace
 * bytes, and must outlive the handle.  The call synchronises `cuda_stream` before returning, so
 * the weight tensors may be freed afterwards.  On failure *out is NULL. */
VD_API vd_status vd_create(const vd_config* cfg, const vd_tensor* weights, int32_t n_weights,
                           void* workspace, size_t workspace_bytes, void* cuda_stream, vd_handle* out);

/* Decodes `batch` latents into frames (Algorithm 1, VAE decode step: I_t = Decode(z_t)).
 *   latents  device, [batch, latent_channels, latent_h, latent_w], NCHW, cfg.dtype
 *   frames   device, [batch, out_channels, 8*latent_h, 8*latent_w], NCHW, cfg.dtype; raw conv_out
 *            values (no clamp).  With VD_FLAG_OUT_U8: [batch, 8*latent_h, 8*latent_w, out_channels]
 *            uint8 (see the flag)
 * Asynchronous on `cuda_stream`: enqueues kernels only, no allocation, no host synchronisation.
 * 1 <= batch <= cfg.max_batch.  Calls on one handle must not overlap (one workspace). */
VD_API vd_status vd_decode(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream);

/* Latent extrapolation fused in front of the decoder (Algorithm 2, hit branch; Eq. 10):
 * z = z_prev + lambda * v_prev is formed on the fly and decoded; if z_out / v_out are non-NULL
 * they receive z and the new motion vector z - z_prev (device, same shape/dtype as latents). */
VD_API vd_status vd_decode_extrapolated(vd_handle h, const void* z_prev, const void* v_prev, float lambda,
                                        void* z_out, void* v_out, void* frames, int32_t batch,
                                        void* cuda_stream);

/* Same as vd_decode with HOST buffers: the "Data Transport" row of Table II (pinned instead of
 * pageable host memory for the latent and frame copies) around the decode step.  Copies the
 * latents to the device, decodes, copies the frames back and waits for the stream.  Pinned
 * buffers are recommended (pageable ones work, slower).  Staging areas for max_batch frames are
 * part of the workspace. */
VD_API vd_status vd_decode_host(vd_handle h, const void* latents_host, void* frames_host, int32_t batch,
                                void* cuda_stream);

/* A stream of frames through host memory with the copies hidden behind the decodes (Algorithm 1's loop:
 * latents arrive, are decoded, frames are pushed to the output queue; Table II's "Data Transport" row, pinned
 * memory).  latents_host holds n_frames latents, frames_host receives n_frames frames (layouts as in
 * vd_decode, contiguous over frames).  Frames are decoded `batch` at a time (the last step may be smaller);
 * while step t is decoded on `cuda_stream`, the latents of step t+1 travel to the device and the frames
 * of step t-1 travel back, on two copy streams of the handle (created on the first call), through two
 * staging buffers each in the workspace.  No host synchronisation per frame: the call returns once the
 * last frame has reached the host.  Use pinned host memory: with pageable memory the copies do not overlap. */
VD_API vd_status vd_decode_host_stream(vd_handle h, const void* latents_host, void* frames_host,
                                       int32_t n_frames, int32_t batch, void* cuda_stream);

/* Reads the device status word (call after the stream has been synchronised): VD_OK, or
 * VD_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded wait (every spin-wait inside the
 * tensor-core kernels has a cycle limit; a kernel that runs into it unwinds, frees its tensor
 * memory, returns, and records a code, its block and a detail word, which vd_last_error then
 * reports).  The word is sticky: it keeps the first failure until vd_clear_status.  The frames of
 * a decode that reported a timeout are undefined.  Synchronises the device copy. */
VD_API vd_status vd_get_status(vd_handle h);

/* Resets the status word to "no failure" (asynchronous on `cuda_stream`). */
VD_API vd_status vd_clear_status(vd_handle h, void* cuda_stream);

/* Last error text of this handle (or of the last failed vd_create/vd_query_workspace when h is
 * NULL).  The string is owned by the library and valid until the next call on the handle. */
VD_API const char* vd_last_error(vd_handle h);

/* Releases the handle (host memory only: the workspace belongs to the caller).  The caller makes
 * sure no decode of this handle is still running. */
VD_API vd_status vd_destroy(vd_handle h);

#ifdef __cplusplus
}
#endif
#endif /* VD_H_ */
