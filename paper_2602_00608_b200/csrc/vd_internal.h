// Internal declarations shared by the translation units of libvd.so (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "vd_ops.h"

namespace vd {

// One fused convolution launch: y = conv(pad0(up2x?(act(x*scale+shift)))) + bias (+ residual).
struct ConvArgs {
    const void* x;          // NHWC [B,Hs,Ws,Cin], in_dtype
    const void* w;          // packed weights (layout depends on the implementation)
    const float* bias;      // [Cout] or null
    const float* scale;     // [B,Cin] or null
    const float* shift;     // [B,Cin] or null
    const float* residual;  // fp32 NHWC [B,H,W,Cout] or null; the tensor-core kernel needs residual == y (accumulate in place)
    void* y;                // out_dtype, NHWC [B,H,W,Cout] or NCHW [B,Cout,H,W]
    int B, Hs, Ws;          // source resolution
    int H, W;               // output resolution (= source, or 2x source with upsample)
    int Cin, Cout, ksize;
    int upsample;           // 0 none; 1 nearest-2x folded into the addressing (9 taps on the 2x grid); 2 phase-collapsed
                            // (four 2x2 convolutions of the source with pre-summed weights; tensor-core kernel only)
    int silu;
    int in_dtype, out_dtype, out_nchw, bf16_operands;
    int out_u8;             // 1: y is the display-packed frame, NHWC uint8 [B,H,W,Cout] (out_dtype and out_nchw are ignored)
    // optional fused 1x1 shortcut (tensor-core kernel only): y += W2 * x2 + bias2
    const void* x2;         // fp32 NHWC [B,H,W,Cin2] at the output resolution, or null
    const void* w2;         // fp32 [Cout][Cin2] (tensor-core kernel: the shortcut's products are tf32)
    const float* bias2;     // [Cout] or null
    int Cin2;
    // optional (tensor-core kernel only): the GroupNorm that follows takes its statistics from this layer's
    // epilogue instead of a pass of its own.  Every epilogue warp adds (sum, sum of squares) of the output it
    // drained, in 64-bit fixed point, per group; the CTA that finishes last turns the sums into scale and shift.
    unsigned long long* stat_sum;   // [B][stat_G][2] sums, or null; zero before the launch, left zero
    unsigned int* stat_counter;  // CTAs done; zero before the launch, left zero
    const float* stat_gamma;     // [Cout]
    const float* stat_beta;      // [Cout]
    float* stat_scale;           // [B,Cout]
    float* stat_shift;           // [B,Cout]
    int stat_G;
    float stat_eps;
    // tensor-core kernel: ceil(2^32 / d) for the divisors of its tile numbering (tiles per image, channel
    // blocks, tiles per row), filled in by its launcher; 0 stands for d = 1
    unsigned int div_tiles, div_nblk, div_tx;
};
constexpr int kConvMaxCtas = 160;         // upper bound on the persistent grid
// bytes of the statistics sums of a convolution's epilogue, then its arrival counter
inline size_t conv_stat_sum_bytes(int B, int G) { return (((size_t)B * G * 2 * sizeof(unsigned long long)) + 255) / 256 * 256; }
inline size_t conv_stat_scratch_bytes(int B, int G) { return conv_stat_sum_bytes(B, G) + 256; }

struct GnArgs {
    const void* x;          // NHWC [B,H,W,C]
    int dtype;
    int B, P, C, G;         // P = H*W
    float eps;
    const float* gamma;     // [C]
    const float* beta;      // [C]
    float* scale;           // [B,C]
    float* shift;           // [B,C]
    float* partial;         // [B, kGnMaxChunks, G, 2] scratch
    unsigned int* counters; // [B] arrival counters, zero before the launch; the kernel leaves them zero
    const float* offset;    // [C] or null: the statistics are those of x + offset[c] (a bias the tensor's producer
                            // left out), and shift takes scale * offset in, so scale * x + shift normalises x + offset
};
constexpr int kGnMaxChunks = 296;      // two blocks per SM on a 148-SM device
// bytes of the partial records / of the whole scratch (records, then the arrival counters)
inline size_t gn_partial_bytes(int B, int G) { return (size_t)B * kGnMaxChunks * G * 2 * sizeof(float); }
inline size_t gn_scratch_bytes(int B, int G) { return gn_partial_bytes(B, G) + (((size_t)B * 4 + 255) / 256) * 256; }

struct AttnArgs {
    const void* q; const void* k; const void* v; void* o;
    int dtype;
    int B, T, C, ld_qkv, ld_o;
    float scale;
    void* vt;               // scratch for the tensor-core kernel: V transposed, [B][C][round_up(T,64)] bf16
};

struct IngestArgs {
    const void* z;          // NCHW latents (or z_prev when v_prev is set)
    const void* v_prev;     // null, or the motion vector for z = z_prev + lambda*v_prev
    void* z_out;            // optional NCHW copy of the extrapolated latents
    void* v_out;            // optional NCHW new motion vector z - z_prev
    float lambda;
    float* x;               // fp32 NHWC [B,h,w,C]
    int dtype, B, C, h, w;
};

// codes the kernels latch in the status word when a bounded wait runs out
constexpr unsigned int kStatusConvTimeout = 0xC0DE0001u, kStatusAttnTimeout = 0xC0DE0002u, kStatusWaitProbe = 0xC0DE0003u;
cudaError_t launch_wait_probe(unsigned int* status_word, long long limit_cycles, cudaStream_t s);   // wait_probe.cu

// records `msg` as the text vd_last_error(NULL) returns (defined in vd_api.cu)
void set_last_error(const char* msg);

// ---- FFMA kernels (kernels_simt.cu)
cudaError_t launch_ingest(const IngestArgs& a, cudaStream_t s);
cudaError_t launch_gn_stats(const GnArgs& a, cudaStream_t s);          // one launch (the last block per sample finalises)
cudaError_t launch_conv_simt(const ConvArgs& a, cudaStream_t s);
cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t s);
// OIHW (or [out,in]) weight of dtype `w_dtype` -> fp32 [tap][Cin][Cout]
// (Cout rows are written at column offset cout_offset of a packed matrix cout_total wide)
cudaError_t launch_pack_weight_simt(const void* w, int w_dtype, float* packed, int Cout, int Cin, int taps,
                                    int cout_total, int cout_offset, cudaStream_t s);
// any vector of dtype -> fp32
cudaError_t launch_to_f32(const void* src, int dtype, float* dst, int64_t n, cudaStream_t s);
// out[c] = in[c] + b[c] + b2[c] + sum_k w2[c][k] * pin[k], c < Cout (absent terms: null pointers)
cudaError_t launch_fold_bias(float* out, const float* in, const float* b, const float* b2, const float* w2, const float* pin,
                             int Cin2, int Cout, cudaStream_t s);
// dst[n][c] = src[c] (src null: 1.0), n < B
cudaError_t launch_fill_rows(float* dst, const float* src, int C, int B, cudaStream_t s);

// ---- tcgen05 kernels (conv_tc.cu, attn_tc.cu)
bool conv_tc_supported(const ConvArgs& a);
bool conv_tc_stats_supported(const ConvArgs& a, int groups);   // the epilogue can take the next GroupNorm's statistics
bool conv_tc_pairs_available();          // can the current device co-schedule the kernels' CTA pairs?
size_t conv_tc_packed_bytes(int Cout, int Cin, int taps, bool phase);
// OIHW weight (bf16) -> bf16 [tap][Cout_pad][Cin] (K-major rows for the B operand); phase: the sixteen
// pre-summed 2x2 taps of the phase-collapsed upsampling convolution, in the order its kernel streams them
cudaError_t launch_pack_weight_tc(const void* w, int w_dtype, void* packed, int Cout, int Cin, int taps,
                                  int cout_total, int cout_offset, bool phase, cudaStream_t s);
// Launch-invariant state of one tensor-core convolution: the TMA descriptor of its packed weights.
struct alignas(64) ConvTcPlan {
    unsigned char tmap[128];
    unsigned char tmap2[128];   // weights of the fused shortcut (copy of tmap when unused)
    unsigned char tmap_y[128];  // output tensor (NHWC outputs leave through bulk tensor stores)
    unsigned char tmap_x2[128]; // input of the fused shortcut (fp32 NHWC, loaded by TMA)
    const void* x2;             // the address tmap_x2 was built for
    void* y;                    // the output address tmap_y was built for
    int batch;                  // frames covered by tmap_y
    int bn;
    int cg;                     // CTAs per MMA: 2 = two-CTA pairs (weight maps built with half-height boxes)
    int phase;                  // 1: phase-collapsed upsampling form (tmap_y / tmap2 are the output maps of row parity 0 / 1)
    int valid;
};
cudaError_t conv_tc_prepare(const ConvArgs& a, ConvTcPlan* plan);      // a.w must be the final packed-weight address
cudaError_t launch_conv_tc(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status_word, cudaStream_t s);
bool attn_tc_supported(const AttnArgs& a);
size_t attn_tc_scratch_bytes(int B, int T, int C);
// Launch-invariant state of the tensor-core attention: the TMA descriptors of q, k and the transposed v.
struct alignas(64) AttnTcPlan {
    unsigned char tq[128], tk[128], tv[128];
    const void* q; const void* k; const void* vt;
    int batch, tokens, valid;
};
cudaError_t attn_tc_prepare(const AttnArgs& a, AttnTcPlan* plan);      // a.B = the largest batch the plan must serve
cudaError_t launch_attn_tc(const AttnArgs& a, const AttnTcPlan* plan, unsigned int* status_word, cudaStream_t s);


// ---- programmatic dependent launch
// Every kernel of the decode path is launched so that its blocks may become resident while the
// kernel before it in the stream is still draining: they set themselves up (barriers, tensor
// memory, weight prefetch), then griddep_wait() returns once the preceding kernel has completed
// and its writes are visible.  Rules that make the chain safe: (1) every such kernel executes
// griddep_wait() in at least one thread before it exits, so "kernel N completed" implies "all
// kernels before N completed"; (2) nothing a predecessor writes is read, and nothing it reads is
// written, before the wait.
// Dependent launches are used only inside a PdlScope (the decode loop): the single-operator entry
// points launch plainly, since their inputs may come from work this library knows nothing about.
bool pdl_enabled();     // inside a PdlScope
struct PdlScope {
    explicit PdlScope(bool on);
    ~PdlScope();
    bool prev;
};

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

#ifdef __CUDACC__
// Display packing of one frame value for transport: [-1, 1] -> 0..255, t = fma(x, 127.5, 127.5) in fp32 (one
// rounding), clamped, rounded to nearest with ties to even; NaN packs to 0.
__device__ __forceinline__ unsigned char pack_u8(float x) {
    float t = fmaf(x, 127.5f, 127.5f);
    t = t > 0.f ? t : 0.f;
    t = fminf(t, 255.f);
    return (unsigned char)__float2int_rn(t);
}
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

}  // namespace vd
