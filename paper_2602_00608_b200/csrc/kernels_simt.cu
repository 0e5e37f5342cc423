// Plain FFMA kernels: latent ingest, GroupNorm statistics, a tiled direct convolution with the
// fused prologue/epilogue, a streaming-softmax attention, and weight repacking.  These run the
// fp32 configuration end to end and serve as the on-GPU cross-check path of the bf16 one.
#include <math.h>

#include <mutex>
#include <string>

#include "vd_internal.h"

namespace vd {

namespace {

template <typename T> __device__ __forceinline__ float ld_f(const T* p, size_t i);
template <> __device__ __forceinline__ float ld_f<float>(const float* p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) {
    return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void st_f(T* p, size_t i, float v);
template <> __device__ __forceinline__ void st_f<float>(float* p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void st_f<__nv_bfloat16>(__nv_bfloat16* p, size_t i, float v) {
    p[i] = __float2bfloat16_rn(v);
}
__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }

// ------------------------------------------------------------------------------------ ingest
// Latents NCHW -> fp32 NHWC; optionally forms z = z_prev + lambda*v_prev first (Algorithm 2,
// hit branch) and writes z and the new motion vector back in the latents' own layout/dtype.
template <typename T>
__global__ void ingest_kernel(IngestArgs a) {
    griddep_launch();
    griddep_wait();
    const int64_t total = (int64_t)a.B * a.C * a.h * a.w;
    const T* z = (const T*)a.z;
    const T* vp = (const T*)a.v_prev;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        // i indexes the NCHW source
        const int x = (int)(i % a.w);
        const int y = (int)((i / a.w) % a.h);
        const int c = (int)((i / ((int64_t)a.w * a.h)) % a.C);
        const int n = (int)(i / ((int64_t)a.w * a.h * a.C));
        float v = ld_f<T>(z, i);
        if (vp) {
            const float zp = v;
            v = fmaf(a.lambda, ld_f<T>(vp, i), zp);
            if (a.z_out) {               // what is decoded is the latent as stored in its own dtype
                st_f<T>((T*)a.z_out, i, v);
                v = ld_f<T>((const T*)a.z_out, i);
            }
            if (a.v_out) st_f<T>((T*)a.v_out, i, v - zp);
        }
        a.x[(((int64_t)n * a.h + y) * a.w + x) * a.C + c] = v;
    }
}

// ------------------------------------------------------------------------------ GroupNorm stats
// One launch.  Every block reduces a run of pixels of one sample to per-group sums of (x - K) and
// (x - K)^2, where K is a reference value per (sample, group) that every block reads from the same
// place (the mean of the group's first four channels at the sample's centre pixel), so the sums
// of different blocks add without correction terms and a large common offset does not cancel.
// A thread owns one 4-channel slot (inside one group, since C/G is a multiple of 4) and walks down
// the pixels.  The block that arrives last for its sample adds the records of all blocks in a
// fixed order and writes scale and shift; the order of every sum is fixed by the sizes alone, so
// the result is bitwise reproducible and independent of the batch a sample is decoded in.
template <typename T> __device__ __forceinline__ void load4(const T* p, float v[4]);
template <> __device__ __forceinline__ void load4<float>(const float* p, float v[4]) {
    const float4 t = __ldg((const float4*)p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float v[4]) {
    const uint2 t = __ldg((const uint2*)p);
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

// Streaming loads of the statistics pass: a line it brings in is the first to leave L2 again, so the lines the
// producing kernel has just written stay resident until the pass reaches them.
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
template <typename T> __device__ __forceinline__ void load4_stream(const T* p, float v[4], uint64_t pol);
template <> __device__ __forceinline__ void load4_stream<float>(const float* p, float v[4], uint64_t pol) {
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "l"(p), "l"(pol));
}
template <> __device__ __forceinline__ void load4_stream<__nv_bfloat16>(const __nv_bfloat16* p, float v[4], uint64_t pol) {
    uint2 t;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v2.u32 {%0, %1}, [%2], %3;" : "=r"(t.x), "=r"(t.y) : "l"(p), "l"(pol));
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

constexpr int kGnThreads = 512;
constexpr int kGnFinalLoads = (kGnMaxChunks + 15) / 16;   // records a thread of the last block reads in one round (32 groups: 16 slices)

template <typename T, int U>
__global__ void __launch_bounds__(kGnThreads, 2) gn_stats_kernel(GnArgs a, int chunks, int pix_per_chunk) {
    __shared__ float2 sm[kGnThreads];
    __shared__ int s_last;
    griddep_launch();
    const int slots = a.C / 4;                       // 4-channel slots per pixel (<= kGnThreads)
    const int cpg = a.C / a.G;
    const int slot = threadIdx.x % slots;
    // The per-channel offset does not depend on the kernel before this one: it is read while that kernel finishes.
    // off_k: what the offset adds to the group's reference value; off_c: this thread's four channels;
    // off_fin: the same reference term for the group this thread finalises (threads below G, last block only).
    float off_k = 0.f, off_fin = 0.f;
    float4 off_c = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.offset) {
        const float4 og = __ldg((const float4*)(a.offset + (slot * 4 / cpg) * cpg));
        off_k = 0.25f * ((og.x + og.y) + (og.z + og.w));
        off_c = __ldg((const float4*)(a.offset + slot * 4));
        if (threadIdx.x < a.G) {
            const float4 of = __ldg((const float4*)(a.offset + threadIdx.x * cpg));
            off_fin = 0.25f * ((of.x + of.y) + (of.z + of.w));
        }
    }
    griddep_wait();
    const int n = blockIdx.y;
    const int chunk = blockIdx.x;
    const int p0 = chunk * pix_per_chunk;
    const int p1 = min(a.P, p0 + pix_per_chunk);
    const T* x = (const T*)a.x + (size_t)n * a.P * a.C;
    const int rows = kGnThreads / slots;             // pixels handled side by side
    const int row = threadIdx.x / slots;

    float s = 0.f, ss = 0.f;
    if (row < rows && p0 + row < p1) {
        float kv[4];
        load4<T>(x + (size_t)(a.P / 2) * a.C + (slot * 4 / cpg) * cpg, kv);
        // a per-channel offset is taken into the reference value: d = (x + off) - k = x - (k - off)
        const float k = 0.25f * ((kv[0] + kv[1]) + (kv[2] + kv[3])) + off_k;
        const float ko[4] = {k - off_c.x, k - off_c.y, k - off_c.z, k - off_c.w};
        int p = p0 + row;
        const uint64_t pol = policy_evict_first();
        for (; p + (U - 1) * rows < p1; p += U * rows) {        // U independent loads in flight
            float u[U][4];
#pragma unroll
            for (int j = 0; j < U; ++j) load4_stream<T>(x + (size_t)(p + j * rows) * a.C + slot * 4, u[j], pol);
#pragma unroll
            for (int j = 0; j < U; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float d = u[j][e] - ko[e];
                    s += d;
                    ss = fmaf(d, d, ss);
                }
        }
        for (; p < p1; p += rows) {
            float v[4];
            load4<T>(x + (size_t)p * a.C + slot * 4, v);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float d = v[e] - ko[e];
                s += d;
                ss = fmaf(d, d, ss);
            }
        }
    }
    sm[threadIdx.x] = make_float2(s, ss);
    __syncthreads();
    // one thread per group adds its members: rows x (slots of the group), in a fixed order
    if (threadIdx.x < a.G) {
        const int g = threadIdx.x;
        const int spg = cpg / 4;
        float2 acc = make_float2(0.f, 0.f);
        for (int r = 0; r < rows; ++r)
            for (int sl = g * spg; sl < (g + 1) * spg; ++sl) {
                const float2 v = sm[r * slots + sl];
                acc.x += v.x;
                acc.y += v.y;
            }
        ((float2*)a.partial)[((size_t)n * kGnMaxChunks + chunk) * a.G + g] = acc;
    }
    __syncthreads();

    // The block of this sample that finishes last folds the records into scale and shift.
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(a.counters + n, 1u);
        s_last = (prev == (unsigned int)chunks - 1u) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // Thread t adds the records k = t / G, t / G + slices, ... of group t % G (a warp reads whole records:
    // coalesced), the slices are added in a fixed order through shared memory, and every thread then writes
    // scale and shift of the channels c = t, t + 512, ...
    const int slices = kGnThreads / a.G;             // >= 1 (checked by the launcher)
    const int g = threadIdx.x % a.G, sl = threadIdx.x / a.G;
    float2 acc = make_float2(0.f, 0.f);
    if (sl < slices) {
        const float2* rec = (const float2*)a.partial + (size_t)n * kGnMaxChunks * a.G + g;
        for (int k0 = sl; k0 < chunks; k0 += kGnFinalLoads * slices) {
            float2 r[kGnFinalLoads];
            // unconditional loads (a record that does not exist re-reads the first and counts as zero), issued
            // back to back before the first use
#pragma unroll
            for (int i = 0; i < kGnFinalLoads; ++i) {
                const int k = k0 + i * slices;
                const float2* q = rec + (size_t)(k < chunks ? k : sl) * a.G;
                asm volatile("ld.global.cg.v2.f32 {%0, %1}, [%2];" : "=f"(r[i].x), "=f"(r[i].y) : "l"(q));
            }
#pragma unroll
            for (int i = 0; i < kGnFinalLoads; ++i) {
                const bool on = k0 + i * slices < chunks;
                acc.x += on ? r[i].x : 0.f;
                acc.y += on ? r[i].y : 0.f;
            }
        }
    }
    __syncthreads();                                 // the block's own use of sm[] above is over
    sm[threadIdx.x] = acc;
    __syncthreads();
    __shared__ float s_mean[kGnThreads], s_rstd[kGnThreads];
    if (threadIdx.x < a.G) {
        float2 t = make_float2(0.f, 0.f);
        for (int q = 0; q < slices; ++q) {
            const float2 v = sm[q * a.G + threadIdx.x];
            t.x += v.x;
            t.y += v.y;
        }
        float kv[4];
        load4<T>(x + (size_t)(a.P / 2) * a.C + threadIdx.x * cpg, kv);
        const float k = 0.25f * ((kv[0] + kv[1]) + (kv[2] + kv[3])) + off_fin;
        const float inv_n = 1.f / ((float)a.P * (float)cpg);
        const float md = t.x * inv_n;
        const float var = fmaxf(fmaf(-md, md, t.y * inv_n), 0.f);
        s_mean[threadIdx.x] = k + md;
        s_rstd[threadIdx.x] = 1.f / sqrtf(var + a.eps);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < a.C; c += kGnThreads) {
        const int gc = c / cpg;
        const float sc = __ldg(a.gamma + c) * s_rstd[gc];
        a.scale[(size_t)n * a.C + c] = sc;
        a.shift[(size_t)n * a.C + c] = __ldg(a.beta + c) - (s_mean[gc] - (a.offset ? __ldg(a.offset + c) : 0.f)) * sc;
    }
    if (threadIdx.x == 0) a.counters[n] = 0u;        // ready for the next launch
}

// ------------------------------------------------------------------------------- direct conv
// Block = TH x TW output pixels x CT output channels; input channels are consumed KC at a time
// through shared memory (the transformed input tile with its halo, and the weight slice).
constexpr int KC = 8;

template <typename TIn, typename TOut, int TH, int TW, int PPT, int CPT, int CGROUPS>
__global__ void __launch_bounds__((TH * TW / PPT) * CGROUPS) conv_simt_kernel(ConvArgs a) {
    griddep_launch();
    griddep_wait();
    constexpr int NPG = TH * TW / PPT;
    constexpr int CT = CPT * CGROUPS;
    constexpr int NT = NPG * CGROUPS;
    constexpr int PW = TW + 2, PH = TH + 2, NPIX = PW * PH;
    __shared__ float s_in[KC][NPIX + 1];
    __shared__ float s_w[9][KC][CT];

    const int tiles_x = (a.W + TW - 1) / TW;
    const int tx0 = (blockIdx.x % tiles_x) * TW;
    const int ty0 = (blockIdx.x / tiles_x) * TH;
    const int ct0 = blockIdx.y * CT;
    const int b = blockIdx.z;
    const int tid = threadIdx.x;
    const int pg = tid % NPG, cg = tid / NPG;
    const int ly = (pg * PPT) / TW, lx = (pg * PPT) % TW;
    const int taps = a.ksize * a.ksize;
    const int up = a.upsample ? 1 : 0;

    float acc[PPT][CPT];
#pragma unroll
    for (int p = 0; p < PPT; ++p)
#pragma unroll
        for (int q = 0; q < CPT; ++q) acc[p][q] = 0.f;

    const TIn* x = (const TIn*)a.x + (size_t)b * a.Hs * a.Ws * a.Cin;
    const float* wp = (const float*)a.w;

    for (int c0 = 0; c0 < a.Cin; c0 += KC) {
        for (int idx = tid; idx < NPIX * KC; idx += NT) {
            const int c = idx % KC, pix = idx / KC;
            const int oy = ty0 + pix / PW - 1, ox = tx0 + pix % PW - 1;
            float v = 0.f;
            if (oy >= 0 && oy < a.H && ox >= 0 && ox < a.W && c0 + c < a.Cin) {
                v = ld_f<TIn>(x, ((size_t)(oy >> up) * a.Ws + (ox >> up)) * a.Cin + c0 + c);
                if (a.scale) v = fmaf(v, a.scale[(size_t)b * a.Cin + c0 + c], a.shift[(size_t)b * a.Cin + c0 + c]);
                if (a.silu) v = silu_f(v);
                if (a.bf16_operands) v = round_bf16(v);
            }
            s_in[c][pix] = v;
        }
        for (int idx = tid; idx < taps * KC * CT; idx += NT) {
            const int ct = idx % CT, c = (idx / CT) % KC, tap = idx / (CT * KC);
            float v = 0.f;
            if (c0 + c < a.Cin && ct0 + ct < a.Cout) v = wp[((size_t)tap * a.Cin + c0 + c) * a.Cout + ct0 + ct];
            s_w[tap][c][ct] = v;
        }
        __syncthreads();
        for (int tap = 0; tap < taps; ++tap) {
            const int dy = a.ksize == 3 ? tap / 3 : 1, dx = a.ksize == 3 ? tap % 3 : 1;
            const int base = (ly + dy) * PW + lx + dx;
#pragma unroll
            for (int c = 0; c < KC; ++c) {
                float iv[PPT], wv[CPT];
#pragma unroll
                for (int p = 0; p < PPT; ++p) iv[p] = s_in[c][base + p];
#pragma unroll
                for (int q = 0; q < CPT; ++q) wv[q] = s_w[tap][c][cg * CPT + q];
#pragma unroll
                for (int p = 0; p < PPT; ++p)
#pragma unroll
                    for (int q = 0; q < CPT; ++q) acc[p][q] = fmaf(iv[p], wv[q], acc[p][q]);
            }
        }
        __syncthreads();
    }

    TOut* y = (TOut*)a.y;
#pragma unroll
    for (int p = 0; p < PPT; ++p) {
        const int oy = ty0 + ly, ox = tx0 + lx + p;
        if (oy >= a.H || ox >= a.W) continue;
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
            const int co = ct0 + cg * CPT + q;
            if (co >= a.Cout) continue;
            float v = acc[p][q];
            if (a.bias) v += a.bias[co];
            const size_t nhwc = (((size_t)b * a.H + oy) * a.W + ox) * a.Cout + co;
            if (a.residual) v += a.residual[nhwc];
            const size_t o = a.out_nchw ? (((size_t)b * a.Cout + co) * a.H + oy) * a.W + ox : nhwc;
            if (a.out_u8) ((unsigned char*)a.y)[nhwc] = pack_u8(v);
            else st_f<TOut>(y, o, v);
        }
    }
}

template <typename TIn, typename TOut>
cudaError_t conv_simt_dispatch(const ConvArgs& a, cudaStream_t s) {
    if (a.Cout <= 8) {
        constexpr int TH = 16, TW = 16, CT = 4;
        dim3 grid(((a.W + TW - 1) / TW) * ((a.H + TH - 1) / TH), (a.Cout + CT - 1) / CT, a.B);
        launch_pdl(conv_simt_kernel<TIn, TOut, TH, TW, 1, 4, 1>, grid, dim3(256), 0, s, a);
    } else {
        constexpr int TH = 8, TW = 8, CT = 64;
        dim3 grid(((a.W + TW - 1) / TW) * ((a.H + TH - 1) / TH), (a.Cout + CT - 1) / CT, a.B);
        launch_pdl(conv_simt_kernel<TIn, TOut, TH, TW, 4, 4, 16>, grid, dim3(256), 0, s, a);
    }
    return cudaGetLastError();
}

// --------------------------------------------------------------------------------- attention
// One warp per query, eight queries per block sharing 32-key K/V tiles in shared memory;
// running maximum / running sum softmax, all in fp32.
constexpr int kAttnQ = 8, kAttnKeys = 32;

template <typename T>
__global__ void __launch_bounds__(kAttnQ * 32) attn_simt_kernel(AttnArgs a) {
    griddep_launch();
    griddep_wait();
    extern __shared__ float smem[];
    const int C = a.C;
    float* s_q = smem;                               // [kAttnQ][C]
    float* s_k = s_q + kAttnQ * C;                   // [kAttnKeys][C+1]
    float* s_v = s_k + kAttnKeys * (C + 1);          // [kAttnKeys][C]
    const int b = blockIdx.y;
    const int q0 = blockIdx.x * kAttnQ;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const T* q = (const T*)a.q + (size_t)b * a.T * a.ld_qkv;
    const T* k = (const T*)a.k + (size_t)b * a.T * a.ld_qkv;
    const T* v = (const T*)a.v + (size_t)b * a.T * a.ld_qkv;
    T* o = (T*)a.o + (size_t)b * a.T * a.ld_o;

    for (int idx = threadIdx.x; idx < kAttnQ * C; idx += blockDim.x) {
        const int qi = idx / C, c = idx % C;
        s_q[idx] = (q0 + qi < a.T) ? ld_f<T>(q, (size_t)(q0 + qi) * a.ld_qkv + c) : 0.f;
    }
    const int nacc = C / 32;                          // channels per lane (C multiple of 32, <= 512)
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    float m = -INFINITY, l = 0.f;

    for (int k0 = 0; k0 < a.T; k0 += kAttnKeys) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < kAttnKeys * C; idx += blockDim.x) {
            const int ki = idx / C, c = idx % C;
            const bool ok = k0 + ki < a.T;
            s_k[ki * (C + 1) + c] = ok ? ld_f<T>(k, (size_t)(k0 + ki) * a.ld_qkv + c) : 0.f;
            s_v[ki * C + c] = ok ? ld_f<T>(v, (size_t)(k0 + ki) * a.ld_qkv + c) : 0.f;
        }
        __syncthreads();
        float sc = 0.f;
        const float* qr = s_q + warp * C;
        const float* kr = s_k + lane * (C + 1);
        for (int c = 0; c < C; ++c) sc = fmaf(qr[c], kr[c], sc);
        sc = (k0 + lane < a.T) ? sc * a.scale : -INFINITY;
        float tmax = sc;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, d));
        const float m_new = fmaxf(m, tmax);
        const float corr = expf(m - m_new);           // m = -inf at the first tile: exp(-inf) = 0
        const float p = expf(sc - m_new);
        float psum = p;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, d);
        l = l * corr + psum;
        m = m_new;
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] *= corr;
        for (int ki = 0; ki < kAttnKeys; ++ki) {
            const float pk = __shfl_sync(0xffffffffu, p, ki);
            const float* vr = s_v + ki * C + lane;
#pragma unroll
            for (int i = 0; i < 16; ++i)
                if (i < nacc) acc[i] = fmaf(pk, vr[i * 32], acc[i]);
        }
    }
    if (q0 + warp < a.T) {
        const float inv = 1.f / l;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < nacc) st_f<T>(o, (size_t)(q0 + warp) * a.ld_o + lane + i * 32, acc[i] * inv);
    }
}

// ------------------------------------------------------------------------------------ repack
template <typename T>
__global__ void pack_weight_simt_kernel(const T* w, float* packed, int Cout, int Cin, int taps, int cout_total,
                                        int cout_offset) {
    const int64_t total = (int64_t)Cout * Cin * taps;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int tap = (int)(i % taps);
        const int c = (int)((i / taps) % Cin);
        const int o = (int)(i / ((int64_t)taps * Cin));
        packed[((size_t)tap * Cin + c) * cout_total + cout_offset + o] = ld_f<T>(w, i);
    }
}

template <typename T>
__global__ void to_f32_kernel(const T* src, float* dst, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = ld_f<T>(src, i);
}

int grid_for(int64_t n, int threads) {
    int64_t g = (n + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

}  // namespace

cudaError_t launch_ingest(const IngestArgs& a, cudaStream_t s) {
    const int64_t n = (int64_t)a.B * a.C * a.h * a.w;
    if (a.dtype == VD_BF16) launch_pdl(ingest_kernel<__nv_bfloat16>, dim3(grid_for(n, 256)), dim3(256), 0, s, a);
    else launch_pdl(ingest_kernel<float>, dim3(grid_for(n, 256)), dim3(256), 0, s, a);
    return cudaGetLastError();
}

cudaError_t launch_gn_stats(const GnArgs& a, cudaStream_t s) {
    if (a.C % 4 != 0 || a.C / 4 > kGnThreads || a.G > kGnThreads || (a.C / a.G) % 4 != 0) return cudaErrorInvalidValue;
    // chunks per sample depend on the sample size only (so a frame's statistics, and with them
    // the frame, do not depend on the batch it is decoded in): at least 32 pixels per chunk
    int ppc = max(32, (a.P + kGnMaxChunks - 1) / kGnMaxChunks);
    int chunks = (a.P + ppc - 1) / ppc;
    dim3 grid(chunks, a.B);
    if (a.dtype == VD_BF16) launch_pdl(gn_stats_kernel<__nv_bfloat16, 16>, grid, dim3(kGnThreads), 0, s, a, chunks, ppc);
    else launch_pdl(gn_stats_kernel<float, 8>, grid, dim3(kGnThreads), 0, s, a, chunks, ppc);
    return cudaGetLastError();
}

// The first convolution (latent channels -> hundreds of channels): K = 9 * Cin <= 72 is too thin for the
// tensor core and for the tiled FFMA kernel's staging.  A block computes 32 consecutive pixels x 128
// output channels: the pixels' 3x3 neighbourhoods sit in shared memory, a thread holds 4 pixels x 4
// channels and reads the weights ([tap][Cin][Cout] fp32) as coalesced float4 straight from L1/L2.
constexpr int kThinPix = 32, kThinCout = 128, kThinMaxK = 72;
template <int CIN>
__global__ void __launch_bounds__(256) conv_thin_kernel(ConvArgs a) {
    __shared__ float in_s[kThinPix][kThinMaxK + 1];
    griddep_launch();
    griddep_wait();
    constexpr int K = 9 * CIN;
    const long long npix = (long long)a.B * a.H * a.W;
    const long long p0 = (long long)blockIdx.x * kThinPix;
    const int co0 = blockIdx.y * kThinCout;
    const float* x = (const float*)a.x;
    for (int i = threadIdx.x; i < kThinPix * K; i += 256) {
        const int p = i / K, k = i - p * K;
        const int tap = k / CIN, c = k - tap * CIN;
        const long long g = p0 + p;
        float v = 0.f;
        if (g < npix) {
            const int b = (int)(g / ((long long)a.H * a.W));
            const int r = (int)(g - (long long)b * a.H * a.W);
            const int oy = r / a.W + tap / 3 - 1, ox = r % a.W + tap % 3 - 1;
            if (oy >= 0 && oy < a.H && ox >= 0 && ox < a.W) v = x[(((size_t)b * a.H + oy) * a.W + ox) * CIN + c];
        }
        in_s[p][k] = a.bf16_operands ? round_bf16(v) : v;
    }
    __syncthreads();
    const int pg = threadIdx.x >> 5, cg = threadIdx.x & 31;          // 4 pixels, 4 channels per thread
    const float* w = (const float*)a.w + co0 + cg * 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[i][q] = 0.f;
#pragma unroll 12
    for (int k = 0; k < K; ++k) {
        const float4 wv = __ldg((const float4*)(w + (size_t)k * a.Cout));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float xv = in_s[pg * 4 + i][k];
            acc[i][0] = fmaf(xv, wv.x, acc[i][0]); acc[i][1] = fmaf(xv, wv.y, acc[i][1]);
            acc[i][2] = fmaf(xv, wv.z, acc[i][2]); acc[i][3] = fmaf(xv, wv.w, acc[i][3]);
        }
    }
    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.bias) bv = __ldg((const float4*)(a.bias + co0 + cg * 4));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long g = p0 + pg * 4 + i;
        if (g < npix)
            *(float4*)((float*)a.y + (size_t)g * a.Cout + co0 + cg * 4) =
                make_float4(acc[i][0] + bv.x, acc[i][1] + bv.y, acc[i][2] + bv.z, acc[i][3] + bv.w);
    }
}

cudaError_t launch_conv_simt(const ConvArgs& a, cudaStream_t s) {
    const bool ib = a.in_dtype == VD_BF16, ob = a.out_dtype == VD_BF16;
    if (!ib && !ob && a.ksize == 3 && (a.Cin == 4 || a.Cin == 8) && a.Cout % kThinCout == 0 && !a.scale && !a.residual &&
        !a.upsample && !a.out_nchw && !a.x2) {
        const long long npix = (long long)a.B * a.H * a.W;
        dim3 grid((unsigned)((npix + kThinPix - 1) / kThinPix), a.Cout / kThinCout);
        return a.Cin == 4 ? launch_pdl(conv_thin_kernel<4>, grid, dim3(256), 0, s, a) : launch_pdl(conv_thin_kernel<8>, grid, dim3(256), 0, s, a);
    }
    if (ib && ob) return conv_simt_dispatch<__nv_bfloat16, __nv_bfloat16>(a, s);
    if (ib && !ob) return conv_simt_dispatch<__nv_bfloat16, float>(a, s);
    if (!ib && ob) return conv_simt_dispatch<float, __nv_bfloat16>(a, s);
    return conv_simt_dispatch<float, float>(a, s);
}

cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t s) {
    if (a.C % 32 != 0 || a.C > 512) return cudaErrorInvalidValue;
    const size_t smem = sizeof(float) * ((size_t)kAttnQ * a.C + (size_t)kAttnKeys * (a.C + 1) + (size_t)kAttnKeys * a.C);
    dim3 grid((a.T + kAttnQ - 1) / kAttnQ, a.B);
    cudaError_t e;
    if (a.dtype == VD_BF16) {
        e = cudaFuncSetAttribute(attn_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        launch_pdl(attn_simt_kernel<__nv_bfloat16>, grid, dim3(kAttnQ * 32), smem, s, a);
    } else {
        e = cudaFuncSetAttribute(attn_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        launch_pdl(attn_simt_kernel<float>, grid, dim3(kAttnQ * 32), smem, s, a);
    }
    return cudaGetLastError();
}

cudaError_t launch_pack_weight_simt(const void* w, int w_dtype, float* packed, int Cout, int Cin, int taps,
                                    int cout_total, int cout_offset, cudaStream_t s) {
    const int64_t n = (int64_t)Cout * Cin * taps;
    if (w_dtype == VD_BF16)
        pack_weight_simt_kernel<__nv_bfloat16><<<grid_for(n, 256), 256, 0, s>>>((const __nv_bfloat16*)w, packed, Cout, Cin, taps, cout_total, cout_offset);
    else
        pack_weight_simt_kernel<float><<<grid_for(n, 256), 256, 0, s>>>((const float*)w, packed, Cout, Cin, taps, cout_total, cout_offset);
    return cudaGetLastError();
}

__global__ void fold_bias_kernel(float* out, const float* in, const float* b, const float* b2, const float* w2, const float* pin,
                                 int Cin2, int Cout) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= Cout) return;
    float v = (in ? in[c] : 0.f) + (b ? b[c] : 0.f) + (b2 ? b2[c] : 0.f);
    if (w2 && pin) {
        float acc = 0.f;
        for (int k = 0; k < Cin2; ++k) acc = fmaf(w2[(size_t)c * Cin2 + k], pin[k], acc);
        v += acc;
    }
    out[c] = v;
}
__global__ void fill_rows_kernel(float* dst, const float* src, int C, int B) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < C * B) dst[i] = src ? src[i % C] : 1.f;
}
cudaError_t launch_fold_bias(float* out, const float* in, const float* b, const float* b2, const float* w2, const float* pin,
                             int Cin2, int Cout, cudaStream_t s) {
    fold_bias_kernel<<<(Cout + 127) / 128, 128, 0, s>>>(out, in, b, b2, w2, pin, Cin2, Cout);
    return cudaGetLastError();
}
cudaError_t launch_fill_rows(float* dst, const float* src, int C, int B, cudaStream_t s) {
    const int n = C * B;
    fill_rows_kernel<<<(n + 255) / 256, 256, 0, s>>>(dst, src, C, B);
    return cudaGetLastError();
}

cudaError_t launch_to_f32(const void* src, int dtype, float* dst, int64_t n, cudaStream_t s) {
    if (dtype == VD_BF16) to_f32_kernel<__nv_bfloat16><<<grid_for(n, 256), 256, 0, s>>>((const __nv_bfloat16*)src, dst, n);
    else to_f32_kernel<float><<<grid_for(n, 256), 256, 0, s>>>((const float*)src, dst, n);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// GroupNorm statistics without any caller-provided or allocated scratch memory.
//
// Some callers may not allocate device memory at the point where they need this operator: a
// render/game loop that must not stall on the allocator's implicit device synchronisation, a
// plug-in whose host application owns the whole memory pool, or code running where the CUDA
// allocator is simply off limits (inside a host callback, after a memory budget was frozen).
// For them the chunk partials of the reduction live in the fixed device array below instead of a
// buffer passed in.  The price is a size limit and shared state: every GPU that loads this
// library carries the array (148 KiB) until the process exits, and all calls on a device use the
// same array, so two calls whose kernels can overlap on the GPU (different streams, no ordering
// between them) race on it.  The chunk records need no clearing (every record read was written
// by the same call); the arrival counters behind them must start at zero and are cleared by an
// asynchronous memset at the start of every call.
namespace {
constexpr int kStaticGnMaxBatchTimesGroups = 64;     // e.g. 2 frames x 32 groups, or 8 x 8
constexpr int kStaticGnCounters = 64;                // arrival counters behind the records (batch <= 64 follows from the limit)
static __device__ __align__(256) float g_gn_static_partial[kStaticGnMaxBatchTimesGroups * kGnMaxChunks * 2 + kStaticGnCounters];   // 148 KiB of chunk records + 64 arrival counters

std::mutex g_static_mu;
constexpr int kMaxDevices = 64;
float* g_static_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle of the symbol, not a device address; the address
// on the current device is looked up once per device and cached.
cudaError_t static_scratch_of_current_device(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_gn_static_partial);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = (float*)p;
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}
}  // namespace

}  // namespace vd

extern "C" VD_API vd_status vd_op_gn_stats_static(const void* x, int32_t dtype, int32_t batch, int32_t h, int32_t w,
                                                  int32_t c, int32_t groups, float eps, const float* gamma,
                                                  const float* beta, float* scale, float* shift, void* cuda_stream) {
    using namespace vd;
    if (!x || !gamma || !beta || !scale || !shift) { set_last_error("vd_op_gn_stats_static: NULL pointer"); return VD_ERR_INVALID_ARG; }
    if (dtype != VD_F32 && dtype != VD_BF16) { set_last_error("vd_op_gn_stats_static: bad dtype"); return VD_ERR_INVALID_ARG; }
    if (batch < 0 || h < 1 || w < 1 || c < 1 || groups < 1 || c % groups != 0 || (c / groups) % 4 != 0 || c > 1024) {
        set_last_error("vd_op_gn_stats_static: bad GroupNorm sizes (groups must hold a multiple of 4 channels)");
        return VD_ERR_INVALID_ARG;
    }
    if ((long long)h * w > 0x7fffffffLL || (long long)batch * h * w * c > (1LL << 40)) {
        set_last_error("vd_op_gn_stats_static: tensor too large (h*w must fit 31 bits, batch*h*w*c 40 bits)");
        return VD_ERR_INVALID_ARG;
    }
    if ((long long)batch * groups > kStaticGnMaxBatchTimesGroups) {
        set_last_error("vd_op_gn_stats_static: batch*groups exceeds 64, the capacity of the built-in scratch array; "
                       "use vd_op_gn_stats with a scratch buffer instead");
        return VD_ERR_UNSUPPORTED;
    }
    if (batch == 0) return VD_OK;
    float* partial = nullptr;
    cudaError_t e = static_scratch_of_current_device(&partial);
    if (e == cudaSuccess) {
        // the arrival counters live behind the records; they must be zero when the kernel starts
        unsigned int* counters = (unsigned int*)(partial + (size_t)kStaticGnMaxBatchTimesGroups * kGnMaxChunks * 2);
        e = cudaMemsetAsync(counters, 0, kStaticGnCounters * sizeof(unsigned int), (cudaStream_t)cuda_stream);
        GnArgs a{x, dtype, batch, h * w, c, groups, eps, gamma, beta, scale, shift, partial, counters, nullptr};
        if (e == cudaSuccess) e = launch_gn_stats(a, (cudaStream_t)cuda_stream);
    }
    if (e != cudaSuccess) {
        set_last_error((std::string("vd_op_gn_stats_static: ") + cudaGetErrorString(e)).c_str());
        return VD_ERR_CUDA;
    }
    return VD_OK;
}
