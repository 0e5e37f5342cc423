// Implicit-GEMM 3x3 / 1x1 convolution on the 5th-generation tensor cores (tcgen05 + TMEM), with
// the paper's fusion folded around it (Section IV-B.1, Eq. 9): the GroupNorm-apply + SiLU of the
// chain runs in the operand prologue, nearest-2x upsampling is an address computation, and bias,
// residual add and the output cast run in the epilogue, so each activation crosses HBM once.
//
// One CTA computes a 16x8-pixel x BN-channel output tile:  D[128 x BN] = sum over taps and
// 64-channel chunks of A_tap[128 x 64] * W_tap[64 x BN].
//   * B operand (weights, bf16 [tap][Cout][Cin]) arrives by TMA into 128B-swizzled stages.
//   * A operand: producer warps read the raw 18x10-pixel halo tile of a 64-channel chunk from
//     global memory once, apply scale/shift (+SiLU), round to bf16 and store it in shared memory
//     in the canonical un-swizzled K-major layout, as eight planes [8 channels][pixel][16 B].
//     Every tap is then a *view* of that one tile: its descriptor starts (ky*10+kx) pixels in,
//     eight-row groups are one tile row (10 pixels) apart, so the transform runs once per
//     element and not once per tap.  Out-of-image halo pixels are written as exact zeros (the
//     zero padding applies to the transformed tensor).
//   * One thread issues tcgen05.mma (M=128, N=BN, K=16); accumulators live in TMEM; stages are
//     recycled through mbarriers signalled by tcgen05.commit.
//   * Epilogue: tcgen05.ld, + bias (+ fp32 residual), store fp32 or bf16 NHWC.
// Two CTAs fit on an SM, so one tile's epilogue overlaps the other's main loop.
// Every wait is bounded: on expiry the CTA records a code in the status word and unwinds.
#include <cuda.h>

#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;

constexpr int TILE_H = 16, TILE_W = 8;
constexpr int PH = TILE_H + 2, PW = TILE_W + 2, NPIX = PH * PW;     // 18 x 10 = 180 halo pixels
constexpr int PLANE = (NPIX + 1) * 16;                               // bytes between 8-channel planes (odd * 16)
constexpr int A_STAGE_BYTES = 8 * PLANE;                             // one 64-channel chunk
constexpr int A_STAGES = 2;
constexpr int NUM_PRODUCERS = 128;                                   // warps 0-3: operand prologue, then epilogue
constexpr int NUM_THREADS = 192;                                     // + warp 4 (TMA, TMEM alloc) + warp 5 (MMA)
constexpr int ITEMS = NPIX * 8;                                      // (pixel, 8-channel group) work items per chunk

template <int BN> struct TileCfg {
    static constexpr int B_STAGE_BYTES = BN * 128;                   // BN rows x 64 bf16
    static constexpr int B_STAGES = (BN == 256) ? 2 : 4;
    static constexpr int SMEM_B = B_STAGES * B_STAGE_BYTES;          // 64 KB
    static constexpr int SMEM_A = A_STAGES * A_STAGE_BYTES;
    static constexpr int SMEM_BAR = 256;
    static constexpr int SMEM_TOTAL = SMEM_B + SMEM_A + SMEM_BAR + 1024;   // + slack for 1024-B alignment
};

struct Raw8 { uint4 lo, hi; };   // eight channels of one pixel: bf16 -> lo only; fp32 -> lo + hi

template <bool IN_BF16>
__device__ __forceinline__ void load_raw(const void* x, size_t elem_off, Raw8& r) {
    if (IN_BF16) {
        r.lo = __ldg((const uint4*)((const __nv_bfloat16*)x + elem_off));
    } else {
        const float4* p = (const float4*)((const float*)x + elem_off);
        const float4 a = __ldg(p), b = __ldg(p + 1);
        r.lo = make_uint4(__float_as_uint(a.x), __float_as_uint(a.y), __float_as_uint(a.z), __float_as_uint(a.w));
        r.hi = make_uint4(__float_as_uint(b.x), __float_as_uint(b.y), __float_as_uint(b.z), __float_as_uint(b.w));
    }
}
template <bool IN_BF16>
__device__ __forceinline__ void unpack_raw(const Raw8& r, float v[8]) {
    if (IN_BF16) {
        const uint32_t w[4] = {r.lo.x, r.lo.y, r.lo.z, r.lo.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else {
        v[0] = __uint_as_float(r.lo.x); v[1] = __uint_as_float(r.lo.y); v[2] = __uint_as_float(r.lo.z); v[3] = __uint_as_float(r.lo.w);
        v[4] = __uint_as_float(r.hi.x); v[5] = __uint_as_float(r.hi.y); v[6] = __uint_as_float(r.hi.z); v[7] = __uint_as_float(r.hi.w);
    }
}

struct Bars {                    // lives in shared memory
    uint64_t a_full[A_STAGES], a_empty[A_STAGES];
    uint64_t b_full[4], b_empty[4];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int BN, bool IN_BF16, bool OUT_BF16>
__global__ void __launch_bounds__(NUM_THREADS, 2)
conv_tc_kernel(const ConvArgs a, const __grid_constant__ CUtensorMap tmap, unsigned int* status) {
    using Cfg = TileCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;
    uint8_t* smem_a = smem + Cfg::SMEM_B;
    Bars* bars = (Bars*)(smem + Cfg::SMEM_B + Cfg::SMEM_A);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_x = (a.W + TILE_W - 1) / TILE_W;
    const int tx0 = (blockIdx.x % tiles_x) * TILE_W;
    const int ty0 = (blockIdx.x / tiles_x) * TILE_H;
    const int n0 = blockIdx.y * BN;
    const int b = blockIdx.z;
    const int taps = a.ksize * a.ksize;
    const int kchunks = a.Cin >> 6;

    if (tid == 0) {
        for (int i = 0; i < A_STAGES; ++i) { mbar_init(smem_u32(&bars->a_full[i]), NUM_PRODUCERS); mbar_init(smem_u32(&bars->a_empty[i]), 1); }
        for (int i = 0; i < 4; ++i) { mbar_init(smem_u32(&bars->b_full[i]), 1); mbar_init(smem_u32(&bars->b_empty[i]), 1); }
        mbar_init(smem_u32(&bars->acc_full), 1);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 4) {             // TMEM: BN fp32 accumulator columns
        tmem_alloc(smem_u32(&bars->tmem_base), (uint32_t)BN);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = bars->tmem_base;

    if (warp < 4) {
        // ------------------------------------------------ operand prologue (producers)
        const int j = tid & 7;                              // this thread's 8-channel group within a chunk
        const bool prologue = a.scale != nullptr;
        const bool silu = a.silu != 0;
        const int up = a.upsample ? 1 : 0;
        const size_t img = (size_t)b * a.Hs * a.Ws;
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int kc = 0; kc < kchunks && ok; ++kc) {
            const int c0 = kc * 64 + j * 8;
            float sc[8], sh[8];
            if (prologue) {
                const float4* ps = (const float4*)(a.scale + (size_t)b * a.Cin + c0);
                const float4* pt = (const float4*)(a.shift + (size_t)b * a.Cin + c0);
                const float4 s0 = __ldg(ps), s1 = __ldg(ps + 1), t0 = __ldg(pt), t1 = __ldg(pt + 1);
                sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
            }
            ok = mbar_wait(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
            if (!ok) break;
            uint8_t* dst_plane = smem_a + stage * A_STAGE_BYTES + j * PLANE;
            constexpr int BATCH = 4;
            constexpr int ITERS = (ITEMS + NUM_PRODUCERS - 1) / NUM_PRODUCERS;          // 12
#pragma unroll 1
            for (int it0 = 0; it0 < ITERS; it0 += BATCH) {
                Raw8 raw[BATCH];
                bool valid[BATCH];
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    const int i = (it0 + u) * NUM_PRODUCERS + tid;
                    const int pix = i >> 3;
                    const int py = pix / PW, px = pix - py * PW;
                    const int oy = ty0 + py - 1, ox = tx0 + px - 1;
                    bool v = (i < ITEMS) && oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                    if (a.ksize == 1) v = v && py >= 1 && py <= TILE_H && px >= 1 && px <= TILE_W;
                    valid[u] = v;
                    if (v) load_raw<IN_BF16>(a.x, (img + (size_t)(oy >> up) * a.Ws + (ox >> up)) * a.Cin + c0, raw[u]);
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    const int i = (it0 + u) * NUM_PRODUCERS + tid;
                    if (i >= ITEMS) continue;
                    uint4 out = make_uint4(0u, 0u, 0u, 0u);
                    if (valid[u]) {
                        float v[8];
                        unpack_raw<IN_BF16>(raw[u], v);
                        if (prologue) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], sc[e], sh[e]);
                        }
                        if (silu) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = silu_fast(v[e]);
                        }
                        out = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                    }
                    *(uint4*)(dst_plane + (i >> 3) * 16) = out;
                }
            }
            fence_proxy_async_smem();                        // generic-proxy stores -> visible to the tensor core
            mbar_arrive(smem_u32(&bars->a_full[stage]));
            if (++stage == A_STAGES) { stage = 0; phase ^= 1; }
        }

        // ------------------------------------------------ epilogue
        ok = mbar_wait(smem_u32(&bars->acc_full), 0, abort_flag);
        ok = __all_sync(0xffffffffu, ok);                    // tcgen05.ld below is warp-collective
        tc_fence_after();
        if (ok) {
            const int m = tid;                               // accumulator row = TMEM lane = pixel of the tile
            const int oy = ty0 + (m >> 3), ox = tx0 + (m & 7);
            const bool inside = oy < a.H && ox < a.W;
            const size_t opix = ((size_t)b * a.H + oy) * a.W + ox;
#pragma unroll 1
            for (int cb = 0; cb < BN; cb += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)cb, r);
                tmem_ld_wait();
                if (inside) {
                    const int co = n0 + cb;
                    float v[32];
#pragma unroll
                    for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
                    if (a.bias) {
#pragma unroll
                        for (int q = 0; q < 32; q += 4) {
                            const float4 t = __ldg((const float4*)(a.bias + co + q));
                            v[q] += t.x; v[q + 1] += t.y; v[q + 2] += t.z; v[q + 3] += t.w;
                        }
                    }
                    if (a.residual) {
                        const float4* rp = (const float4*)(a.residual + opix * a.Cout + co);
#pragma unroll
                        for (int q = 0; q < 32; q += 4) {
                            const float4 t = __ldg(rp + (q >> 2));
                            v[q] += t.x; v[q + 1] += t.y; v[q + 2] += t.z; v[q + 3] += t.w;
                        }
                    }
                    if (OUT_BF16) {
                        uint4* yp = (uint4*)((__nv_bfloat16*)a.y + opix * a.Cout + co);
#pragma unroll
                        for (int q = 0; q < 32; q += 8)
                            yp[q >> 3] = make_uint4(pack_bf16(v[q], v[q + 1]), pack_bf16(v[q + 2], v[q + 3]),
                                                    pack_bf16(v[q + 4], v[q + 5]), pack_bf16(v[q + 6], v[q + 7]));
                    } else {
                        float4* yp = (float4*)((float*)a.y + opix * a.Cout + co);
#pragma unroll
                        for (int q = 0; q < 32; q += 4) yp[q >> 2] = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                    }
                }
            }
        }
    } else if (warp == 4) {
        // ------------------------------------------------ weight loads (TMA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int kc = 0; kc < kchunks && ok; ++kc) {
                for (int tap = 0; tap < taps; ++tap) {
                    ok = mbar_wait(smem_u32(&bars->b_empty[stage]), phase ^ 1, abort_flag);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&bars->b_full[stage]);
                    mbar_arrive_expect_tx(full, Cfg::B_STAGE_BYTES);
                    tma_load_2d(smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES), &tmap, kc * 64, tap * a.Cout + n0, full);
                    ++issued;
                    if (++stage == Cfg::B_STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // unwinding: let the copies already in flight land before the CTA's memory is released
                uint32_t s = stage, ph = phase;
                for (int k = 0; k < min(issued, Cfg::B_STAGES); ++k) {
                    if (s == 0) { s = Cfg::B_STAGES; ph ^= 1; }
                    --s;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(smem_u32(&bars->b_full[s]), ph) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
                }
            }
        }
    } else {
        // ------------------------------------------------ MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, BN);
            uint32_t as = 0, aph = 0, bs = 0, bph = 0;
            bool ok = true;
            for (int kc = 0; kc < kchunks && ok; ++kc) {
                ok = mbar_wait(smem_u32(&bars->a_full[as]), aph, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_stage = smem_u32(smem_a + as * A_STAGE_BYTES);
                for (int tap = 0; tap < taps; ++tap) {
                    ok = mbar_wait(smem_u32(&bars->b_full[bs]), bph, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const int ky = a.ksize == 3 ? tap / 3 : 1, kx = a.ksize == 3 ? tap - 3 * (tap / 3) : 1;
                    const uint32_t a_tap = a_stage + (uint32_t)(ky * PW + kx) * 16;
                    const uint32_t b_stage = smem_u32(smem_b + bs * Cfg::B_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t adesc = make_smem_desc(a_tap + (uint32_t)(2 * k) * PLANE, PLANE, PW * 16, 0);
                        const uint64_t bdesc = make_smem_desc(b_stage + (uint32_t)k * 32, 16, 1024, 2);
                        umma_bf16(tmem_d, adesc, bdesc, idesc, (kc | tap | k) != 0);
                    }
                    umma_commit(smem_u32(&bars->b_empty[bs]));
                    if (++bs == Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                }
                umma_commit(smem_u32(&bars->a_empty[as]));
                if (++as == A_STAGES) { as = 0; aph ^= 1; }
            }
            if (ok) umma_commit(smem_u32(&bars->acc_full));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && bars->abort_flag && status) {
        if (atomicCAS(status, 0u, 0xC0DE0001u) == 0u) {
            status[1] = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
            status[2] = (uint32_t)BN;
        }
    }
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem_d, (uint32_t)BN);
    }
}

// pack OIHW -> bf16 [tap][cout_total][Cin]
template <typename T>
__global__ void pack_weight_tc_kernel(const T* w, __nv_bfloat16* packed, int Cout, int Cin, int taps, int cout_total, int cout_offset) {
    const int64_t total = (int64_t)Cout * Cin * taps;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int tap = (int)(i % taps);
        const int c = (int)((i / taps) % Cin);
        const int o = (int)(i / ((int64_t)taps * Cin));
        float v;
        if (sizeof(T) == 2) v = __bfloat162float(((const __nv_bfloat16*)w)[i]);
        else v = ((const float*)w)[i];
        packed[((size_t)tap * cout_total + cout_offset + o) * Cin + c] = __float2bfloat16_rn(v);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

int pick_bn(int Cout) { return (Cout % 256 == 0) ? 256 : 128; }

template <int BN, bool IB, bool OB>
cudaError_t launch_one(const ConvArgs& a, const CUtensorMap& tm, unsigned int* status, cudaStream_t s) {
    auto kern = conv_tc_kernel<BN, IB, OB>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<BN>::SMEM_TOTAL);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(((a.W + TILE_W - 1) / TILE_W) * ((a.H + TILE_H - 1) / TILE_H), a.Cout / BN, a.B);
    kern<<<grid, NUM_THREADS, TileCfg<BN>::SMEM_TOTAL, s>>>(a, tm, status);
    return cudaGetLastError();
}

}  // namespace

bool conv_tc_supported(const ConvArgs& a) {
    if (a.Cin % 64 != 0 || a.Cin < 64) return false;
    if (a.Cout % 128 != 0) return false;
    if (a.out_nchw || !a.bf16_operands) return false;
    if (a.ksize != 1 && a.ksize != 3) return false;
    return true;
}

size_t conv_tc_packed_bytes(int Cout, int Cin, int taps) { return (size_t)taps * Cout * Cin * 2; }

cudaError_t launch_pack_weight_tc(const void* w, int w_dtype, void* packed, int Cout, int Cin, int taps, int cout_total,
                                  int cout_offset, cudaStream_t s) {
    const int64_t n = (int64_t)Cout * Cin * taps;
    int grid = (int)((n + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    if (w_dtype == VD_BF16)
        pack_weight_tc_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)packed, Cout, Cin, taps, cout_total, cout_offset);
    else
        pack_weight_tc_kernel<float><<<grid, 256, 0, s>>>((const float*)w, (__nv_bfloat16*)packed, Cout, Cin, taps, cout_total, cout_offset);
    return cudaGetLastError();
}

cudaError_t conv_tc_prepare(const ConvArgs& a, ConvTcPlan* plan) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const int taps = a.ksize * a.ksize;
    const int bn = pick_bn(a.Cout);
    CUtensorMap* tm = (CUtensorMap*)plan->tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)a.Cin, (cuuint64_t)taps * a.Cout};
    const cuuint64_t strides[1] = {(cuuint64_t)a.Cin * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)bn};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.w), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    plan->bn = bn;
    plan->valid = 1;
    return cudaSuccess;
}

cudaError_t launch_conv_tc(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    if (!plan.valid) return cudaErrorInvalidValue;
    const CUtensorMap& tm = *(const CUtensorMap*)plan.tmap;
    const bool ib = a.in_dtype == VD_BF16, ob = a.out_dtype == VD_BF16;
    if (plan.bn == 256) {
        if (ib && ob) return launch_one<256, true, true>(a, tm, status, s);
        if (ib && !ob) return launch_one<256, true, false>(a, tm, status, s);
        if (!ib && ob) return launch_one<256, false, true>(a, tm, status, s);
        return launch_one<256, false, false>(a, tm, status, s);
    }
    if (ib && ob) return launch_one<128, true, true>(a, tm, status, s);
    if (ib && !ob) return launch_one<128, true, false>(a, tm, status, s);
    if (!ib && ob) return launch_one<128, false, true>(a, tm, status, s);
    return launch_one<128, false, false>(a, tm, status, s);
}

}  // namespace vd
