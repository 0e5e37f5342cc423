// Implicit-GEMM 3x3 / 1x1 convolution on the 5th-generation tensor cores (tcgen05 + TMEM), with
// the paper's fusion folded around it (Section IV-B.1, Eq. 9): the GroupNorm-apply + SiLU of the
// chain runs in the operand prologue, nearest-2x upsampling is an address computation, and bias,
// residual add, the 1x1 shortcut and the output cast run in / next to the same accumulation, so
// each activation crosses HBM once.
//
// Persistent kernel, one CTA per SM, roles decoupled through mbarrier rings:
//   * work item = (one or two 16x8-pixel tiles side by side, BN-channel block, frame); per tile
//     D[128 x BN] = sum over taps and 64-channel chunks of A_tap[128 x 64] * W_tap[64 x BN];
//     CTAs walk the item list with stride gridDim.x.
//   * 16 producer warps read the raw halo tile (18 x 10 or 18 x 18 pixels) of a 64-channel chunk
//     from global memory once (loads of the next batch in flight while this one is transformed), apply scale/shift (+SiLU), round to bf16 and store it in shared memory in the
//     canonical un-swizzled K-major layout, as eight planes [8 channels][pixel][16 B].  Every tap
//     is a *view* of that one tile (descriptor start (ky*10+kx) pixels in; eight-row groups are
//     one tile row = 10 pixels apart), so the transform runs once per element, not once per tap.
//     Out-of-image halo pixels are exact zeros (padding applies to the transformed tensor).
//     An optional second input (the block's raw input for a width-changing ResNet block) is
//     appended as extra K with a single centre tap: the 1x1 shortcut without its own round trip.
//   * 1 warp streams the weights (bf16 [tap][Cout][Cin]) by TMA into 128B-swizzled stages.
//   * 1 thread issues tcgen05.mma (M=128, N=BN, K=16) into one of two TMEM accumulators.
//   * 4 epilogue warps drain the other accumulator: tcgen05.ld, + bias (+ fp32 residual,
//     prefetched one column block ahead), store fp32/bf16 NHWC or the NCHW frame.
// Every wait is bounded: on expiry the CTA records a code in the status word and unwinds.
#include <cuda.h>
#include <string.h>

#include <algorithm>

#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;

constexpr int TILE_H = 16, TILE_W = 8;                               // one MMA tile: 128 output pixels
constexpr int PH = TILE_H + 2;
constexpr int NUM_PRODUCER_WARPS = 16;                               // enough loads in flight to cover DRAM latency
constexpr int NUM_PRODUCERS = NUM_PRODUCER_WARPS * 32;               // warps 0-15
constexpr int EPI_WARP0 = 16;                                        // warps 16-19 (warp % 4 = TMEM lane quarter)
constexpr int TMA_WARP = 20, MMA_WARP = 21;
constexpr int NUM_THREADS = 22 * 32;
constexpr int BATCH = 2;                                             // (pixel, 8-channel) loads per thread per batch
constexpr int MAX_B_STAGES = 8, MAX_A_STAGES = 4;

// BN = output channels per work item; MT = 16x8 MMA tiles per work item (side by side in x) that
// share every weight stage, which halves the weight traffic through shared memory where the
// channel block is narrow.
template <int BN> struct TileCfg {
    static constexpr int MT = BN == 128 ? 2 : 1;
    static constexpr int SUPER_W = TILE_W * MT;                      // item width in pixels
    static constexpr int PW = SUPER_W + 2;                           // halo tile: PH x PW pixels
    static constexpr int NPIX = PH * PW;
    static constexpr int PLANE = (NPIX | 1) * 16;                    // bytes between 8-channel planes (odd * 16)
    static constexpr int A_STAGE_BYTES = 8 * PLANE;                  // one 64-channel chunk of the halo tile
    static constexpr int ITEMS = NPIX * 8;                           // (pixel, 8-channel group) pairs per chunk
    static constexpr int NSUB = (ITEMS + NUM_PRODUCERS * BATCH - 1) / (NUM_PRODUCERS * BATCH);
    static constexpr int B_STAGE_BYTES = BN * 128;                   // BN rows x 64 bf16
    static constexpr int B_STAGES = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int A_STAGES = BN == 16 ? 4 : (BN == 128 ? 2 : 3);
    static constexpr int SMEM_B = (B_STAGES * B_STAGE_BYTES + 1023) / 1024 * 1024;
    static constexpr int SMEM_A = A_STAGES * A_STAGE_BYTES;
    static constexpr int SMEM_TOTAL = SMEM_B + SMEM_A + 512 + 1024;  // + barriers + slack for 1024-B alignment
    static constexpr int ACC_COLS = BN < 32 ? 32 : BN;               // TMEM columns per accumulator
    static constexpr int TMEM_COLS = 2 * MT * ACC_COLS;              // double-buffered
};

struct Raw8 { uint4 lo, hi; };   // eight channels of one pixel: bf16 -> lo only; fp32 -> lo + hi

__device__ __forceinline__ void load_raw(bool is_bf16, const void* x, size_t elem_off, Raw8& r) {
    if (is_bf16) {
        r.lo = __ldg((const uint4*)((const __nv_bfloat16*)x + elem_off));
    } else {
        const float4* p = (const float4*)((const float*)x + elem_off);
        const float4 a = __ldg(p), b = __ldg(p + 1);
        r.lo = make_uint4(__float_as_uint(a.x), __float_as_uint(a.y), __float_as_uint(a.z), __float_as_uint(a.w));
        r.hi = make_uint4(__float_as_uint(b.x), __float_as_uint(b.y), __float_as_uint(b.z), __float_as_uint(b.w));
    }
}
__device__ __forceinline__ void unpack_raw(bool is_bf16, const Raw8& r, float v[8]) {
    if (is_bf16) {
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
    uint64_t a_full[MAX_A_STAGES], a_empty[MAX_A_STAGES];
    uint64_t b_full[MAX_B_STAGES], b_empty[MAX_B_STAGES];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

struct Item { int tx0, ty0, n0, b; };

struct Sched {                   // static round-robin over (item tile, channel block, frame)
    int tiles_x, tiles, nblk, total;
    __device__ __forceinline__ Item get(int w, int bn, int super_w) const {
        Item it;
        const int per_frame = tiles * nblk;
        it.b = w / per_frame;
        const int r = w - it.b * per_frame;
        const int t = r / nblk;
        it.n0 = (r - t * nblk) * bn;
        it.ty0 = (t / tiles_x) * TILE_H;
        it.tx0 = (t % tiles_x) * super_w;
        return it;
    }
};

// OUT_MODE: 0 = fp32 NHWC, 1 = bf16 NHWC, 2 = NCHW frame (dtype from a.out_dtype)
template <int BN, bool IN_BF16, int OUT_MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_tc_kernel(const ConvArgs a, const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap2,
               unsigned int* status) {
    using Cfg = TileCfg<BN>;
    constexpr int MT = Cfg::MT, PW = Cfg::PW, PLANE = Cfg::PLANE, ITEMS = Cfg::ITEMS, NSUB = Cfg::NSUB;
    constexpr int A_STAGE_BYTES = Cfg::A_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;
    uint8_t* smem_a = smem + Cfg::SMEM_B;
    Bars* bars = (Bars*)(smem + Cfg::SMEM_B + Cfg::SMEM_A);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int taps = a.ksize * a.ksize;
    const int kchunks = a.Cin >> 6;
    const int kchunks2 = a.x2 ? (a.Cin2 >> 6) : 0;          // extra K: 1x1 shortcut on a second input
    const int ktotal = kchunks + kchunks2;
    const int cout_pad = (a.Cout % 128 == 0) ? a.Cout : 16; // rows per tap in the packed weights
    Sched sched;
    sched.tiles_x = (a.W + Cfg::SUPER_W - 1) / Cfg::SUPER_W;
    sched.tiles = sched.tiles_x * ((a.H + TILE_H - 1) / TILE_H);
    sched.nblk = cout_pad / BN;
    sched.total = sched.tiles * sched.nblk * a.B;

    if (tid == 0) {
        for (int i = 0; i < Cfg::A_STAGES; ++i) { mbar_init(smem_u32(&bars->a_full[i]), NUM_PRODUCERS); mbar_init(smem_u32(&bars->a_empty[i]), 1); }
        for (int i = 0; i < Cfg::B_STAGES; ++i) { mbar_init(smem_u32(&bars->b_full[i]), 1); mbar_init(smem_u32(&bars->b_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bars->acc_full[i]), 1); mbar_init(smem_u32(&bars->acc_empty[i]), 128); }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == MMA_WARP) tmem_alloc(smem_u32(&bars->tmem_base), (uint32_t)Cfg::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp < NUM_PRODUCER_WARPS) {
        // ------------------------------------------------ operand prologue (producers)
        // The work is a flat sequence of batches (item, chunk, sub-batch); the loads of batch n+1
        // are issued before batch n is transformed, so global-memory latency stays covered.
        const int j = tid & 7;                              // this thread's 8-channel group within a chunk
        const bool prologue = a.scale != nullptr;
        const bool silu = a.silu != 0;
        const int up = a.upsample ? 1 : 0;
        struct Pos { int w, kc, sub; Item it; };
        auto advance = [&](Pos& p) {
            if (++p.sub == NSUB) {
                p.sub = 0;
                if (++p.kc == ktotal) {
                    p.kc = 0;
                    p.w += gridDim.x;
                    if (p.w < sched.total) p.it = sched.get(p.w, BN, Cfg::SUPER_W);
                }
            }
        };
        auto issue = [&](const Pos& p, Raw8 (&raw)[BATCH], uint32_t& vmask) {
            const bool second = p.kc >= kchunks;
            const int c0 = (second ? p.kc - kchunks : p.kc) * 64 + j * 8;
            const bool centre_only = second || a.ksize == 1;
            vmask = 0;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int i = (p.sub * BATCH + u) * NUM_PRODUCERS + tid;
                const int pix = i >> 3;
                const int py = pix / PW, px = pix - py * PW;
                const int oy = p.it.ty0 + py - 1, ox = p.it.tx0 + px - 1;
                bool v = (i < ITEMS) && oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                if (centre_only) v = v && py >= 1 && py <= TILE_H && px >= 1 && px <= Cfg::SUPER_W;
                if (v) {
                    vmask |= 1u << u;
                    if (second) load_raw(false, a.x2, (((size_t)p.it.b * a.H + oy) * a.W + ox) * a.Cin2 + c0, raw[u]);
                    else load_raw(IN_BF16, a.x, (((size_t)p.it.b * a.Hs + (oy >> up)) * a.Ws + (ox >> up)) * a.Cin + c0, raw[u]);
                }
            }
        };
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        Pos cur;
        cur.w = blockIdx.x; cur.kc = 0; cur.sub = 0;
        if (cur.w < sched.total) cur.it = sched.get(cur.w, BN, Cfg::SUPER_W);
        Raw8 raw_cur[BATCH], raw_next[BATCH];
        uint32_t vm_cur = 0, vm_next = 0;
        if (cur.w < sched.total) issue(cur, raw_cur, vm_cur);
        while (cur.w < sched.total && ok) {
            Pos nxt = cur;
            advance(nxt);
            if (nxt.w < sched.total) issue(nxt, raw_next, vm_next);
            const bool second = cur.kc >= kchunks;
            const bool pro = prologue && !second;
            float sc[8], sh[8];
            if (pro) {
                const int c0 = cur.kc * 64 + j * 8;
                const float4* ps = (const float4*)(a.scale + (size_t)cur.it.b * a.Cin + c0);
                const float4* pt = (const float4*)(a.shift + (size_t)cur.it.b * a.Cin + c0);
                const float4 s0 = __ldg(ps), s1 = __ldg(ps + 1), t0 = __ldg(pt), t1 = __ldg(pt + 1);
                sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
            }
            if (cur.sub == 0) {
                ok = mbar_wait(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
                if (!ok) break;
            }
            uint8_t* dst_plane = smem_a + stage * A_STAGE_BYTES + j * PLANE;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int i = (cur.sub * BATCH + u) * NUM_PRODUCERS + tid;
                if (i >= ITEMS) continue;
                uint4 out = make_uint4(0u, 0u, 0u, 0u);
                if (vm_cur & (1u << u)) {
                    float v[8];
                    unpack_raw(second ? false : IN_BF16, raw_cur[u], v);
                    if (pro) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], sc[e], sh[e]);
                        if (silu) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = silu_fast(v[e]);
                        }
                    }
                    out = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                }
                *(uint4*)(dst_plane + (i >> 3) * 16) = out;
            }
            if (cur.sub == NSUB - 1) {
                fence_proxy_async_smem();                    // generic-proxy stores -> visible to the tensor core
                mbar_arrive(smem_u32(&bars->a_full[stage]));
                if (++stage == Cfg::A_STAGES) { stage = 0; phase ^= 1; }
            }
            cur = nxt;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) raw_cur[u] = raw_next[u];
            vm_cur = vm_next;
        }
    } else if (warp < EPI_WARP0 + 4) {
        // ------------------------------------------------ epilogue
        const int ew = warp - EPI_WARP0;                     // TMEM lane quarter
        const int m = ew * 32 + lane;                        // accumulator row = pixel of the MMA tile
        bool ok = true;
        int n_item = 0;
        for (int w = blockIdx.x; w < sched.total && ok; w += gridDim.x, ++n_item) {
            const Item it = sched.get(w, BN, Cfg::SUPER_W);
            const int buf = n_item & 1;
            ok = mbar_wait(smem_u32(&bars->acc_full[buf]), (n_item >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);                // tcgen05.ld below is warp-collective
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int t = 0; t < MT; ++t) {
                const uint32_t tacc = tmem_base + (uint32_t)((buf * MT + t) * Cfg::ACC_COLS) + ((uint32_t)(ew * 32) << 16);
                const int oy = it.ty0 + (m >> 3), ox = it.tx0 + t * TILE_W + (m & 7);
                const bool inside = oy < a.H && ox < a.W;
                const size_t opix = ((size_t)it.b * a.H + oy) * a.W + ox;
                const bool last_tile = t == MT - 1;
                if (OUT_MODE == 2) {
                    uint32_t r[16];
                    tmem_ld16(tacc, r);
                    tmem_ld_wait();
                    if (last_tile) {
                        tc_fence_before();
                        mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                    }
                    if (inside) {
#pragma unroll
                        for (int co = 0; co < 16; ++co) {
                            if (co < a.Cout) {
                                const float v = __uint_as_float(r[co]) + (a.bias ? __ldg(a.bias + co) : 0.f);
                                const size_t o = (((size_t)it.b * a.Cout + co) * a.H + oy) * a.W + ox;
                                if (a.out_dtype == VD_BF16) ((__nv_bfloat16*)a.y)[o] = __float2bfloat16_rn(v);
                                else ((float*)a.y)[o] = v;
                            }
                        }
                    }
                } else {
                    constexpr int NCB = BN / 16;                  // 16 accumulator columns at a time
                    const float4* rp = a.residual ? (const float4*)(a.residual + opix * a.Cout + it.n0) : nullptr;
                    float4 res[4];
                    if (rp && inside) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) res[q] = __ldg(rp + q);
                    }
#pragma unroll 1
                    for (int cb = 0; cb < NCB; ++cb) {
                        uint32_t r[16];
                        tmem_ld16(tacc + (uint32_t)(cb * 16), r);
                        tmem_ld_wait();
                        if (last_tile && cb == NCB - 1) {         // accumulators fully read: hand them back to the MMA warp
                            tc_fence_before();
                            mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                        }
                        if (inside) {
                            const int co = it.n0 + cb * 16;
                            float v[16];
#pragma unroll
                            for (int q = 0; q < 16; ++q) v[q] = __uint_as_float(r[q]);
                            if (a.bias) {
#pragma unroll
                                for (int q = 0; q < 16; q += 4) {
                                    const float4 tb = __ldg((const float4*)(a.bias + co + q));
                                    v[q] += tb.x; v[q + 1] += tb.y; v[q + 2] += tb.z; v[q + 3] += tb.w;
                                }
                            }
                            if (a.bias2) {
#pragma unroll
                                for (int q = 0; q < 16; q += 4) {
                                    const float4 tb = __ldg((const float4*)(a.bias2 + co + q));
                                    v[q] += tb.x; v[q + 1] += tb.y; v[q + 2] += tb.z; v[q + 3] += tb.w;
                                }
                            }
                            if (rp) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    v[4 * q] += res[q].x; v[4 * q + 1] += res[q].y; v[4 * q + 2] += res[q].z; v[4 * q + 3] += res[q].w;
                                }
                                if (cb + 1 < NCB) {               // prefetch the next column block's residual
#pragma unroll
                                    for (int q = 0; q < 4; ++q) res[q] = __ldg(rp + (cb + 1) * 4 + q);
                                }
                            }
                            if (OUT_MODE == 1) {
                                uint4* yp = (uint4*)((__nv_bfloat16*)a.y + opix * a.Cout + co);
#pragma unroll
                                for (int q = 0; q < 16; q += 8)
                                    yp[q >> 3] = make_uint4(pack_bf16(v[q], v[q + 1]), pack_bf16(v[q + 2], v[q + 3]),
                                                            pack_bf16(v[q + 4], v[q + 5]), pack_bf16(v[q + 6], v[q + 7]));
                            } else {
                                float4* yp = (float4*)((float*)a.y + opix * a.Cout + co);
#pragma unroll
                                for (int q = 0; q < 16; q += 4) yp[q >> 2] = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                            }
                        }
                    }
                }
            }
        }
    } else if (warp == TMA_WARP) {
        // ------------------------------------------------ weight loads (TMA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < sched.total && ok; w += gridDim.x) {
                const Item it = sched.get(w, BN, Cfg::SUPER_W);
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    for (int tap = 0; tap < ntap; ++tap) {
                        ok = mbar_wait(smem_u32(&bars->b_empty[stage]), phase ^ 1, abort_flag);
                        if (!ok) break;
                        const uint32_t full = smem_u32(&bars->b_full[stage]);
                        mbar_arrive_expect_tx(full, Cfg::B_STAGE_BYTES);
                        if (second) tma_load_2d(smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES), &tmap2, (kc - kchunks) * 64, it.n0, full);
                        else tma_load_2d(smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES), &tmap, kc * 64, tap * cout_pad + it.n0, full);
                        ++issued;
                        if (++stage == Cfg::B_STAGES) { stage = 0; phase ^= 1; }
                    }
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
            int n_item = 0;
            for (int w = blockIdx.x; w < sched.total && ok; w += gridDim.x, ++n_item) {
                const int buf = n_item & 1;
                ok = mbar_wait(smem_u32(&bars->acc_empty[buf]), ((n_item >> 1) & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * MT * Cfg::ACC_COLS);
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    ok = mbar_wait(smem_u32(&bars->a_full[as]), aph, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_stage = smem_u32(smem_a + as * A_STAGE_BYTES);
                    for (int tap = 0; tap < ntap; ++tap) {
                        ok = mbar_wait(smem_u32(&bars->b_full[bs]), bph, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const bool centre = second || a.ksize == 1;
                        const int ky = centre ? 1 : tap / 3, kx = centre ? 1 : tap - 3 * (tap / 3);
                        const uint32_t b_stage = smem_u32(smem_b + bs * Cfg::B_STAGE_BYTES);
#pragma unroll
                        for (int t = 0; t < MT; ++t) {
                            const uint32_t a_tap = a_stage + (uint32_t)(ky * PW + kx + t * TILE_W) * 16;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint64_t adesc = make_smem_desc(a_tap + (uint32_t)(2 * k) * PLANE, PLANE, PW * 16, 0);
                                const uint64_t bdesc = make_smem_desc(b_stage + (uint32_t)k * 32, 16, 1024, 2);
                                umma_bf16(tmem_d + (uint32_t)(t * Cfg::ACC_COLS), adesc, bdesc, idesc, (kc | tap | k) != 0);
                            }
                        }
                        umma_commit(smem_u32(&bars->b_empty[bs]));
                        if (++bs == Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                    }
                    umma_commit(smem_u32(&bars->a_empty[as]));
                    if (++as == Cfg::A_STAGES) { as = 0; aph ^= 1; }
                }
                if (ok) umma_commit(smem_u32(&bars->acc_full[buf]));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && bars->abort_flag && status) {
        if (atomicCAS(status, 0u, 0xC0DE0001u) == 0u) {
            status[1] = blockIdx.x;
            status[2] = (uint32_t)BN;
        }
    }
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)Cfg::TMEM_COLS);
    }
}

// pack OIHW -> bf16 [tap][cout_pad][Cin]
template <typename T>
__global__ void pack_weight_tc_kernel(const T* w, __nv_bfloat16* packed, int Cout, int Cin, int taps, int cout_pad, int cout_offset) {
    const int64_t total = (int64_t)Cout * Cin * taps;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int tap = (int)(i % taps);
        const int c = (int)((i / taps) % Cin);
        const int o = (int)(i / ((int64_t)taps * Cin));
        float v;
        if (sizeof(T) == 2) v = __bfloat162float(((const __nv_bfloat16*)w)[i]);
        else v = ((const float*)w)[i];
        packed[((size_t)tap * cout_pad + cout_offset + o) * Cin + c] = __float2bfloat16_rn(v);
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

int padded_cout(int Cout) { return (Cout % 128 == 0) ? Cout : 16; }
int pick_bn(int Cout) { return (Cout % 128 != 0) ? 16 : ((Cout % 256 == 0) ? 256 : 128); }

bool encode_weights(CUtensorMap* tm, const void* w, int Cin, int rows, int bn) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)Cin, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)Cin * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)bn};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int num_sms() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

template <int BN, bool IB, int OM>
cudaError_t launch_one(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    auto kern = conv_tc_kernel<BN, IB, OM>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<BN>::SMEM_TOTAL);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int tiles = ((a.W + TileCfg<BN>::SUPER_W - 1) / TileCfg<BN>::SUPER_W) * ((a.H + TILE_H - 1) / TILE_H);
    const long long total = (long long)tiles * (padded_cout(a.Cout) / BN) * a.B;
    const int grid = (int)std::min<long long>(total, num_sms());
    kern<<<grid, NUM_THREADS, TileCfg<BN>::SMEM_TOTAL, s>>>(a, *(const CUtensorMap*)plan.tmap, *(const CUtensorMap*)plan.tmap2, status);
    return cudaGetLastError();
}

}  // namespace

bool conv_tc_supported(const ConvArgs& a) {
    if (a.Cin % 64 != 0 || a.Cin < 64) return false;
    if (!a.bf16_operands) return false;
    if (a.ksize != 1 && a.ksize != 3) return false;
    if (a.x2 && (a.Cin2 % 64 != 0 || a.Cin2 < 64)) return false;
    if (a.Cout % 128 == 0) return !a.out_nchw;
    return a.Cout <= 16 && a.out_nchw && !a.residual && !a.x2;      // the frame head: Cout padded to 16
}

size_t conv_tc_packed_bytes(int Cout, int Cin, int taps) { return (size_t)taps * padded_cout(Cout) * Cin * 2; }

cudaError_t launch_pack_weight_tc(const void* w, int w_dtype, void* packed, int Cout, int Cin, int taps, int cout_total,
                                  int cout_offset, cudaStream_t s) {
    const int cpad = padded_cout(cout_total);
    if (cpad != cout_total && cout_offset == 0) {
        cudaError_t e = cudaMemsetAsync(packed, 0, (size_t)taps * cpad * Cin * 2, s);
        if (e != cudaSuccess) return e;
    }
    const int64_t n = (int64_t)Cout * Cin * taps;
    int grid = (int)((n + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    if (w_dtype == VD_BF16)
        pack_weight_tc_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)packed, Cout, Cin, taps, cpad, cout_offset);
    else
        pack_weight_tc_kernel<float><<<grid, 256, 0, s>>>((const float*)w, (__nv_bfloat16*)packed, Cout, Cin, taps, cpad, cout_offset);
    return cudaGetLastError();
}

cudaError_t conv_tc_prepare(const ConvArgs& a, ConvTcPlan* plan) {
    const int taps = a.ksize * a.ksize;
    const int bn = pick_bn(a.Cout);
    if (!encode_weights((CUtensorMap*)plan->tmap, a.w, a.Cin, taps * padded_cout(a.Cout), bn)) return cudaErrorInvalidValue;
    if (a.x2) {
        if (!encode_weights((CUtensorMap*)plan->tmap2, a.w2, a.Cin2, a.Cout, bn)) return cudaErrorInvalidValue;
    } else {
        memcpy(plan->tmap2, plan->tmap, sizeof(plan->tmap));
    }
    plan->bn = bn;
    plan->valid = 1;
    return cudaSuccess;
}

cudaError_t launch_conv_tc(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    if (!plan.valid) return cudaErrorInvalidValue;
    const bool ib = a.in_dtype == VD_BF16, ob = a.out_dtype == VD_BF16;
    if (plan.bn == 16) {
        return ib ? launch_one<16, true, 2>(a, plan, status, s) : launch_one<16, false, 2>(a, plan, status, s);
    }
    if (plan.bn == 256) {
        if (ib && ob) return launch_one<256, true, 1>(a, plan, status, s);
        if (ib && !ob) return launch_one<256, true, 0>(a, plan, status, s);
        if (!ib && ob) return launch_one<256, false, 1>(a, plan, status, s);
        return launch_one<256, false, 0>(a, plan, status, s);
    }
    if (ib && ob) return launch_one<128, true, 1>(a, plan, status, s);
    if (ib && !ob) return launch_one<128, true, 0>(a, plan, status, s);
    if (!ib && ob) return launch_one<128, false, 1>(a, plan, status, s);
    return launch_one<128, false, 0>(a, plan, status, s);
}

}  // namespace vd
