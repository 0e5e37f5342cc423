// Implicit-GEMM 3x3 / 1x1 convolution on the 5th-generation tensor cores (tcgen05 + TMEM), with
// the paper's fusion folded around it (Section IV-B.1, Eq. 9): the GroupNorm-apply + SiLU of the
// chain runs in the operand prologue, nearest-2x upsampling is an address computation, and bias,
// residual add, the 1x1 shortcut and the output cast run in / next to the same accumulation, so
// each activation crosses HBM once.
//
// Persistent kernel, one CTA per SM, roles decoupled through mbarrier rings:
//   * tile = 16x8 output pixels x BN output channels:  D[128 x BN] = sum over taps and 64-channel
//     chunks of A_tap[128 x 64] * W_tap[64 x BN].  Every CTA owns a contiguous, balanced range of
//     tiles and walks it in work items of two tiles that share every weight stage.
//   * 15 producer warps read the raw 18x10-pixel halo tile of a 64-channel chunk from global
//     memory once, apply
//     scale/shift (+SiLU), round to bf16 and store it in shared memory in the canonical
//     un-swizzled K-major layout, as eight planes [8 channels][pixel][16 B].  Every tap is a *view*
//     of that one tile (descriptor start (ky*10+kx) pixels in; eight-row groups are one tile row
//     = 10 pixels apart), so the transform runs once per element, not once per tap.
//     Out-of-image halo pixels are exact zeros (padding applies to the transformed tensor).
//     An optional second input (the block's raw input for a width-changing ResNet block) is
//     appended as extra K with a single centre tap: the 1x1 shortcut without its own round trip.
//   * 1 warp streams the weights (bf16 [tap][Cout][Cin]) by TMA into 128B-swizzled stages.
//   * 1 thread issues tcgen05.mma (M=128, N=BN, K=16) into TMEM accumulators (double-buffered
//     where 4 x BN columns fit).
//   * 4 epilogue warps drain the accumulators: tcgen05.ld, + bias, and the tile leaves through
//     shared memory as 128-byte-wide slices written by bulk tensor stores, which coalesce the
//     traffic and clip the ragged image edge.  Where the layer has a residual, the output buffer
//     IS the residual stream and the store is a bulk tensor reduce-add (the fp32 add x + conv(h)
//     is done once, by the memory system), so the residual never passes through the SM.
//     The 3-channel frame head writes its NCHW planes directly.
// Every wait is bounded: on expiry the CTA records a code in the status word and unwinds.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>

#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;

constexpr int TILE_H = 16, TILE_W = 8;                               // one MMA tile: 128 output pixels
constexpr int PH = TILE_H + 2, PW = TILE_W + 2, NPIX = PH * PW;     // 18 x 10 = 180 halo pixels
constexpr int A_TILE_BYTES = (NPIX * 128 + 1023) / 1024 * 1024;      // one 64-channel chunk of one halo tile: 180 rows of 128 B
constexpr int ITEMS = NPIX * 8;                                      // (pixel, 8-channel group) pairs per tile chunk
constexpr int NUM_PRODUCER_WARPS = 15;
constexpr int NUM_PRODUCERS = NUM_PRODUCER_WARPS * 32;               // 480 = ITEMS / 3: three pairs per thread
constexpr int BATCH = ITEMS / NUM_PRODUCERS;                         // 3
static_assert(BATCH * NUM_PRODUCERS == ITEMS, "producer threads must tile the halo chunk exactly");
constexpr int TMA_WARP = 15;
constexpr int EPI_WARP0 = 16;                                        // warps 16-19 (warp % 4 = TMEM lane quarter)
constexpr int MMA_WARP = 20;
constexpr int NUM_THREADS = 21 * 32;
constexpr int MAX_B_STAGES = 8, MAX_A_STAGES = 4;
constexpr int STAT_MAX_GROUPS = 64;                                  // GroupNorm groups the fused statistics can hold
constexpr int OUT_SLICE_BYTES = 128 * 128;                           // 128 pixels x 128 B: one output slice in smem

// BN = output channels per work item.  Where the channel block is narrow (BN <= 128) a work
// item is two 16x8-pixel tiles whose MMAs consume every weight stage together, which halves the
// weight traffic through shared memory and the bytes the TMA pipeline must keep in flight.
template <int BN> struct TileCfg {
    static constexpr int PAIR = BN == 256 ? 1 : 2;                   // tiles per work item
    static constexpr int B_STAGE_BYTES = BN * 128;                   // BN rows x 64 bf16
    static constexpr int B_STAGES = BN == 256 ? 4 : (BN == 128 ? 5 : 8);
    static constexpr int A_STAGES = 2;
    static constexpr int A_STAGE_BYTES = PAIR * A_TILE_BYTES;
    static constexpr int SMEM_B = (B_STAGES * B_STAGE_BYTES + 1023) / 1024 * 1024;
    static constexpr int SMEM_OUT = BN >= 128 ? 3 * OUT_SLICE_BYTES : 0;   // rotating output / residual slices
    static constexpr int SMEM_A = A_STAGES * A_STAGE_BYTES;
    static constexpr int SMEM_TOTAL = SMEM_B + SMEM_OUT + SMEM_A + 512 + 2048 + 1024;  // + barriers + statistics + alignment slack
    static constexpr int ACC_COLS = BN < 32 ? 32 : BN;               // TMEM columns per accumulator
    static constexpr int NBUF = 2;                                   // accumulator sets (PAIR tiles each)
    static constexpr int TMEM_COLS = NBUF * PAIR * ACC_COLS;
};

struct Raw8 { uint4 lo, hi; };   // eight channels of one pixel: bf16 -> lo only; fp32 -> lo + hi

// bf16: the thread's 16 bytes are channels [8j, 8j+8) of the chunk.  fp32: two 16-byte loads,
// channels [4j, 4j+4) and [32+4j, 32+4j+4), so that the eight threads of a pixel read two
// contiguous 128-byte lines.
__device__ __forceinline__ void load_raw(bool is_bf16, const void* x, size_t pix_off, int c0, int j, Raw8& r) {
    if (is_bf16) {
        r.lo = __ldg((const uint4*)((const __nv_bfloat16*)x + pix_off + c0 + j * 8));
    } else {
        const float* p = (const float*)x + pix_off + c0 + j * 4;
        const float4 a = __ldg((const float4*)p), b = __ldg((const float4*)(p + 32));
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

// Per-group sum and sum of squares of 32 consecutive channels (registers v[32]) of the 32 pixels
// a warp holds, added to the warp's accumulators in shared memory ([2][STAT_MAX_GROUPS]: sums,
// then sums of squares).  The 2*32/CPG lane-local values are reduced across the warp with a
// halving butterfly (a fixed order, so the result is reproducible).
template <int CPG>
__device__ __forceinline__ void warp_group_stats(const float (&v)[32], bool inside, int lane, float* wacc, int g0) {
    constexpr int NG = 32 / CPG, NV = 2 * NG;
    float vals[NV];
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        float s = 0.f, q = 0.f;
#pragma unroll
        for (int e = 0; e < CPG; ++e) {
            const float x = v[g * CPG + e];
            s += x;
            q = fmaf(x, x, q);
        }
        vals[g] = inside ? s : 0.f;
        vals[NG + g] = inside ? q : 0.f;
    }
    // after the step with lane mask M a lane keeps the half of the values selected by its bit M
    int idx = 0;
#pragma unroll
    for (int half = NV / 2, mask = 16; half >= 1; half >>= 1, mask >>= 1) {
        const bool upper = (lane & mask) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float send = upper ? vals[i] : vals[i + half];
            const float keep = upper ? vals[i + half] : vals[i];
            vals[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
        }
        idx += upper ? half : 0;
    }
    // NV values took log2(NV) steps; the remaining lane bits still hold partial sums of the same value
    constexpr int STEPS = NV == 16 ? 4 : (NV == 8 ? 3 : 2);
#pragma unroll
    for (int mask = 16 >> STEPS; mask >= 1; mask >>= 1) vals[0] += __shfl_xor_sync(0xffffffffu, vals[0], mask);
    if ((lane & ((32 >> STEPS) - 1)) == 0) {
        const int stat = idx / NG, g = idx - stat * NG;
        wacc[stat * STAT_MAX_GROUPS + g0 + g] += vals[0];
    }
}

struct Bars {                    // lives in shared memory
    uint64_t a_full[MAX_A_STAGES], a_empty[MAX_A_STAGES];
    uint64_t b_full[MAX_B_STAGES], b_empty[MAX_B_STAGES];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t epi_sync;           // rendezvous of the 128 epilogue threads (a bounded stand-in for bar.sync)
    uint64_t res_full[3];        // residual slice has landed in output buffer i
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t is_last;
};

struct Tile { int tx0, ty0, n0, b; };

// Debug timeline: role r of this CTA appends (code << 48 | clock) records when a trace buffer is given.
struct Tracer {
    unsigned long long* p;
    int n;
    __device__ __forceinline__ void init(unsigned long long* base, int role) {
        p = base ? base + ((size_t)blockIdx.x * 4 + role) * kConvTraceEvents : nullptr;
        n = 0;
    }
    __device__ __forceinline__ void mark(unsigned code) {
        if (p && n < kConvTraceEvents) p[n++] = ((unsigned long long)code << 48) | ((unsigned long long)clock64() & 0xFFFFFFFFFFFFull);
    }
};

// Tiles are numbered (frame, channel block, tile row, tile column), column fastest.  Every CTA
// owns a contiguous, balanced range of tile numbers and walks it in items of `pair` tiles (one
// when the range or the channel block ends).
struct Sched {
    int tiles_x, tiles, nblk, total;
    int begin, end, pair;
    __device__ __forceinline__ Tile get(int t, int bn) const {
        Tile r;
        const int blk = t / tiles;               // frame * nblk + channel block
        const int s = t - blk * tiles;
        r.b = blk / nblk;
        r.n0 = (blk - r.b * nblk) * bn;
        r.ty0 = (s / tiles_x) * TILE_H;
        r.tx0 = (s % tiles_x) * TILE_W;
        return r;
    }
    // number of tiles of the item that starts at tile t
    __device__ __forceinline__ int count(int t) const {
        return (pair == 2 && t + 1 < end && (t + 1) / tiles == t / tiles) ? 2 : 1;
    }
};

// OUT_MODE: 0 = fp32 NHWC, 1 = bf16 NHWC (both through shared memory and TMA stores),
//           2 = NCHW frame written directly (dtype from a.out_dtype)
template <int BN, bool IN_BF16, int OUT_MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_tc_kernel(const ConvArgs a, const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap2,
               const __grid_constant__ CUtensorMap tmap_y, unsigned int* status) {
    using Cfg = TileCfg<BN>;
    constexpr int NBUF = Cfg::NBUF, PAIR = Cfg::PAIR, A_STAGE_BYTES = Cfg::A_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;
    uint8_t* smem_out = smem + Cfg::SMEM_B;
    uint8_t* smem_a = smem_out + Cfg::SMEM_OUT;
    Bars* bars = (Bars*)(smem_a + Cfg::SMEM_A);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int taps = a.ksize * a.ksize;
    const int kchunks = a.Cin >> 6;
    const int kchunks2 = a.x2 ? (a.Cin2 >> 6) : 0;          // extra K: 1x1 shortcut on a second input
    const int ktotal = kchunks + kchunks2;
    const int cout_pad = (a.Cout % 128 == 0) ? a.Cout : 16; // rows per tap in the packed weights
    Sched sched;
    sched.tiles_x = (a.W + TILE_W - 1) / TILE_W;
    sched.tiles = sched.tiles_x * ((a.H + TILE_H - 1) / TILE_H);
    sched.nblk = cout_pad / BN;
    sched.total = sched.tiles * sched.nblk * a.B;
    sched.begin = (int)(((long long)sched.total * blockIdx.x) / gridDim.x);
    sched.end = (int)(((long long)sched.total * (blockIdx.x + 1)) / gridDim.x);
    sched.pair = PAIR;

    if (tid == 0) {
        for (int i = 0; i < Cfg::A_STAGES; ++i) { mbar_init(smem_u32(&bars->a_full[i]), NUM_PRODUCER_WARPS); mbar_init(smem_u32(&bars->a_empty[i]), 1); }
        for (int i = 0; i < Cfg::B_STAGES; ++i) { mbar_init(smem_u32(&bars->b_full[i]), 1); mbar_init(smem_u32(&bars->b_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bars->acc_full[i]), 1); mbar_init(smem_u32(&bars->acc_empty[i]), 4); }
        mbar_init(smem_u32(&bars->epi_sync), 128);
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&bars->res_full[i]), 1);
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
        // The work is a flat sequence of units (item, chunk, tile slot); a unit's loads (three
        // 8-channel groups per thread, 480 threads) are all in flight before any is consumed.
        const int j = tid & 7;                              // this thread's channel group within a chunk
        const bool prologue = a.scale != nullptr;
        const bool silu = a.silu != 0;
        const int up = a.upsample ? 1 : 0;
        struct Pos { int t, cnt, kc, slot; Tile tile; };
        auto advance = [&](Pos& p) {
            if (++p.slot == p.cnt) {
                p.slot = 0;
                if (++p.kc == ktotal) {
                    p.kc = 0;
                    p.t += p.cnt;
                    if (p.t < sched.end) p.cnt = sched.count(p.t);
                }
            }
            if (p.t < sched.end) p.tile = sched.get(p.t + p.slot, BN);
        };
        Tracer tr; tr.init(tid == 0 ? a.trace : nullptr, 0);
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        Pos cur;
        cur.t = sched.begin; cur.kc = 0; cur.slot = 0; cur.cnt = 1;
        if (cur.t < sched.end) { cur.cnt = sched.count(cur.t); cur.tile = sched.get(cur.t, BN); }
        while (cur.t < sched.end && ok) {
            const bool second = cur.kc >= kchunks;
            const bool in_bf16 = second ? false : IN_BF16;
            const int c0 = (second ? cur.kc - kchunks : cur.kc) * 64;
            const bool centre_only = second || a.ksize == 1;
            tr.mark(1);
            Raw8 raw[BATCH];
            uint32_t vm = 0;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int pix = (u * NUM_PRODUCERS + tid) >> 3;
                const int py = pix / PW, px = pix - py * PW;
                const int oy = cur.tile.ty0 + py - 1, ox = cur.tile.tx0 + px - 1;
                bool v = oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                if (centre_only) v = v && py >= 1 && py <= TILE_H && px >= 1 && px <= TILE_W;
                if (v) {
                    vm |= 1u << u;
                    if (second) load_raw(false, a.x2, (((size_t)cur.tile.b * a.H + oy) * a.W + ox) * a.Cin2, c0, j, raw[u]);
                    else load_raw(IN_BF16, a.x, (((size_t)cur.tile.b * a.Hs + (oy >> up)) * a.Ws + (ox >> up)) * a.Cin, c0, j, raw[u]);
                }
            }
            const bool pro = prologue && !second;
            float sc[8], sh[8];
            if (pro) {
                // channels of v[0..3] and v[4..7] (see load_raw)
                const int ca = c0 + (in_bf16 ? j * 8 : j * 4), cb = in_bf16 ? ca + 4 : ca + 32;
                const float* ps = a.scale + (size_t)cur.tile.b * a.Cin;
                const float* pt = a.shift + (size_t)cur.tile.b * a.Cin;
                const float4 s0 = __ldg((const float4*)(ps + ca)), s1 = __ldg((const float4*)(ps + cb));
                const float4 t0 = __ldg((const float4*)(pt + ca)), t1 = __ldg((const float4*)(pt + cb));
                sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
            }
            if (cur.slot == 0) {
                ok = mbar_wait(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
                if (!ok) break;
            }
            tr.mark(2);
            uint8_t* dst_tile = smem_a + stage * A_STAGE_BYTES + cur.slot * A_TILE_BYTES;
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                uint32_t o0 = 0u, o1 = 0u, o2 = 0u, o3 = 0u;
                if (vm & (1u << u)) {
                    float v[8];
                    unpack_raw(in_bf16, raw[u], v);
                    if (pro) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], sc[e], sh[e]);
                        if (silu) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = silu_fast(v[e]);
                        }
                    }
                    o0 = pack_bf16(v[0], v[1]); o1 = pack_bf16(v[2], v[3]); o2 = pack_bf16(v[4], v[5]); o3 = pack_bf16(v[6], v[7]);
                }
                // row = halo pixel (128 B = 64 channels), 16-byte chunk c stored at c ^ (row & 7): the
                // 128-byte swizzle of the K-major operand layout (tile bases are 1024-byte aligned)
                const int pix = (u * NUM_PRODUCERS + tid) >> 3;
                uint8_t* prow = dst_tile + pix * 128;
                if (in_bf16) {
                    *(uint4*)(prow + ((j ^ (pix & 7)) << 4)) = make_uint4(o0, o1, o2, o3);
                } else {     // channels 4j..4j+3 -> chunk j/2, half j&1; channels 32+4j.. -> chunk 4 + j/2
                    const int c = j >> 1, hb = (j & 1) * 8;
                    *(uint2*)(prow + ((c ^ (pix & 7)) << 4) + hb) = make_uint2(o0, o1);
                    *(uint2*)(prow + (((c + 4) ^ (pix & 7)) << 4) + hb) = make_uint2(o2, o3);
                }
            }
            if (cur.slot == cur.cnt - 1) {
                fence_proxy_async_smem();                    // generic-proxy stores -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->a_full[stage]));
                if (++stage == Cfg::A_STAGES) { stage = 0; phase ^= 1; }
            }
            tr.mark(3);
            advance(cur);
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------ epilogue
        const int ew = warp - EPI_WARP0;                     // TMEM lane quarter
        const int m = ew * 32 + lane;                        // accumulator row = pixel of the MMA tile
        const int et = tid - EPI_WARP0 * 32;                 // 0..127
        const bool leader = et == 0;                         // issues the bulk loads / stores
        const bool want_stats = OUT_MODE != 2 && a.stat_partial != nullptr;
        // y holds the residual stream.  Plain case: the tile is added into it by a bulk reduce-add (the
        // residual never enters the SM).  With fused statistics the final values are needed on chip,
        // so the residual slice is loaded, added and the sum stored back.
        const bool has_res = a.residual != nullptr && want_stats;
        const bool reduce_add = a.residual != nullptr && !want_stats;
        const int cpg = want_stats ? a.Cout / a.stat_groups : 4;
        float* stat_acc = (float*)(smem + Cfg::SMEM_B + Cfg::SMEM_OUT + Cfg::SMEM_A + sizeof(Bars));   // [4 warps][2][64]
        Tracer tr; tr.init(leader ? a.trace : nullptr, 2);
        bool ok = true;
        int n_item = 0;
        uint32_t n_slice = 0, sync_phase = 0;
        int stat_b = -1;                                     // frame the shared-memory statistics belong to
        auto epi_rendezvous = [&]() {                        // all 128 epilogue threads meet here; bounded like every wait
            mbar_arrive(smem_u32(&bars->epi_sync));
            const bool r = mbar_wait(smem_u32(&bars->epi_sync), sync_phase, abort_flag);
            sync_phase ^= 1;
            return r;
        };
        // moves this CTA's statistics of frame `b` to global memory (one record per CTA and frame)
        auto flush_stats = [&](int b) {
            bool r = epi_rendezvous();
            if (et < 2 * STAT_MAX_GROUPS) {
                float tot = 0.f;
#pragma unroll
                for (int w4 = 0; w4 < 4; ++w4) tot += stat_acc[w4 * 2 * STAT_MAX_GROUPS + et];
                // layout [frame][stat][group][cta]: a warp of the finalising CTA reads 32 CTAs' records at once
                a.stat_partial[(((size_t)b * 2 * STAT_MAX_GROUPS) + et) * gridDim.x + blockIdx.x] = tot;
            }
            r = epi_rendezvous() && r;
            for (int i = et; i < 4 * 2 * STAT_MAX_GROUPS; i += 128) stat_acc[i] = 0.f;
            return epi_rendezvous() && r;
        };
        if (want_stats) {
            for (int i = et; i < 4 * 2 * STAT_MAX_GROUPS; i += 128) stat_acc[i] = 0.f;
            ok = __all_sync(0xffffffffu, epi_rendezvous());
        }
        constexpr int CS = OUT_MODE == 1 ? 64 : 32;          // channels per 128-byte output slice
        constexpr int NS = BN >= CS ? BN / CS : 1;
        // coordinates of the slice after (t, cnt, slot, sidx), for the residual prefetch
        auto next_slice = [&](int t, int cnt, int slot, int sidx, Tile& tl, int& ns) {
            if (sidx + 1 < NS) { tl = sched.get(t + slot, BN); ns = sidx + 1; return true; }
            if (slot + 1 < cnt) { tl = sched.get(t + slot + 1, BN); ns = 0; return true; }
            if (t + cnt < sched.end) { tl = sched.get(t + cnt, BN); ns = 0; return true; }
            return false;
        };
        if (OUT_MODE != 2 && has_res && leader && sched.begin < sched.end) {
            const Tile tl = sched.get(sched.begin, BN);     // first residual slice
            mbar_arrive_expect_tx(smem_u32(&bars->res_full[0]), OUT_SLICE_BYTES);
            tma_load_4d(smem_u32(smem_out), &tmap_y, tl.n0, tl.tx0, tl.ty0, tl.b, smem_u32(&bars->res_full[0]));
        }
        for (int t = sched.begin; t < sched.end && ok; ++n_item) {
            const int cnt = sched.count(t);
            const int buf = n_item % NBUF;
            tr.mark(10);
            ok = mbar_wait(smem_u32(&bars->acc_full[buf]), (n_item / NBUF) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);                // tcgen05.ld below is warp-collective
            if (!ok) break;
            tc_fence_after();
            tr.mark(11);
#pragma unroll 1
            for (int slot = 0; slot < cnt && ok; ++slot) {
                const Tile tl = sched.get(t + slot, BN);
                const uint32_t tacc = tmem_base + (uint32_t)((buf * PAIR + slot) * Cfg::ACC_COLS) + ((uint32_t)(ew * 32) << 16);
                const bool last_tile = slot == cnt - 1;
                const int oy = tl.ty0 + (m >> 3), ox = tl.tx0 + (m & 7);
                const bool inside = oy < a.H && ox < a.W;
                if (OUT_MODE == 2) {
                    uint32_t r[16];
                    tmem_ld16(tacc, r);
                    tmem_ld_wait();
                    if (last_tile) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                    }
                    if (inside) {
#pragma unroll
                        for (int co = 0; co < 16; ++co) {
                            if (co < a.Cout) {
                                const float v = __uint_as_float(r[co]) + (a.bias ? __ldg(a.bias + co) : 0.f);
                                const size_t o = (((size_t)tl.b * a.Cout + co) * a.H + oy) * a.W + ox;
                                if (a.out_dtype == VD_BF16) ((__nv_bfloat16*)a.y)[o] = __float2bfloat16_rn(v);
                                else ((float*)a.y)[o] = v;
                            }
                        }
                    }
                } else {
                    if (want_stats && tl.b != stat_b) {
                        if (stat_b >= 0) ok = __all_sync(0xffffffffu, flush_stats(stat_b));
                        stat_b = tl.b;
                        if (!ok) break;
                    }
                    // The tile leaves through shared memory in 128-byte-wide slices (32 fp32 or 64
                    // bf16 channels), written row-per-thread in the 128B-swizzled layout of a bulk
                    // tensor copy; the copy clips the ragged image edge by itself.  Three slice
                    // buffers rotate: one being stored, one being filled, one receiving the next
                    // slice of the residual stream.
#pragma unroll 1
                    for (int sidx = 0; sidx < NS; ++sidx, ++n_slice) {
                        uint8_t* obuf = smem_out + (n_slice % 3) * OUT_SLICE_BYTES;
                        tr.mark(12);
                        if (leader) {
                            bulk_wait_group_read<1>();                // the store issued two slices ago has drained its buffer
                            Tile ntl;
                            int nsidx;
                            if (has_res && next_slice(t, cnt, slot, sidx, ntl, nsidx)) {
                                const uint32_t nb = (n_slice + 1) % 3;
                                mbar_arrive_expect_tx(smem_u32(&bars->res_full[nb]), OUT_SLICE_BYTES);
                                tma_load_4d(smem_u32(smem_out + nb * OUT_SLICE_BYTES), &tmap_y, ntl.n0 + nsidx * CS, ntl.tx0, ntl.ty0,
                                            ntl.b, smem_u32(&bars->res_full[nb]));
                            }
                        }
                        ok = __all_sync(0xffffffffu, epi_rendezvous());
                        if (!ok) break;
                        if (has_res) {
                            ok = mbar_wait(smem_u32(&bars->res_full[n_slice % 3]), (n_slice / 3) & 1, abort_flag);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                        }
                        tr.mark(13);
                        uint8_t* orow = obuf + m * 128;
#pragma unroll
                        for (int h = 0; h < CS / 32; ++h) {
                            uint32_t r[32];
                            tmem_ld32(tacc + (uint32_t)(sidx * CS + h * 32), r);
                            tmem_ld_wait();
                            if (last_tile && sidx == NS - 1 && h == CS / 32 - 1) {   // accumulators fully read
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                            }
                            const int co = tl.n0 + sidx * CS + h * 32;
                            float v[32];
#pragma unroll
                            for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
                            if (a.bias) {
#pragma unroll
                                for (int q = 0; q < 32; q += 4) {
                                    const float4 tb = __ldg((const float4*)(a.bias + co + q));
                                    v[q] += tb.x; v[q + 1] += tb.y; v[q + 2] += tb.z; v[q + 3] += tb.w;
                                }
                            }
                            if (a.bias2) {
#pragma unroll
                                for (int q = 0; q < 32; q += 4) {
                                    const float4 tb = __ldg((const float4*)(a.bias2 + co + q));
                                    v[q] += tb.x; v[q + 1] += tb.y; v[q + 2] += tb.z; v[q + 3] += tb.w;
                                }
                            }
                            if (OUT_MODE == 0) {
                                if (has_res) {
#pragma unroll
                                    for (int c = 0; c < 8; ++c) {
                                        const float4 x = *(const float4*)(orow + ((c ^ (m & 7)) << 4));
                                        v[4 * c] += x.x; v[4 * c + 1] += x.y; v[4 * c + 2] += x.z; v[4 * c + 3] += x.w;
                                    }
                                }
#pragma unroll
                                for (int c = 0; c < 8; ++c)
                                    *(float4*)(orow + ((c ^ (m & 7)) << 4)) = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                            } else {
#pragma unroll
                                for (int c = 0; c < 4; ++c) {
                                    const uint4 pk = make_uint4(pack_bf16(v[8 * c], v[8 * c + 1]), pack_bf16(v[8 * c + 2], v[8 * c + 3]),
                                                                pack_bf16(v[8 * c + 4], v[8 * c + 5]), pack_bf16(v[8 * c + 6], v[8 * c + 7]));
                                    *(uint4*)(orow + (((h * 4 + c) ^ (m & 7)) << 4)) = pk;
                                    if (want_stats) {         // statistics are those of the values as stored
                                        const uint32_t w4[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                                        for (int e = 0; e < 4; ++e) {
                                            v[8 * c + 2 * e] = __uint_as_float(w4[e] << 16);
                                            v[8 * c + 2 * e + 1] = __uint_as_float(w4[e] & 0xffff0000u);
                                        }
                                    }
                                }
                            }
                            if (want_stats) {
                                float* wacc = stat_acc + ew * 2 * STAT_MAX_GROUPS;
                                const int g0 = co / cpg;          // first group of these 32 channels
                                if (cpg == 4) warp_group_stats<4>(v, inside, lane, wacc, g0);
                                else if (cpg == 8) warp_group_stats<8>(v, inside, lane, wacc, g0);
                                else warp_group_stats<16>(v, inside, lane, wacc, g0);
                            }
                        }
                        tr.mark(14);
                        fence_proxy_async_smem();
                        ok = __all_sync(0xffffffffu, epi_rendezvous());
                        if (!ok) break;
                        tr.mark(15);
                        if (leader) {
                            if (reduce_add) tma_reduce_add_4d(&tmap_y, smem_u32(obuf), tl.n0 + sidx * CS, tl.tx0, tl.ty0, tl.b);
                            else tma_store_4d(&tmap_y, smem_u32(obuf), tl.n0 + sidx * CS, tl.tx0, tl.ty0, tl.b);
                            bulk_commit_group();
                        }
                    }
                }
            }
            t += cnt;
        }
        if (leader) bulk_wait_group<0>();                    // all stores have landed before the CTA retires
        if (want_stats && ok) {
            if (stat_b >= 0) ok = __all_sync(0xffffffffu, flush_stats(stat_b));
            // The CTA that finishes last turns the per-CTA records into the next layer's per-(frame,
            // channel) scale and shift: scale = gamma * rstd, shift = beta - mean * scale.
            if (ok) {
                if (leader) {
                    __threadfence();
                    const unsigned int prev = atomicAdd(a.stat_counter, 1u);
                    bars->is_last = (prev == gridDim.x - 1) ? 1u : 0u;
                }
                ok = __all_sync(0xffffffffu, epi_rendezvous());
            }
            if (ok && bars->is_last) {
                __threadfence();
                const int G = a.stat_groups;
                const int tiles_per_frame = sched.tiles * sched.nblk;
                const double count = (double)a.H * a.W * cpg;
                for (int row = ew; row < a.B * G; row += 4) {       // one (frame, group) per warp at a time
                    const int b = row / G, g = row - b * G;
                    // CTAs whose tile range meets this frame wrote a record; sum them in a fixed order
                    double s = 0.0, q = 0.0;
                    for (int c = lane; c < (int)gridDim.x; c += 32) {
                        const long long cb = ((long long)sched.total * c) / gridDim.x, ce = ((long long)sched.total * (c + 1)) / gridDim.x;
                        if (ce > (long long)b * tiles_per_frame && cb < (long long)(b + 1) * tiles_per_frame) {
                            s += (double)__ldcg(a.stat_partial + (((size_t)b * 2 * STAT_MAX_GROUPS) + g) * gridDim.x + c);
                            q += (double)__ldcg(a.stat_partial + (((size_t)b * 2 * STAT_MAX_GROUPS) + STAT_MAX_GROUPS + g) * gridDim.x + c);
                        }
                    }
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) {
                        s += __shfl_xor_sync(0xffffffffu, s, d);
                        q += __shfl_xor_sync(0xffffffffu, q, d);
                    }
                    const double mean = s / count;
                    const double var = fmax(q / count - mean * mean, 0.0);
                    const float rstd = (float)(1.0 / sqrt(var + (double)a.stat_eps));
                    for (int cc = lane; cc < cpg; cc += 32) {
                        const int ch = g * cpg + cc;
                        const float sc = a.stat_gamma[ch] * rstd;
                        a.stat_scale[(size_t)b * a.Cout + ch] = sc;
                        a.stat_shift[(size_t)b * a.Cout + ch] = a.stat_beta[ch] - (float)mean * sc;
                    }
                }
                if (leader) *a.stat_counter = 0u;            // ready for the next launch
            }
        }
    } else if (warp == TMA_WARP) {
        // ------------------------------------------------ weight loads (TMA)
        if (lane == 0) {
            Tracer tr; tr.init(a.trace, 3);
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int t = sched.begin; t < sched.end && ok; t += sched.count(t)) {
                const Tile tl = sched.get(t, BN);
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    for (int tap = 0; tap < ntap; ++tap) {
                        tr.mark(30);
                        ok = mbar_wait(smem_u32(&bars->b_empty[stage]), phase ^ 1, abort_flag);
                        if (!ok) break;
                        tr.mark(31);
                        const uint32_t full = smem_u32(&bars->b_full[stage]);
                        mbar_arrive_expect_tx(full, Cfg::B_STAGE_BYTES);
                        if (second) tma_load_2d(smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES), &tmap2, (kc - kchunks) * 64, tl.n0, full);
                        else tma_load_2d(smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES), &tmap, kc * 64, tap * cout_pad + tl.n0, full);
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
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------ MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, BN);
            const uint32_t a_hi = desc_hi(PW * 128, 2), b_hi = desc_hi(1024, 2);
            const uint32_t a_lo0 = desc_lo(smem_u32(smem_a)), b_lo0 = desc_lo(smem_u32(smem_b));
            Tracer tr; tr.init(a.trace, 1);
            uint32_t as = 0, aph = 0, bs = 0, bph = 0;
            bool ok = true;
            int n_item = 0;
            for (int t = sched.begin; t < sched.end && ok; ++n_item) {
                const int cnt = sched.count(t);
                const int buf = n_item % NBUF;
                tr.mark(20);
                ok = mbar_wait(smem_u32(&bars->acc_empty[buf]), ((n_item / NBUF) & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                tr.mark(21);
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * PAIR * Cfg::ACC_COLS);
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    tr.mark(22);
                    ok = mbar_wait(smem_u32(&bars->a_full[as]), aph, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    tr.mark(23);
                    for (int tap = 0; tap < ntap; ++tap) {
                        tr.mark(25);
                        ok = mbar_wait(smem_u32(&bars->b_full[bs]), bph, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        tr.mark(24);
                        // tap view: rows start (ky*PW + kx) pixels into the halo tile; eight-row groups are
                        // one tile row (PW pixels) apart.  The tensor core applies the 128-byte swizzle to the
                        // absolute shared-memory address, so any 128-byte-aligned start works (base_offset 0).
                        const bool centre = second || a.ksize == 1;
                        const int ky = centre ? 1 : tap / 3, kx = centre ? 1 : tap - 3 * (tap / 3);
                        const uint32_t b_lo = b_lo0 + bs * (Cfg::B_STAGE_BYTES >> 4);
                        uint32_t a_lo = a_lo0 + as * (A_STAGE_BYTES >> 4) + (uint32_t)(ky * PW + kx) * 8;
                        uint32_t acc = (kc | tap) != 0;
                        uint32_t td = tmem_d;
                        for (int slot = 0; slot < cnt; ++slot) {
                            umma_bf16_split(td, a_lo, a_hi, b_lo, b_hi, idesc, acc);
                            umma_bf16_split(td, a_lo + 2, a_hi, b_lo + 2, b_hi, idesc, 1u);
                            umma_bf16_split(td, a_lo + 4, a_hi, b_lo + 4, b_hi, idesc, 1u);
                            umma_bf16_split(td, a_lo + 6, a_hi, b_lo + 6, b_hi, idesc, 1u);
                            a_lo += A_TILE_BYTES >> 4;
                            td += Cfg::ACC_COLS;
                        }
                        umma_commit(smem_u32(&bars->b_empty[bs]));
                        if (++bs == Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                    }
                    umma_commit(smem_u32(&bars->a_empty[as]));
                    if (++as == Cfg::A_STAGES) { as = 0; aph ^= 1; }
                }
                if (ok) umma_commit(smem_u32(&bars->acc_full[buf]));
                t += cnt;
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
    const int tiles = ((a.W + TILE_W - 1) / TILE_W) * ((a.H + TILE_H - 1) / TILE_H);
    const long long total = (long long)tiles * (padded_cout(a.Cout) / BN) * a.B;
    int grid = (int)std::min<long long>(total, std::min(num_sms(), kConvStatMaxCtas));
    if (getenv("VD_CONV_GRID")) grid = std::min(grid, atoi(getenv("VD_CONV_GRID")));   // timing studies
    kern<<<grid, NUM_THREADS, TileCfg<BN>::SMEM_TOTAL, s>>>(a, *(const CUtensorMap*)plan.tmap, *(const CUtensorMap*)plan.tmap2,
                                                            *(const CUtensorMap*)plan.tmap_y, status);
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
    if (!a.out_nchw) {
        // output [B][H][W][Cout] as a 4-D tensor (channels innermost); a box is one 128-byte-wide slice of a tile
        EncodeTiledFn enc = get_encode_fn();
        if (!enc) return cudaErrorNotSupported;
        const bool ob = a.out_dtype == VD_BF16;
        const cuuint64_t es = ob ? 2 : 4;
        const cuuint64_t dims[4] = {(cuuint64_t)a.Cout, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)std::max(a.B, 1)};
        const cuuint64_t strides[3] = {(cuuint64_t)a.Cout * es, (cuuint64_t)a.W * a.Cout * es, (cuuint64_t)a.H * a.W * a.Cout * es};
        const cuuint32_t box[4] = {ob ? 64u : 32u, (cuuint32_t)TILE_W, (cuuint32_t)TILE_H, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc((CUtensorMap*)plan->tmap_y, ob ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.y, dims,
                strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    } else {
        memcpy(plan->tmap_y, plan->tmap, sizeof(plan->tmap));
    }
    plan->bn = bn;
    plan->batch = a.B;
    plan->y = a.y;
    plan->valid = 1;
    return cudaSuccess;
}

unsigned long long* g_conv_trace = nullptr;   // debug hook, see vd_debug_conv_trace

cudaError_t launch_conv_tc(const ConvArgs& a_in, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    if (!plan.valid) return cudaErrorInvalidValue;
    ConvArgs a = a_in;
    a.trace = g_conv_trace;
    if (!a.out_nchw && (a.y != plan.y || a.B > plan.batch)) return cudaErrorInvalidValue;   // the output map is bound at prepare time
    if (a.residual && a.residual != a.y) return cudaErrorInvalidValue;                      // residual is accumulated in place
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
