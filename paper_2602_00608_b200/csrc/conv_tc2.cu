// Two-CTA variant of the implicit-GEMM convolution (see conv_tc.cu for the fusion and the
// operand layout): a cluster of two CTAs on neighbouring SMs issues every MMA as one
// tcgen05.mma.cta_group::2 of M = 256 (one 16x8-pixel tile per CTA) x N = BN.  Each CTA stages
// only half of every weight tile (BN/2 rows) and the tensor cores of the pair read both halves,
// so the weight traffic through each SM's shared memory, and the operand bytes an MMA reads from
// it, drop; shared-memory bandwidth is what bounds the one-CTA kernel.
//
// Per CTA the roles are those of the one-CTA kernel (15 producer warps, a weight-loading thread,
// four epilogue warps); the MMA-issuing thread is active in the leader CTA (cluster rank 0) only.
// Barriers that gate the MMA live in the leader: the peer's producers and its weight loads signal
// the leader's "full" barriers across the cluster, and the leader's tcgen05.commit multicasts to
// the "empty" / "accumulator ready" barriers of both CTAs.  Every wait is bounded.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>

#include <algorithm>

#include "conv_tile.cuh"
#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;
using namespace convtile;

constexpr int MAX_B_STAGES2 = 8, MAX_A_STAGES2 = 4;

template <int BN> struct PairCfg {
    static constexpr int PAIR = BN == 256 ? 1 : 2;                   // tiles per CTA per work item
    static constexpr int B_STAGE_BYTES = (BN / 2) * 128;             // this CTA's half: BN/2 rows x 64 bf16
    static constexpr int B_STAGES = BN == 256 ? 6 : 8;
    static constexpr int B_GROUP = 2;                                // weight stages handed back per tcgen05.commit
    static constexpr int A_STAGES = BN == 256 ? 3 : 2;
    static constexpr int A_STAGE_BYTES = PAIR * A_TILE_BYTES;
    static constexpr int SMEM_B = B_STAGES * B_STAGE_BYTES;          // multiples of 1024
    static constexpr int SMEM_OUT = 2 * OUT_SLICE_BYTES;
    static constexpr int SMEM_A = A_STAGES * A_STAGE_BYTES;
    static constexpr int SMEM_TOTAL = SMEM_B + SMEM_OUT + SMEM_A + 512 + 1024;
    static constexpr int NBUF = 2;
    static constexpr int TMEM_COLS = NBUF * PAIR * BN;               // 512
};

struct Bars2 {
    uint64_t a_full[MAX_A_STAGES2], a_empty[MAX_A_STAGES2];
    uint64_t b_full[MAX_B_STAGES2], b_empty[MAX_B_STAGES2];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t epi_sync;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// ---- cluster / cta_group::2 PTX
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta) {     // shared::cta -> shared::cluster of `cta`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// tile load into this CTA's shared memory whose completion is reported to a barrier of the leader CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const void* tmap, int x, int y, uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
__device__ __forceinline__ void umma2_bf16_split(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                 uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 da, db;\nsetp.ne.b32 p, %6, 0;\n"
        "mov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n}\n"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// Tiles are numbered (frame, channel block, tile row, tile column), column fastest.  Every cluster
// owns a contiguous, balanced range of tile numbers and walks it in items of up to 2*PAIR tiles of
// one channel block; within an item CTA `rank` takes tiles t + 2*slot + rank.
struct Sched2 {
    int tiles_x, tiles, nblk, total, begin, end, per_item;
    __device__ __forceinline__ Tile get(int t, int bn) const {
        Tile r;
        const int blk = t / tiles;
        const int s = t - blk * tiles;
        r.b = blk / nblk;
        r.n0 = (blk - r.b * nblk) * bn;
        r.ty0 = (s / tiles_x) * TILE_H;
        r.tx0 = (s % tiles_x) * TILE_W;
        return r;
    }
    __device__ __forceinline__ int count(int t) const {          // tiles in the item that starts at t
        const int block_end = (t / tiles + 1) * tiles;
        return min(per_item, min(end, block_end) - t);
    }
};

// OUT_MODE: 0 = fp32 NHWC, 1 = bf16 NHWC
template <int BN, bool IN_BF16, int OUT_MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_tc2_kernel(const ConvArgs a, const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap2,
                const __grid_constant__ CUtensorMap tmap_y, unsigned int* status) {
    using Cfg = PairCfg<BN>;
    constexpr int NBUF = Cfg::NBUF, PAIR = Cfg::PAIR, A_STAGE_BYTES = Cfg::A_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;
    uint8_t* smem_out = smem + Cfg::SMEM_B;
    uint8_t* smem_a = smem_out + Cfg::SMEM_OUT;
    Bars2* bars = (Bars2*)(smem_a + Cfg::SMEM_A);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                 // 0 = leader (issues the MMAs), 1 = peer
    const int taps = a.ksize * a.ksize;
    const int kchunks = a.Cin >> 6;
    const int kchunks2 = a.x2 ? (a.Cin2 >> 6) : 0;
    const int ktotal = kchunks + kchunks2;
    const int nclusters = gridDim.x >> 1, cid = blockIdx.x >> 1;
    Sched2 sched;
    sched.tiles_x = (a.W + TILE_W - 1) / TILE_W;
    sched.tiles = sched.tiles_x * ((a.H + TILE_H - 1) / TILE_H);
    sched.nblk = a.Cout / BN;
    sched.total = sched.tiles * sched.nblk * a.B;
    sched.begin = (int)(((long long)sched.total * cid) / nclusters);
    sched.end = (int)(((long long)sched.total * (cid + 1)) / nclusters);
    sched.per_item = 2 * PAIR;

    if (tid == 0) {
        for (int i = 0; i < Cfg::A_STAGES; ++i) { mbar_init(smem_u32(&bars->a_full[i]), 2 * NUM_PRODUCER_WARPS); mbar_init(smem_u32(&bars->a_empty[i]), 1); }
        for (int i = 0; i < Cfg::B_STAGES; ++i) { mbar_init(smem_u32(&bars->b_full[i]), 2); mbar_init(smem_u32(&bars->b_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bars->acc_full[i]), 1); mbar_init(smem_u32(&bars->acc_empty[i]), 8); }
        mbar_init(smem_u32(&bars->epi_sync), 128);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == MMA_WARP) tmem_alloc2(smem_u32(&bars->tmem_base), (uint32_t)Cfg::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp < NUM_PRODUCER_WARPS) {
        // ------------------------------------------------ operand prologue (producers)
        const int j = tid & 7;
        const bool prologue = a.scale != nullptr;
        const bool silu = a.silu != 0;
        const int up = a.upsample ? 1 : 0;
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int t = sched.begin; t < sched.end && ok;) {
            const int n = sched.count(t);
            const int slots = (n + 1) >> 1;
            for (int kc = 0; kc < ktotal && ok; ++kc) {
                const bool second = kc >= kchunks;
                const bool in_bf16 = second ? false : IN_BF16;
                const int c0 = (second ? kc - kchunks : kc) * 64;
                const bool centre_only = second || a.ksize == 1;
                const bool pro = prologue && !second;
                for (int slot = 0; slot < slots && ok; ++slot) {
                    const int my = t + 2 * slot + (int)rank;
                    const bool have = my < t + n;             // an odd item leaves the peer without a tile
                    Tile tl = sched.get(have ? my : t, BN);
                    Raw8 raw[BATCH];
                    uint32_t vm = 0;
                    if (have) {
#pragma unroll
                        for (int u = 0; u < BATCH; ++u) {
                            const int pix = (u * NUM_PRODUCERS + tid) >> 3;
                            const int py = pix / PW, px = pix - py * PW;
                            const int oy = tl.ty0 + py - 1, ox = tl.tx0 + px - 1;
                            bool v = oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                            if (centre_only) v = v && py >= 1 && py <= TILE_H && px >= 1 && px <= TILE_W;
                            if (v) {
                                vm |= 1u << u;
                                if (second) load_raw(false, a.x2, (((size_t)tl.b * a.H + oy) * a.W + ox) * a.Cin2, c0, j, raw[u]);
                                else load_raw(IN_BF16, a.x, (((size_t)tl.b * a.Hs + (oy >> up)) * a.Ws + (ox >> up)) * a.Cin, c0, j, raw[u]);
                            }
                        }
                    }
                    float sc[8], sh[8];
                    if (pro && have) {
                        const int ca = c0 + (in_bf16 ? j * 8 : j * 4), cb = in_bf16 ? ca + 4 : ca + 32;
                        const float* ps = a.scale + (size_t)tl.b * a.Cin;
                        const float* pt = a.shift + (size_t)tl.b * a.Cin;
                        const float4 s0 = __ldg((const float4*)(ps + ca)), s1 = __ldg((const float4*)(ps + cb));
                        const float4 t0 = __ldg((const float4*)(pt + ca)), t1 = __ldg((const float4*)(pt + cb));
                        sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                        sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
                    }
                    if (slot == 0) {
                        ok = mbar_wait(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
                        if (!ok) break;
                    }
                    if (have) {
                        uint8_t* dst_tile = smem_a + stage * A_STAGE_BYTES + slot * A_TILE_BYTES;
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
                            const int pix = (u * NUM_PRODUCERS + tid) >> 3;
                            uint8_t* prow = dst_tile + pix * 128;
                            if (in_bf16) {
                                *(uint4*)(prow + ((j ^ (pix & 7)) << 4)) = make_uint4(o0, o1, o2, o3);
                            } else {
                                const int c = j >> 1, hb = (j & 1) * 8;
                                *(uint2*)(prow + ((c ^ (pix & 7)) << 4) + hb) = make_uint2(o0, o1);
                                *(uint2*)(prow + (((c + 4) ^ (pix & 7)) << 4) + hb) = make_uint2(o2, o3);
                            }
                        }
                    }
                    if (slot == slots - 1) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->a_full[stage]), 0));   // the leader's barrier
                        if (++stage == Cfg::A_STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            t += n;
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------ epilogue (this CTA's tiles)
        const int ew = warp - EPI_WARP0;
        const int m = ew * 32 + lane;
        const int et = tid - EPI_WARP0 * 32;
        const bool leader_thread = et == 0;
        const bool reduce_add = a.residual != nullptr;       // y is the residual stream: add the tile into it
        bool ok = true;
        int n_item = 0;
        uint32_t n_slice = 0, sync_phase = 0;
        auto epi_rendezvous = [&]() {
            mbar_arrive(smem_u32(&bars->epi_sync));
            const bool r = mbar_wait(smem_u32(&bars->epi_sync), sync_phase, abort_flag);
            sync_phase ^= 1;
            return r;
        };
        constexpr int CS = OUT_MODE == 1 ? 64 : 32;
        constexpr int NS = BN / CS;
        for (int t = sched.begin; t < sched.end && ok; ++n_item) {
            const int n = sched.count(t);
            const int slots = (n + 1) >> 1;
            const int buf = n_item % NBUF;
            ok = mbar_wait(smem_u32(&bars->acc_full[buf]), (n_item / NBUF) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            int my_slots = 0;                                // slots for which this CTA has a tile
            for (int slot = 0; slot < slots; ++slot) my_slots += (t + 2 * slot + (int)rank < t + n) ? 1 : 0;
            if (my_slots == 0) {                             // nothing of ours in the accumulators: hand them back at once
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[buf]), 0));
            }
#pragma unroll 1
            for (int slot = 0; slot < my_slots && ok; ++slot) {
                const Tile tl = sched.get(t + 2 * slot + (int)rank, BN);
                const uint32_t tacc = tmem_base + (uint32_t)((buf * PAIR + slot) * BN) + ((uint32_t)(ew * 32) << 16);
                const bool last_tile = slot == my_slots - 1;
#pragma unroll 1
                for (int sidx = 0; sidx < NS; ++sidx, ++n_slice) {
                    uint8_t* obuf = smem_out + (n_slice & 1) * OUT_SLICE_BYTES;
                    if (leader_thread) bulk_wait_group_read<1>();     // the store that last read this buffer is done
                    ok = __all_sync(0xffffffffu, epi_rendezvous());
                    if (!ok) break;
                    uint8_t* orow = obuf + m * 128;
#pragma unroll
                    for (int h = 0; h < CS / 32; ++h) {
                        uint32_t r[32];
                        tmem_ld32(tacc + (uint32_t)(sidx * CS + h * 32), r);
                        tmem_ld_wait();
                        if (last_tile && sidx == NS - 1 && h == CS / 32 - 1) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[buf]), 0));
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
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                *(float4*)(orow + ((c ^ (m & 7)) << 4)) = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                *(uint4*)(orow + (((h * 4 + c) ^ (m & 7)) << 4)) =
                                    make_uint4(pack_bf16(v[8 * c], v[8 * c + 1]), pack_bf16(v[8 * c + 2], v[8 * c + 3]),
                                               pack_bf16(v[8 * c + 4], v[8 * c + 5]), pack_bf16(v[8 * c + 6], v[8 * c + 7]));
                        }
                    }
                    fence_proxy_async_smem();
                    ok = __all_sync(0xffffffffu, epi_rendezvous());
                    if (!ok) break;
                    if (leader_thread) {
                        if (reduce_add) tma_reduce_add_4d(&tmap_y, smem_u32(obuf), tl.n0 + sidx * CS, tl.tx0, tl.ty0, tl.b);
                        else tma_store_4d(&tmap_y, smem_u32(obuf), tl.n0 + sidx * CS, tl.tx0, tl.ty0, tl.b);
                        bulk_commit_group();
                    }
                }
            }
            t += n;
        }
        if (leader_thread) bulk_wait_group<0>();
    } else if (warp == TMA_WARP) {
        // ------------------------------------------------ this CTA's half of every weight tile (TMA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const int half = BN / 2;
            for (int t = sched.begin; t < sched.end && ok; t += sched.count(t)) {
                const Tile tl = sched.get(t, BN);
                const int row0 = tl.n0 + (int)rank * half;
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    for (int tap = 0; tap < ntap; ++tap) {
                        if (stage % Cfg::B_GROUP == 0) {     // stages come back in groups (see the MMA thread)
                            ok = mbar_wait(smem_u32(&bars->b_empty[stage / Cfg::B_GROUP]), phase ^ 1, abort_flag);
                            if (!ok) break;
                        }
                        const uint32_t full = map_to_cta(smem_u32(&bars->b_full[stage]), 0);      // the leader's barrier
                        mbar_arrive_expect_tx_cluster(full, Cfg::B_STAGE_BYTES);
                        const uint32_t dst = smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES);
                        if (second) tma_load_2d_pair(dst, &tmap2, (kc - kchunks) * 64, row0, full);
                        else tma_load_2d_pair(dst, &tmap, kc * 64, tap * a.Cout + row0, full);
                        if (++stage == Cfg::B_STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------ MMA issue (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, BN);
            const uint32_t a_hi = desc_hi(PW * 128, 2), b_hi = desc_hi(1024, 2);
            const uint32_t a_lo0 = desc_lo(smem_u32(smem_a)), b_lo0 = desc_lo(smem_u32(smem_b));
            Tracer tr; tr.init(a.trace, 1);
            uint32_t as = 0, aph = 0, bs = 0, bph = 0;
            bool ok = true;
            int n_item = 0;
            for (int t = sched.begin; t < sched.end && ok; ++n_item) {
                const int n = sched.count(t);
                const int slots = (n + 1) >> 1;
                const int buf = n_item % NBUF;
                tr.mark(20);
                ok = mbar_wait(smem_u32(&bars->acc_empty[buf]), ((n_item / NBUF) & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * PAIR * BN);
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
                        const bool centre = second || a.ksize == 1;
                        const int ky = centre ? 1 : tap / 3, kx = centre ? 1 : tap - 3 * (tap / 3);
                        const uint32_t b_lo = b_lo0 + bs * (Cfg::B_STAGE_BYTES >> 4);
                        uint32_t a_lo = a_lo0 + as * (A_STAGE_BYTES >> 4) + (uint32_t)(ky * PW + kx) * 8;
                        const uint32_t acc = (kc | tap) != 0;
                        uint32_t td = tmem_d;
                        for (int slot = 0; slot < slots; ++slot) {
                            umma2_bf16_split(td, a_lo, a_hi, b_lo, b_hi, idesc, acc);
                            umma2_bf16_split(td, a_lo + 2, a_hi, b_lo + 2, b_hi, idesc, 1u);
                            umma2_bf16_split(td, a_lo + 4, a_hi, b_lo + 4, b_hi, idesc, 1u);
                            umma2_bf16_split(td, a_lo + 6, a_hi, b_lo + 6, b_hi, idesc, 1u);
                            a_lo += A_TILE_BYTES >> 4;
                            td += BN;
                        }
                        // tcgen05.commit is served at a limited rate, so stages are handed back in groups
                        if (bs % Cfg::B_GROUP == Cfg::B_GROUP - 1) umma2_commit_both(smem_u32(&bars->b_empty[bs / Cfg::B_GROUP]));
                        if (++bs == Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                    }
                    umma2_commit_both(smem_u32(&bars->a_empty[as]));
                    if (++as == Cfg::A_STAGES) { as = 0; aph ^= 1; }
                }
                if (ok) umma2_commit_both(smem_u32(&bars->acc_full[buf]));
                t += n;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // nobody leaves while the pair may still touch its memory
    if (tid == 0 && bars->abort_flag && status) {
        if (atomicCAS(status, 0u, 0xC0DE0003u) == 0u) {
            status[1] = blockIdx.x;
            status[2] = (uint32_t)BN;
        }
    }
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, (uint32_t)Cfg::TMEM_COLS);
    }
}

int max_clusters_cached(const void* kern, int smem) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) n = 0;
    return n;
}

template <int BN, bool IB, int OM>
cudaError_t launch_pair(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    auto kern = conv_tc2_kernel<BN, IB, OM>;
    static int max_clusters = -1;
    if (max_clusters < 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<BN>::SMEM_TOTAL);
        if (e != cudaSuccess) return e;
        max_clusters = max_clusters_cached((const void*)kern, PairCfg<BN>::SMEM_TOTAL);
        if (getenv("VD_CONV_VERBOSE")) fprintf(stderr, "conv_tc2<%d>: max active clusters %d\n", BN, max_clusters);
    }
    if (max_clusters <= 0) return cudaErrorNotSupported;
    const int tiles = ((a.W + TILE_W - 1) / TILE_W) * ((a.H + TILE_H - 1) / TILE_H);
    const long long total = (long long)tiles * (a.Cout / BN) * a.B;
    const int nclusters = (int)std::min<long long>((total + 1) / 2, max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * nclusters, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = PairCfg<BN>::SMEM_TOTAL;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a, *(const CUtensorMap*)plan.tmap_half, *(const CUtensorMap*)plan.tmap2_half,
                              *(const CUtensorMap*)plan.tmap_y, status);
}

}  // namespace

bool conv_tc2_supported(const ConvArgs& a) {
    return a.Cout % 128 == 0 && !a.out_nchw && a.Cin % 64 == 0 && (!a.x2 || a.Cin2 % 64 == 0);
}

cudaError_t launch_conv_tc2(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    const bool ib = a.in_dtype == VD_BF16, ob = a.out_dtype == VD_BF16;
    if (plan.bn == 256) {
        if (ib && ob) return launch_pair<256, true, 1>(a, plan, status, s);
        if (ib && !ob) return launch_pair<256, true, 0>(a, plan, status, s);
        if (!ib && ob) return launch_pair<256, false, 1>(a, plan, status, s);
        return launch_pair<256, false, 0>(a, plan, status, s);
    }
    if (ib && ob) return launch_pair<128, true, 1>(a, plan, status, s);
    if (ib && !ob) return launch_pair<128, true, 0>(a, plan, status, s);
    if (!ib && ob) return launch_pair<128, false, 1>(a, plan, status, s);
    return launch_pair<128, false, 0>(a, plan, status, s);
}

}  // namespace vd
