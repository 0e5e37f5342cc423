// Implicit-GEMM 3x3 / 1x1 convolution on the 5th-generation tensor cores (tcgen05 + TMEM), with
// the paper's fusion folded around it (Section IV-B.1, Eq. 9): the GroupNorm-apply + SiLU of the
// chain runs in the operand prologue, nearest-2x upsampling is collapsed into four 2x2 convolutions
// of the source (or, in the 9-tap form, an address computation), and bias, residual add, the 1x1
// shortcut and the output cast run in / next to the same accumulation, so each activation crosses
// HBM once.
//
// Persistent kernel, one CTA per SM, roles decoupled through mbarrier rings:
//   * tile = 16x8 output pixels x BN output channels:  D[128 x BN] = sum over taps and 64-channel
//     chunks of A_tap[128 x 64] * W_tap[64 x BN].  Every CTA owns a contiguous, balanced range of
//     tiles; where BN <= 128 it walks it in work items of two tiles that share every weight stage.
//   * 15 producer warps (on the SM sub-partitions the MMA warp is not on) read the raw 18x10-pixel
//     halo tile of a 64-channel chunk once, apply scale/shift (+SiLU), round to bf16 and store it
//     in shared memory as 180 rows of 128 bytes in the 128-byte-swizzled K-major layout.  Every
//     tap is a *view* of that one tile (descriptor start (ky*10+kx) rows in; eight-row groups are
//     one tile row = 10 pixels apart), so the transform runs once per element, not once per tap.
//     Out-of-image halo pixels are exact zeros (padding applies to the transformed tensor).
//     For two-tile items and two-CTA pairs the raw input of the next unit is staged in shared
//     memory by cp.async while the current unit is transformed.
//     An optional second input (the block's raw fp32 input for a width-changing ResNet block) is
//     appended as extra K: the 1x1 shortcut without its own round trip.  It needs no transform, so
//     bulk tensor loads put it into the operand stages as it is and it is multiplied in tf32.
//   * 1 warp streams the weights (bf16 [tap][Cout][Cin]) by TMA into 128B-swizzled stages.
//   * 1 warp issues tcgen05.mma (M=128, N=BN, K=16) into TMEM accumulators, double-buffered so an
//     item's epilogue overlaps the next item.  The whole warp runs the loop and the tensor
//     instructions are predicated on one elected lane (no branch), so the issue sequence is
//     warp-uniform code with its descriptor arithmetic in uniform registers.
//   * 4 epilogue warps drain the accumulators: tcgen05.ld, + bias, and the tile leaves through
//     shared memory as 128-byte-wide slices written by bulk tensor stores, which coalesce the
//     traffic and clip the ragged image edge.  Where the layer has a residual, the output buffer
//     IS the residual stream and the store is a bulk tensor reduce-add (the fp32 add x + conv(h)
//     is done once, by the memory system), so the residual never passes through the SM.
//     The 3-channel frame head writes its NCHW planes directly.  Outputs are stored with the
//     evict-last L2 policy: the statistics pass and the layer that follow read them from L2.
//   * Upsampling layers run as pairs of CTAs (tcgen05.mma.cta_group::2) in the phase-collapsed
//     form: one halo tile of 16x8 SOURCE pixels, four parity accumulators, 16 instead of 36 tap
//     products (see TileCfg and PhaseSched).
// Every wait is bounded: on expiry the CTA records a code in the status word and unwinds.
#include <cuda.h>
#include <cuda_fp16.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <type_traits>

#include "conv_tile.cuh"
#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;
using namespace convtile;

constexpr int MAX_B_STAGES = 8, MAX_A_STAGES = 6;
constexpr int WARP_SLICE_BYTES = 32 * 128;                           // one epilogue warp's share of an output slice

// BN = output channels per work item.  Where the channel block is narrow (BN <= 128) a work
// item is two 16x8-pixel tiles whose MMAs consume every weight stage together, which halves the
// weight traffic through shared memory and the bytes the TMA pipeline must keep in flight.
//
// CG = 2 (BN = 256 only): a cluster of two CTAs on neighbouring SMs issues every MMA as one
// tcgen05.mma.cta_group::2 of M = 256 (one tile per CTA) x N = 256.  Each CTA stages only its half of
// every weight tile (128 rows) and the tensor cores of the pair read both halves, so the weight bytes
// each SM pulls from L2 are halved; the one-CTA kernel is bound there by that traffic (32 KB per 513
// tensor cycles and SM).  The MMA warp is active in the leader CTA (cluster rank 0) only.  Barriers
// that gate the MMAs live in the leader: the peer's producers and weight loads signal the leader's
// "full" barriers across the cluster, its epilogue the leader's "accumulator free" barrier, and the
// leader's tcgen05.commit arrives on the "empty" / "accumulator ready" barriers of both CTAs.
//
// PH (phase-collapsed nearest-2x upsampling + 3x3, BN = 128 on CTA pairs): a 3x3 convolution of the
// upsampled tensor is, for each of the four output parities (a, b) = (row & 1, column & 1), a 2x2
// convolution of the SOURCE tensor whose weights are sums of the 3x3 taps that fall on the same source
// pixel (rows: parity 0 reads source rows {i-1 <- ky 0; i <- ky 1+2}, parity 1 {i <- ky 0+1; i+1 <- ky 2};
// columns alike).  So the tile is 16x8 SOURCE pixels, its one halo tile feeds four accumulators
// (one per parity, 128 columns each: all of tensor memory) through 4 x 4 tap views, and 16 instead
// of 4 x 9 = 36 tap products are issued per source pixel and 64-channel chunk: 4/9 of the work.
// The accumulators have no second set; instead each parity has its own "full"/"empty" barriers and
// is drained as soon as its last tap has completed, while the MMAs of the other parities go on.
// A weight stage holds the two column taps (dx = 0, 1) of one (parity, dy): 8 MMAs per stage, so
// the issue sequence per stage is as long as that of the other forms.
// With four accumulators and no spare set, an accumulator is needed again right after its item's last
// chunk, and draining it takes about as long as a chunk's MMAs.  So the parities are staggered (where
// the input has at least four chunks): parity p works on the chunk that came p chunks earlier, the four
// accumulators complete one chunk apart, and within a chunk slot the parities run in a rotating order in
// which the one that completes goes first and the one that completed a slot before goes last: between an
// accumulator's last MMA and its next first MMA lie the MMAs of six (parity, chunk) blocks.  An operand
// chunk therefore stays in shared memory for four slots (five stages).  PhaseSched is that schedule; the
// weight loader follows it step by step.
template <int BN, int CG = 1, bool PH = false, bool IN_BF16 = false> struct TileCfg {
    static_assert(CG == 1 || BN >= 128, "the two-CTA form exists for 128- and 256-channel blocks");
    static_assert(!PH || (BN == 128 && CG == 2), "the phase form runs 128-channel blocks on CTA pairs");
    static constexpr int PAIR = PH ? 1 : (BN == 256 ? 1 : 2);        // tiles per work item (and CTA)
    static constexpr int B_STAGE_BYTES = (PH ? 2 : 1) * (BN / CG) * 128;   // this CTA's rows x 64 bf16 (phase: two taps)
    // output slices per epilogue warp (128-channel blocks: a second slice buffer pays more than a fourth weight stage)
    static constexpr int OUT_BUFS = (PH || BN == 128) ? 2 : 1;
    // weight stages: as many as fit (the weight stream waits on the latency of L2, which the SM clock does not shorten)
    // (128-channel blocks: the staging of a bf16 input is half the size, which buys a fourth stage; measured, the MMA
    // warp of such a layer waits on weights for a quarter of its time with three)
    static constexpr int B_STAGES = PH ? 4 : (CG == 2 ? (BN == 256 ? 7 : 8) : (BN == 256 ? 5 : (BN == 128 ? (IN_BF16 ? 4 : 3) : 8)));
    static constexpr int B_GROUP = BN >= 128 ? 1 : 2;                // weight stages handed back per tcgen05.commit
    static constexpr int A_STAGES = PH ? 5 : 2;                    // phase form: a chunk stays until the parity that lags most has used it
    static constexpr int A_STAGE_BYTES = PAIR * A_TILE_BYTES;
    static constexpr int SMEM_B = (B_STAGES * B_STAGE_BYTES + 1023) / 1024 * 1024;
    static constexpr int SMEM_OUT = BN >= 128 ? OUT_BUFS * OUT_SLICE_BYTES : 0;       // output slice(s) per epilogue warp
    static constexpr int SMEM_A = A_STAGES * A_STAGE_BYTES - (A_TILE_BYTES - NPIX * 128);   // the last tile needs no padding
    static constexpr int SMEM_BIAS = BN >= 128 ? 4 * BN * 4 : 0;     // one bias copy per epilogue warp
    static constexpr int SMEM_BARS = 512;
    // two-tile items and two-CTA pairs: the producers stage the raw input of the next unit in shared memory (cp.async)
    static constexpr bool STAGED = !PH && (PAIR == 2 || CG == 2);
    static constexpr int SMEM_RAW = STAGED ? ITEMS * (IN_BF16 ? 16 : 32) : 0;
    static constexpr int SMEM_TOTAL = SMEM_B + SMEM_OUT + SMEM_A + SMEM_BIAS + SMEM_BARS + SMEM_RAW + 1024;  // + barriers + alignment slack
    static constexpr int ACC_COLS = BN < 32 ? 32 : BN;               // TMEM columns per accumulator
    static constexpr int NBUF = PH ? 1 : 2;                          // accumulator sets (PAIR tiles each; phase: four parities)
    static constexpr int TMEM_COLS = PH ? 4 * ACC_COLS : NBUF * PAIR * ACC_COLS;
};

struct Bars {                    // lives in shared memory
    uint64_t a_full[MAX_A_STAGES], a_empty[MAX_A_STAGES];
    uint64_t b_full[MAX_B_STAGES], b_empty[MAX_B_STAGES];
    uint64_t acc_full[4], acc_empty[4];
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t stat_last;          // this CTA is the last to finish (it folds the statistics records)
};

// Tiles are numbered (frame, channel block, tile row, tile column), column fastest.  Every CTA
// owns a contiguous, balanced range of tile numbers and walks it in items of `pair` tiles (one
// when the range or the channel block ends).
//
// Two-CTA form: the range belongs to the cluster, an item is up to two tiles of one channel block,
// and CTA `rank` of the pair takes tile t + rank (the peer has none in an odd tail item).
//
// Every role decodes tile numbers once per item, the fifteen producer warps among them, so the three
// divisions are multiplications by a reciprocal the launcher computed: floor(t / d) = umulhi(t, ceil(2^32 / d)),
// exact while t * d < 2^32 (the launcher checks it).
struct Sched {
    int tiles_x, tiles, nblk, total;
    int begin, end, pair;
    int cg, rank;
    uint32_t m_tiles, m_nblk, m_tx;
    static __device__ __forceinline__ int fdiv(int t, uint32_t m) { return m ? (int)__umulhi((uint32_t)t, m) : t; }
    __device__ __forceinline__ Tile get(int t, int bn) const {
        Tile r;
        const int blk = fdiv(t, m_tiles);        // frame * nblk + channel block
        const int s = t - blk * tiles;
        r.b = fdiv(blk, m_nblk);
        r.n0 = (blk - r.b * nblk) * bn;
        const int row = fdiv(s, m_tx);
        r.ty0 = row * TILE_H;
        r.tx0 = (s - row * tiles_x) * TILE_W;
        return r;
    }
    // number of tiles of the item that starts at tile t: up to pair * cg consecutive tiles of one (frame, channel block)
    __device__ __forceinline__ int count(int t) const {
        const int cap = pair * cg;
        const int blk = fdiv(t, m_tiles);
        int n = 1;
        while (n < cap && t + n < end && fdiv(t + n, m_tiles) == blk) ++n;
        return n;
    }
    // of those, the tiles this CTA works on (the pair's CTAs take alternate tiles), and the s-th of them
    __device__ __forceinline__ int mine(int n) const { return cg == 2 ? ((n - rank + 1) >> 1) : n; }
    __device__ __forceinline__ int index(int t, int s) const { return cg == 2 ? t + 2 * s + rank : t + s; }
};

// The phase form's order of (parity, chunk) blocks.  The CTA's work is a sequence of chunk slots
// q = item * K + chunk (K chunks per item); in step s the parities run in the order (r + j) & 3, j = 0..3, and
// parity p works on slot q = s - p * lag (skipped while that is outside [0, S)).
struct PhaseSched {
    int K, S, lag;
    uint32_t m_k;                // ceil(2^32 / K), 0 for K = 1
    __device__ __forceinline__ void init(int kchunks, int nitems) {
        K = kchunks; S = nitems * kchunks; lag = kchunks >= 4 ? 1 : 0;
        m_k = K == 1 ? 0u : (uint32_t)((0x100000000ull + (uint32_t)K - 1) / (uint32_t)K);
    }
    __device__ __forceinline__ int steps() const { return S + 3 * lag; }
    __device__ __forceinline__ int rot(int s) const { return lag ? ((s + 1 + 3 * K) & 3) : 0; }
    __device__ __forceinline__ int item_of(int q) const { return m_k ? (int)__umulhi((uint32_t)q, m_k) : q; }
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
// Arrival on a barrier of the pair's leader CTA.  Release at CTA scope: the arriving warp's own shared-memory
// stores (already made visible to the tensor core's proxy by its fence) are what the arrival publishes; nothing of
// the peer CTA's memory is.  The cluster-scope form of the same instruction costs about 1600 cycles per arrival
// here instead of about 100 (measured: stamps around the producers' hand-over).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cta.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
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
__device__ __forceinline__ void umma2_bf16_split_on(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                    uint32_t idesc, uint32_t accumulate, uint32_t on) {
    asm volatile(
        "{\n.reg .pred p, q;\n.reg .b64 da, db;\nsetp.ne.b32 p, %6, 0;\nsetp.ne.b32 q, %7, 0;\n"
        "mov.b64 da, {%1, %2};\nmov.b64 db, {%3, %4};\n"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n}\n"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(on) : "memory");
}
__device__ __forceinline__ void umma2_commit_both_on(uint32_t bar, uint32_t on) {
    const uint32_t peer = map_to_cta(bar, 1);
    asm volatile("{\n.reg .pred q;\nsetp.ne.b32 q, %2, 0;\n"
                 "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
                 "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%1];\n}\n" ::"r"(bar), "r"(peer), "r"(on) : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs of the pair:
// one commit to the leader's own barrier, one to the peer's through its cluster address
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(map_to_cta(bar, 1)) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---- GroupNorm statistics of the output, taken in the epilogue (Section IV-B.1: the normalisation's reduction
// rides on the tensor that is already on chip instead of reading it back from memory).
// An epilogue thread holds 32 consecutive channels of one pixel per pass.  It adds the values and their squares in
// quads of four channels, and a transposing butterfly over the warp's 32 pixels leaves the total of value
// i = lane >> 1 (i < 8: sum of quad i; i >= 8: sum of squares of quad i - 8) in every lane: 15 exchanges instead of
// 16 full reductions.  The first exchange pairs a quad's sum with its own sum of squares, so it runs quad by quad
// while the pass is still being converted and stored.
// The total of a (tile, pass) depends on the tile's values alone.  It is turned into 64-bit fixed point there and
// then, and every later addition (over the tiles of a CTA, over the CTAs by atomic adds, in the fold) is an
// integer addition: the result does not depend on how the tiles are divided among the CTAs, on the batch a frame
// is decoded in, or on the order the atomic adds arrive in.
constexpr float kStatSumFix = 1048576.f;      // 2^20: sums        (|total| < 2^43 * 2^20 units ... values to about 1e6 in magnitude)
constexpr float kStatSqFix = 65536.f;         // 2^16: sums of squares (values to about 1e4 in magnitude over 1.4e6 elements)
__device__ __forceinline__ float stat_quad_first(float a0, float a1, float a2, float a3, bool valid, bool hi) {
    float s = (a0 + a1) + (a2 + a3);
    float q = fmaf(a0, a0, fmaf(a1, a1, fmaf(a2, a2, a3 * a3)));
    s = valid ? s : 0.f;
    q = valid ? q : 0.f;
    const float keep = hi ? q : s, send = hi ? s : q;
    return keep + __shfl_xor_sync(0xffffffffu, send, 16);
}
__device__ __forceinline__ long long stat_reduce(float (&v)[8], int lane) {
#pragma unroll
    for (int st = 0; st < 3; ++st) {
        const int half = 4 >> st, bit = 8 >> st;
        const bool hi = (lane & bit) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float keep = hi ? v[i + half] : v[i];
            const float send = hi ? v[i] : v[i + half];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
        }
    }
    const float r = v[0] + __shfl_xor_sync(0xffffffffu, v[0], 1);
    return __float2ll_rn(r * ((lane & 16) ? kStatSqFix : kStatSumFix));
}

// Adds a warp's accumulated pass totals of channel block [n0, n0 + 32 * NP) of frame b to the layer's sums
// stat_sum[b][group][2] (sum, sum of squares).
template <int NP>
__device__ __forceinline__ void stat_flush(const ConvArgs& a, long long (&acc)[NP], int b, int n0, int lane) {
    const int cpg = a.Cout / a.stat_G;
    const int vi = lane >> 1, quad = vi & 7, is_q = vi >> 3;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        if ((lane & 1) == 0) {
            const int g = (n0 + p * 32 + quad * 4) / cpg;
            atomicAdd(a.stat_sum + ((size_t)b * a.stat_G + g) * 2 + is_q, (unsigned long long)acc[p]);
        }
        acc[p] = 0;
    }
}

// The CTA that finishes last turns the sums into the affine map of the normalisation (scale = gamma * rstd,
// shift = beta - mean * scale) and clears them for the next launch.
__device__ void stat_finalize(const ConvArgs& a, int tid, void* smem_scratch) {
    float* s_mean = (float*)smem_scratch;
    float* s_rstd = s_mean + 32;
    const int G = a.stat_G, cpg = a.Cout / G;
    for (int b = 0; b < a.B; ++b) {
        if (tid < G) {
            unsigned long long* p = a.stat_sum + ((size_t)b * G + tid) * 2;
            const double S = (double)(long long)__ldcg(p) * (1.0 / (double)kStatSumFix);
            const double Q = (double)(long long)__ldcg(p + 1) * (1.0 / (double)kStatSqFix);
            p[0] = 0ull;
            p[1] = 0ull;
            const double inv_n = 1.0 / ((double)a.H * (double)a.W * (double)cpg);
            const double mean = S * inv_n;
            const double var = fmax(Q * inv_n - mean * mean, 0.0);
            s_mean[tid] = (float)mean;
            s_rstd[tid] = 1.0f / sqrtf((float)(var + (double)a.stat_eps));
        }
        __syncthreads();
        for (int c = tid; c < a.Cout; c += NUM_THREADS) {
            const int gc = c / cpg;
            const float sc = __ldg(a.stat_gamma + c) * s_rstd[gc];
            a.stat_scale[(size_t)b * a.Cout + c] = sc;
            a.stat_shift[(size_t)b * a.Cout + c] = __ldg(a.stat_beta + c) - s_mean[gc] * sc;
        }
        __syncthreads();
    }
}

// OUT_MODE: 0 = fp32 NHWC, 1 = bf16 NHWC (both through shared memory and TMA stores),
//           2 = NCHW frame written directly (dtype from a.out_dtype)
// STATS: the epilogue also takes the GroupNorm statistics of the output (a build of its own: compiled in but switched
// off, the extra live values cost the bf16-output kernels 1.4 % of a decode in spills)
// BIAS: the epilogue adds the bias (a build without it for the layers whose bias is accounted for downstream: the
// additions and the bias loads are more than half of a pass's instructions)
// X2: the layer has a second input (the fused 1x1 shortcut); the other builds carry none of its code
// KS: kernel size, 3 or 1 (the 1x1 layers take the centre view of the halo tile only)
template <int BN, bool IN_BF16, int OUT_MODE, int CG = 1, bool PH = false, bool STATS = false, bool BIAS = true, bool X2 = false, int KS = 3>
__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_tc_kernel(const ConvArgs a, const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap2,
               const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_x2, unsigned int* status) {
    using Cfg = TileCfg<BN, CG, PH, IN_BF16>;
    constexpr int NBUF = Cfg::NBUF, PAIR = Cfg::PAIR, A_STAGE_BYTES = Cfg::A_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;
    uint8_t* smem_out = smem + Cfg::SMEM_B;
    uint8_t* smem_a = smem_out + Cfg::SMEM_OUT;
    uint8_t* smem_bias = smem_a + Cfg::SMEM_A;
    Bars* bars = (Bars*)(smem_bias + Cfg::SMEM_BIAS);
    static_assert(sizeof(Bars) <= Cfg::SMEM_BARS, "barrier block");
    static_assert(Cfg::SMEM_TOTAL <= 232448, "shared memory of one CTA");
    uint8_t* smem_stage = smem_bias + Cfg::SMEM_BIAS + Cfg::SMEM_BARS;  // raw input of the next unit (two-tile items only)
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int taps = KS * KS;
    const int kchunks = a.Cin >> 6;
    // Extra K: the 1x1 shortcut on a second input (fp32, at the output resolution), in sub-chunks of 32 channels.
    // It needs no halo and no transform, so it does not go through the producers: a bulk tensor load puts the
    // fp32 tile (16 x 8 pixels x 32 channels = 128 rows of 128 bytes) straight into an operand stage, the weights
    // come as fp32 too, and the products are tcgen05.mma kind::tf32 (K = 8) into the same accumulator.  Operands
    // keep 10 significant bits instead of bf16's 8; the tensor time of these chunks doubles, the producers' is gone.
    const int kchunks2 = X2 ? (a.Cin2 >> 5) : 0;
    constexpr uint32_t SC_TILE_BYTES = TILE_H * TILE_W * 128;
    const int ktotal = kchunks + kchunks2;
    const int cout_pad = (a.Cout % 128 == 0) ? a.Cout : 16; // rows per tap in the packed weights
    Sched sched;
    sched.tiles_x = (a.W + TILE_W - 1) / TILE_W;
    sched.tiles = sched.tiles_x * ((a.H + TILE_H - 1) / TILE_H);
    sched.nblk = cout_pad / BN;
    sched.total = sched.tiles * sched.nblk * a.B;
    // work is divided among the CTAs (CG = 1) or among the clusters of two (CG = 2)
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;  // 0 = leader (issues the MMAs), 1 = peer
    const int nworkers = (int)gridDim.x / CG, worker = (int)blockIdx.x / CG;
    sched.begin = (int)((uint32_t)sched.total * (uint32_t)worker / (uint32_t)nworkers);          // the launcher checked the range
    sched.end = (int)((uint32_t)sched.total * (uint32_t)(worker + 1) / (uint32_t)nworkers);
    sched.m_tiles = a.div_tiles; sched.m_nblk = a.div_nblk; sched.m_tx = a.div_tx;
    sched.pair = PAIR;
    sched.cg = CG;
    sched.rank = (int)rank;

    if (tid == 0) {
        // CG = 2: the leader's "full" barriers collect the arrivals of both CTAs; commits go to both CTAs
        for (int i = 0; i < Cfg::A_STAGES; ++i) { mbar_init(smem_u32(&bars->a_full[i]), CG * NUM_PRODUCER_WARPS); mbar_init(smem_u32(&bars->a_empty[i]), 1); }
        for (int i = 0; i < Cfg::B_STAGES; ++i) { mbar_init(smem_u32(&bars->b_full[i]), CG); mbar_init(smem_u32(&bars->b_empty[i]), 1); }
        for (int i = 0; i < 4; ++i) { mbar_init(smem_u32(&bars->acc_full[i]), 1); mbar_init(smem_u32(&bars->acc_empty[i]), 4 * CG); }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == MMA_WARP) {
        if (CG == 2) tmem_alloc2(smem_u32(&bars->tmem_base), (uint32_t)Cfg::TMEM_COLS);
        else tmem_alloc(smem_u32(&bars->tmem_base), (uint32_t)Cfg::TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                         // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    // addresses, in the leader CTA, of the barriers that both CTAs signal
    auto leader_bar = [&](uint64_t* b) -> uint32_t { return CG == 2 ? map_to_cta(smem_u32(b), 0) : smem_u32(b); };
    auto arrive_leader = [&](uint64_t* b) {
        if (CG == 2) mbar_arrive_cluster(map_to_cta(smem_u32(b), 0));
        else mbar_arrive(smem_u32(b));
    };
    const uint32_t tmem_base = bars->tmem_base;
    // The kernel after this one may set itself up from here on.  Of this kernel, only the roles
    // that touch activations wait for the kernel before it; weights (TMA warp) and the MMA issue
    // loop (fed by the other roles) need no wait.
    griddep_launch();

    if (is_producer_warp(warp)) {
        // ------------------------------------------------ operand prologue (producers)
        // The work is a sequence of units (item, chunk, tile slot); a thread owns three (pixel,
        // 8-channel group) entries of every unit, all loaded before any is consumed.  The role is
        // bound by instruction issue, so whatever depends only on the thread (where an entry sits
        // in the halo tile, in shared memory and relative to the tile's first source pixel) is
        // computed once, and tiles whose halo lies inside the image skip the bounds checks.
        const int ptid = producer_index(warp) * 32 + lane;  // 0..479 over the producer warps
        const int j = ptid & 7;                             // this thread's channel group within a chunk
        const bool prologue = a.scale != nullptr;
        const bool silu = a.silu != 0;
        const int up = a.upsample ? 1 : 0;
        constexpr int ESZ = IN_BF16 ? 2 : 4;
        uint32_t soff[BATCH];        // byte offset of the entry's (first) 8/16-byte store within a tile chunk
        int goff[BATCH];             // byte offset of the entry's source pixel from the tile's first source pixel
        uint32_t pyx[BATCH];         // py | px << 8 | (entry lies in the tile proper, not the halo) << 16
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int pix = (u * NUM_PRODUCERS + ptid) >> 3;
            const int py = pix / PW, px = pix - py * PW;
            // row = halo pixel (128 B = 64 channels), 16-byte chunk c stored at c ^ (row & 7): the
            // 128-byte swizzle of the K-major operand layout (tile bases are 1024-byte aligned).
            // bf16 input: the thread's channels [8j, 8j+8) are chunk j.  fp32 input: channels
            // [4j, 4j+4) are half (j & 1) of chunk j / 2 and [32+4j, ..) the same half of chunk 4 + j / 2,
            // whose offset differs from the first by exactly 64 bytes (bit 2 of the chunk number).
            soff[u] = IN_BF16 ? (uint32_t)(pix * 128 + ((j ^ (pix & 7)) << 4))
                              : (uint32_t)(pix * 128 + (((j >> 1) ^ (pix & 7)) << 4) + (j & 1) * 8);
            goff[u] = ((((py - 1) >> up) * a.Ws + ((px - 1) >> up)) * a.Cin) * ESZ;
            const bool inner = py >= 1 && py <= TILE_H && px >= 1 && px <= TILE_W;
            pyx[u] = (uint32_t)py | ((uint32_t)px << 8) | (inner ? 1u << 16 : 0u);
        }
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        griddep_wait();              // everything above is arithmetic on the thread's own indices
        if constexpr (Cfg::STAGED) {
            // Two-tile items (narrow channel blocks) and two-CTA pairs are bound by this role, and a thread's registers hold
            // one unit of input only.  So the raw input of the NEXT unit travels by cp.async into a
            // shared-memory staging area while the current unit is transformed: every thread copies exactly
            // the entries it later reads back (16-byte pieces at [half][entry][thread]), so the staging needs
            // no synchronisation between threads, and invalid entries are zero-filled by the copy.
            struct Pos { int t, n, cnt, kc, slot; Tile tile; };   // n tiles in the item, cnt of them this CTA's; tile = its slot-th
            auto first_of_item = [&](Pos& p) {
                p.n = sched.count(p.t);
                p.cnt = sched.mine(p.n);                         // 0: the peer of a two-CTA pair in an odd tail item
                p.tile = sched.get(p.cnt > 0 ? sched.index(p.t, 0) : p.t, BN);
            };
            auto advance = [&](Pos& p) {
                if (++p.slot < p.cnt) {                          // the item's second tile of this CTA: CG tiles on in its channel block
#pragma unroll
                    for (int k = 0; k < CG; ++k) {
                        p.tile.tx0 += TILE_W;
                        if (p.tile.tx0 >= sched.tiles_x * TILE_W) { p.tile.tx0 = 0; p.tile.ty0 += TILE_H; }
                    }
                    return;
                }
                const bool two = p.slot == 2;
                p.slot = 0;
                if (++p.kc < ktotal) {                           // next chunk of the same item: back to its first tile
                    if (two) {
#pragma unroll
                        for (int k = 0; k < CG; ++k) {
                            if (p.tile.tx0 == 0) { p.tile.tx0 = (sched.tiles_x - 1) * TILE_W; p.tile.ty0 -= TILE_H; }
                            else p.tile.tx0 -= TILE_W;
                        }
                    }
                    return;
                }
                p.kc = 0;
                p.t += p.n;
                if (p.t < sched.end) first_of_item(p);
            };
            // Interior tiles of a 3x3 layer (nine in ten) take a short form of the copy: every entry exists, so
            // its address is the tile's origin (the source pixel one row and one column before the tile's
            // first, this thread's channels) plus an offset that depends on the thread only.
            const uint32_t pixbytes = (uint32_t)a.Cin * ESZ;
            const uint32_t halo_off = ((uint32_t)a.Ws + 1u) * pixbytes;
            uint32_t goffp[BATCH];
#pragma unroll
            for (int u = 0; u < BATCH; ++u) goffp[u] = (uint32_t)(goff[u] + (int)halo_off);
            const char* x_thread = (const char*)a.x + j * 16;
            const uint32_t st_lo = smem_u32(smem_stage) + (uint32_t)ptid * 16u;           // + u * NUM_PRODUCERS * 16
            const uint32_t st_hi = st_lo + (uint32_t)(ITEMS * 16);
            // starts the copies of unit p; returns which of this thread's entries exist
            auto issue = [&](const Pos& p) -> uint32_t {
                const bool second = X2 && p.kc >= kchunks;
                const int c0 = (second ? p.kc - kchunks : p.kc) * 64;
                constexpr bool centre_only = KS == 1;
                const Tile& tile = p.tile;
                if (p.cnt == 0 || second) { cp_async_commit(); return 0u; }  // no tile of this CTA in the item, or a shortcut chunk (loaded by TMA): nothing to copy
                uint32_t vm = 7u;
                const bool interior = tile.ty0 > 0 && tile.tx0 > 0 && tile.ty0 + TILE_H < a.H && tile.tx0 + TILE_W < a.W;
                if (interior && !centre_only) {
                    const uint32_t pix = ((uint32_t)tile.b * a.Hs + (uint32_t)(tile.ty0 >> up)) * a.Ws + (uint32_t)(tile.tx0 >> up);
                    const char* org = x_thread + ((size_t)pix * pixbytes - halo_off) + (uint32_t)(c0 * ESZ);
                    auto copy = [&](auto uc) {
                        constexpr int u = decltype(uc)::value;
                        const char* src = org + goffp[u];
                        cp_async16_at<u * NUM_PRODUCERS * 16, 0>(st_lo, src);
                        if (!IN_BF16) cp_async16_at<u * NUM_PRODUCERS * 16, 128>(st_hi, src);
                    };
                    copy(std::integral_constant<int, 0>{});
                    copy(std::integral_constant<int, 1>{});
                    copy(std::integral_constant<int, 2>{});
                    static_assert(BATCH == 3, "one copy call per entry");
                    cp_async_commit();
                    return 7u;
                }
                if (!interior || centre_only) {
                    vm = 0u;
#pragma unroll
                    for (int u = 0; u < BATCH; ++u) {
                        const int oy = tile.ty0 + (int)(pyx[u] & 0xffu) - 1, ox = tile.tx0 + (int)((pyx[u] >> 8) & 0xffu) - 1;
                        bool v = oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                        if (centre_only) v = v && (pyx[u] >> 16) != 0u;
                        vm |= (v ? 1u : 0u) << u;
                    }
                }
                {
                    const char* xb = (const char*)a.x
                        + ((((size_t)tile.b * a.Hs + (tile.ty0 >> up)) * a.Ws + (tile.tx0 >> up)) * a.Cin + c0 + (IN_BF16 ? j * 8 : j * 4)) * ESZ;
#pragma unroll
                    for (int u = 0; u < BATCH; ++u) {
                        const bool v = (vm >> u) & 1u;
                        const char* src = v ? xb + goff[u] : (const char*)a.x;
                        cp_async16(st_lo + (uint32_t)(u * NUM_PRODUCERS * 16), src, v ? 16u : 0u);
                        if (!IN_BF16) cp_async16(st_hi + (uint32_t)(u * NUM_PRODUCERS * 16), src + (v ? 128 : 0), v ? 16u : 0u);
                    }
                }
                cp_async_commit();
                return vm;
            };
            float sc[8], sh[8];
            auto load_affine = [&](const Pos& p) {               // GroupNorm scale/shift of the unit's channels
                if (!prologue || (X2 && p.kc >= kchunks)) return;
                // channels of v[0..3] and v[4..7] (see load_raw); the tiles of an item lie in one frame
                const int ca = p.kc * 64 + (IN_BF16 ? j * 8 : j * 4), cb = IN_BF16 ? ca + 4 : ca + 32;
                const float* ps = a.scale + (size_t)p.tile.b * a.Cin;
                const float* pt = a.shift + (size_t)p.tile.b * a.Cin;
                const float4 s0 = __ldg((const float4*)(ps + ca)), s1 = __ldg((const float4*)(ps + cb));
                const float4 t0 = __ldg((const float4*)(pt + ca)), t1 = __ldg((const float4*)(pt + cb));
                sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
                if (silu) {          // SiLU is evaluated as h + h*tanh(h) with h = v/2: the 1/2 folds into the affine map
#pragma unroll
                    for (int e = 0; e < 8; ++e) { sc[e] *= 0.5f; sh[e] *= 0.5f; }
                }
            };
            Pos nx;
            nx.t = sched.begin; nx.kc = 0; nx.slot = 0; nx.cnt = 1; nx.n = 1;
            bool have = nx.t < sched.end;
            uint32_t vm_next = 0u;
            if (have) {
                first_of_item(nx);
                vm_next = issue(nx);
                load_affine(nx);
            }
            while (have && ok) {
                const int cur_kc = nx.kc, cur_slot = nx.slot, cur_cnt = nx.cnt, cur_t = nx.t;
                const bool cur_have = cur_cnt > 0;               // without a tile the CTA still follows the barriers
                const uint32_t cur_vm = vm_next;
                const bool second = X2 && cur_kc >= kchunks;
                const bool pro = prologue;
                constexpr bool in_bf16 = IN_BF16;
                advance(nx);
                const bool have_next = nx.t < sched.end;
                cp_async_wait_all();                             // this thread's pieces of the current unit have landed
                Raw8 raw[BATCH];
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    raw[u].lo = lds_u4(st_lo + (uint32_t)(u * NUM_PRODUCERS * 16));
                    if (!in_bf16) raw[u].hi = lds_u4(st_hi + (uint32_t)(u * NUM_PRODUCERS * 16));
                }
                if (have_next) vm_next = issue(nx);              // the staging slots are free again: the next unit is on its way
                if (cur_slot == 0) {
                    ok = mbar_wait(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
                    if (!ok) break;
                    // a shortcut chunk: the stage will be filled by bulk tensor loads (one per tile of this CTA)
                    if (second && ptid == 0 && cur_have) mbar_expect_tx(smem_u32(&bars->a_full[stage]), (uint32_t)cur_cnt * SC_TILE_BYTES);
                }
                uint8_t* dst_tile = smem_a + stage * A_STAGE_BYTES + cur_slot * A_TILE_BYTES;
                if (second && ptid == 0 && cur_have) {
                    const Tile ct = sched.get(sched.index(cur_t, cur_slot), BN);
                    tma_load_4d(smem_u32(dst_tile), &tmap_x2, (cur_kc - kchunks) * 32, ct.tx0, ct.ty0, ct.b, smem_u32(&bars->a_full[stage]));
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    if (!cur_have || second) break;
                    uint32_t o0 = 0u, o1 = 0u, o2 = 0u, o3 = 0u;
                    if (cur_vm & (1u << u)) {
                        float v[8];
                        unpack_raw(in_bf16, raw[u], v);
                        if (pro) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], sc[e], sh[e]);
                            if (silu) {
#pragma unroll
                                for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], tanh_fast(v[e]), v[e]);
                            }
                        }
                        o0 = pack_bf16(v[0], v[1]); o1 = pack_bf16(v[2], v[3]); o2 = pack_bf16(v[4], v[5]); o3 = pack_bf16(v[6], v[7]);
                    }
                    if (in_bf16) {
                        *(uint4*)(dst_tile + soff[u]) = make_uint4(o0, o1, o2, o3);
                    } else {
                        const uint32_t so = soff[u];
                        *(uint2*)(dst_tile + so) = make_uint2(o0, o1);
                        *(uint2*)(dst_tile + (so ^ 64u)) = make_uint2(o2, o3);
                    }
                }
                if (cur_slot >= cur_cnt - 1) {
                    fence_proxy_async_smem();                    // generic-proxy stores -> visible to the tensor core
                    __syncwarp();
                    if (lane == 0) arrive_leader(&bars->a_full[stage]);
                    if (++stage == Cfg::A_STAGES) { stage = 0; phase ^= 1; }
                }
                if (have_next && (nx.kc != cur_kc || nx.t != cur_t)) load_affine(nx);
                have = have_next;
            }
            cp_async_wait_all();
        } else
        for (int t = sched.begin; t < sched.end && ok;) {
            const int n = sched.count(t);
            const int cnt = sched.mine(n);                   // 0: the peer of a two-CTA pair in an odd tail item
            const Tile tile0 = sched.get(cnt > 0 ? sched.index(t, 0) : t, BN);
            for (int kc = 0; kc < ktotal && ok; ++kc) {
                const bool second = X2 && kc >= kchunks;       // a shortcut chunk: loaded by TMA, nothing to transform
                const int c0 = kc * 64;
                constexpr bool centre_only = KS == 1;
                const bool pro = prologue && !second;
                float sc[8], sh[8];
                if (pro) {
                    // channels of v[0..3] and v[4..7] (see load_raw); the tiles of an item lie in one frame
                    const int ca = c0 + (IN_BF16 ? j * 8 : j * 4), cb = IN_BF16 ? ca + 4 : ca + 32;
                    const float* ps = a.scale + (size_t)tile0.b * a.Cin;
                    const float* pt = a.shift + (size_t)tile0.b * a.Cin;
                    const float4 s0 = __ldg((const float4*)(ps + ca)), s1 = __ldg((const float4*)(ps + cb));
                    const float4 t0 = __ldg((const float4*)(pt + ca)), t1 = __ldg((const float4*)(pt + cb));
                    sc[0] = s0.x; sc[1] = s0.y; sc[2] = s0.z; sc[3] = s0.w; sc[4] = s1.x; sc[5] = s1.y; sc[6] = s1.z; sc[7] = s1.w;
                    sh[0] = t0.x; sh[1] = t0.y; sh[2] = t0.z; sh[3] = t0.w; sh[4] = t1.x; sh[5] = t1.y; sh[6] = t1.z; sh[7] = t1.w;
                    if (silu) {          // SiLU is evaluated as h + h*tanh(h) with h = v/2: the 1/2 folds into the affine map
#pragma unroll
                        for (int e = 0; e < 8; ++e) { sc[e] *= 0.5f; sh[e] *= 0.5f; }
                    }
                }
#pragma unroll
                for (int slot = 0; slot < PAIR; ++slot) {
                    if (slot < max(cnt, 1)) {
                        const bool have = slot < cnt;        // without a tile the CTA still follows the barriers
                        Tile tile = tile0;                   // the second tile of an item is the next one in its channel block
                        if (slot == 1) {
                            tile.tx0 += TILE_W;
                            if (tile.tx0 >= sched.tiles_x * TILE_W) { tile.tx0 = 0; tile.ty0 += TILE_H; }
                        }
                        // which entries exist: all of them where the halo lies inside the image
                        uint32_t vm = 7u;
                        const bool interior = tile.ty0 > 0 && tile.tx0 > 0 && tile.ty0 + TILE_H < a.H && tile.tx0 + TILE_W < a.W;
                        if (!interior || centre_only) {
                            vm = 0u;
#pragma unroll
                            for (int u = 0; u < BATCH; ++u) {
                                const int oy = tile.ty0 + (int)(pyx[u] & 0xffu) - 1, ox = tile.tx0 + (int)((pyx[u] >> 8) & 0xffu) - 1;
                                bool v = oy >= 0 && oy < a.H && ox >= 0 && ox < a.W;
                                if (centre_only) v = v && (pyx[u] >> 16) != 0u;
                                vm |= (v ? 1u : 0u) << u;
                            }
                        }
                        if (!have || second) vm = 0u;
                        Raw8 raw[BATCH];
                        {
                            const char* xb = (const char*)a.x
                                + ((((size_t)tile.b * a.Hs + (tile.ty0 >> up)) * a.Ws + (tile.tx0 >> up)) * a.Cin + c0 + (IN_BF16 ? j * 8 : j * 4)) * ESZ;
#pragma unroll
                            for (int u = 0; u < BATCH; ++u)
                                if (vm & (1u << u)) load_raw_at(IN_BF16, xb + goff[u], raw[u]);
                        }
                        if (slot == 0) {
                            ok = mbar_wait<PH ? 256 : 0>(smem_u32(&bars->a_empty[stage]), phase ^ 1, abort_flag);
                            if (!ok) break;
                            if (second && ptid == 0 && cnt > 0) mbar_expect_tx(smem_u32(&bars->a_full[stage]), (uint32_t)cnt * SC_TILE_BYTES);
                        }
                        uint8_t* dst_tile = smem_a + stage * A_STAGE_BYTES + slot * A_TILE_BYTES;
                        if (second && ptid == 0 && have)
                            tma_load_4d(smem_u32(dst_tile), &tmap_x2, (kc - kchunks) * 32, tile.tx0, tile.ty0, tile.b, smem_u32(&bars->a_full[stage]));
                        constexpr bool in_bf16 = IN_BF16;
#pragma unroll
                        for (int u = 0; u < BATCH; ++u) {
                            if (!have || second) break;
                            uint32_t o0 = 0u, o1 = 0u, o2 = 0u, o3 = 0u;
                            if (vm & (1u << u)) {
                                float v[8];
                                unpack_raw(in_bf16, raw[u], v);
                                if (pro) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], sc[e], sh[e]);
                                    if (silu) {
#pragma unroll
                                        for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], tanh_fast(v[e]), v[e]);
                                    }
                                }
                                // phase form: fp16 operands (see pack_weight_phase_kernel); out-of-range values saturate
                                if (PH) { o0 = pack_f16(v[0], v[1]); o1 = pack_f16(v[2], v[3]); o2 = pack_f16(v[4], v[5]); o3 = pack_f16(v[6], v[7]); }
                                else { o0 = pack_bf16(v[0], v[1]); o1 = pack_bf16(v[2], v[3]); o2 = pack_bf16(v[4], v[5]); o3 = pack_bf16(v[6], v[7]); }
                            }
                            if (in_bf16) {
                                *(uint4*)(dst_tile + soff[u]) = make_uint4(o0, o1, o2, o3);
                            } else {
                                const uint32_t so = soff[u];
                                *(uint2*)(dst_tile + so) = make_uint2(o0, o1);
                                *(uint2*)(dst_tile + (so ^ 64u)) = make_uint2(o2, o3);
                            }
                        }
                    }
                }
                if (!ok) break;
                fence_proxy_async_smem();                    // generic-proxy stores -> visible to the tensor core
                __syncwarp();
                if (lane == 0) arrive_leader(&bars->a_full[stage]);
                if (++stage == Cfg::A_STAGES) { stage = 0; phase ^= 1; }
            }
            t += n;
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------ epilogue
        // Each warp owns a quarter of the accumulator rows (32 pixels = four rows of the 16x8 tile)
        // and works on its own: no synchronisation between the four warps.  TMEM reads are issued
        // one column block ahead of the one being processed.
        griddep_wait();
        const int ew = warp - EPI_WARP0;                     // TMEM lane quarter
        const bool reduce_add = a.residual != nullptr;       // y is the residual stream: the tile is added into it
        bool ok = true;
        int n_item = 0;
        uint32_t n_slice = 0;
        if (OUT_MODE == 2) {
            for (int t = sched.begin; t < sched.end && ok; ++n_item) {
                const int cnt = sched.count(t);
                const int buf = n_item % NBUF;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->acc_full[buf]), (n_item / NBUF) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                for (int slot = 0; slot < cnt; ++slot) {
                    const Tile tl = sched.get(t + slot, BN);
                    const int m = ew * 32 + lane;
                    const int oy = tl.ty0 + (m >> 3), ox = tl.tx0 + (m & 7);
                    uint32_t r[16];
                    tmem_ld16(tmem_base + (uint32_t)((buf * PAIR + slot) * Cfg::ACC_COLS) + ((uint32_t)(ew * 32) << 16), r);
                    tmem_ld_wait();
                    if (slot == cnt - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                    }
                    if (oy < a.H && ox < a.W) {
#pragma unroll
                        for (int co = 0; co < 16; ++co) {
                            if (co < a.Cout) {
                                const float v = __uint_as_float(r[co]) + (a.bias ? __ldg(a.bias + co) : 0.f);
                                const size_t o = (((size_t)tl.b * a.Cout + co) * a.H + oy) * a.W + ox;
                                if (a.out_u8) ((unsigned char*)a.y)[(((size_t)tl.b * a.H + oy) * a.W + ox) * a.Cout + co] = pack_u8(v);
                                else if (a.out_dtype == VD_BF16) ((__nv_bfloat16*)a.y)[o] = __float2bfloat16_rn(v);
                                else ((float*)a.y)[o] = v;
                            }
                        }
                    }
                }
                t += cnt;
            }
        } else {
            // The warp's 32 rows leave through shared memory as 128-byte-wide slices (32 fp32 or 64
            // bf16 channels), written row-per-lane in the 128B-swizzled layout of a bulk tensor
            // store of a [4 rows x 8 pixels x slice] box; the store clips the ragged image edge.
            constexpr int NP = BN / 32;                       // 32-column passes per tile
            constexpr int PPS = OUT_MODE == 1 ? 2 : 1;        // passes per 128-byte slice
            // One slice buffer per warp: before it is rewritten the warp waits until the store of the slice
            // before has read it out.  That wait is short against an item's MMAs, the epilogue is off the
            // critical path (two accumulator sets), and the shared memory saved is one more weight stage.
            uint8_t* wout = smem_out + ew * (Cfg::OUT_BUFS * WARP_SLICE_BYTES);
            float* wbias = (float*)(smem_bias) + ew * BN;                    // this warp's copy of the block's bias
            constexpr bool has_bias = BIAS || OUT_MODE == 2;
            int bias_n0 = -1;
            const uint64_t pol_out = l2_policy_evict_last();
            // statistics for the normalisation that follows: per-pass totals of the current (frame, channel block) run
            constexpr int NPS = NP > 0 ? NP : 1;
            constexpr bool stats = STATS && OUT_MODE == 1 && !PH && NP > 0;
            long long sacc[NPS];
#pragma unroll
            for (int p = 0; p < NPS; ++p) sacc[p] = 0;
            int stat_b = -1, stat_n0 = 0;
            constexpr int TAIL_BUFS = Cfg::SMEM_B / (4 * WARP_SLICE_BYTES) >= 2 ? Cfg::SMEM_B / (4 * WARP_SLICE_BYTES) : 2;
            for (int t = sched.begin; t < sched.end && ok; ++n_item) {
                const int n = sched.count(t);
                const int cnt = sched.mine(n);
                const int buf = n_item % NBUF;
                // (phase form: the weight stages stay in use while the first parities are drained)
                const bool last_item = !PH && t + n >= sched.end && Cfg::SMEM_B >= 8 * WARP_SLICE_BYTES;
                if (!PH) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->acc_full[buf]), (n_item / NBUF) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    if (cnt == 0) {                          // nothing of this CTA in the accumulators: hand them back at once
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) arrive_leader(&bars->acc_empty[buf]);
                    }
                }
                // sub-tiles of the item: its tiles, or (phase form) the four output parities of its one source tile
                const int nsub = PH ? 4 : cnt;
#pragma unroll 1
                for (int slot = 0; slot < nsub; ++slot) {
                    if (PH) {                                // parity `slot` is complete once its last tap has been committed
                        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->acc_full[slot]), n_item & 1, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                        if (cnt == 0) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) arrive_leader(&bars->acc_empty[slot]);
                            continue;
                        }
                    }
                    const Tile tl = sched.get(sched.index(t, PH ? 0 : slot), BN);
                    bool stat_valid = true;
                    if (stats) {
                        if (tl.b != stat_b || tl.n0 != stat_n0) {
                            if (stat_b >= 0) stat_flush<NPS>(a, sacc, stat_b, stat_n0, lane);
                            stat_b = tl.b; stat_n0 = tl.n0;
                        }
                        const int m = ew * 32 + lane;
                        stat_valid = tl.ty0 + (m >> 3) < a.H && tl.tx0 + (m & 7) < a.W;
                    }
                    if (has_bias && tl.n0 != bias_n0) {       // (re)load bias (+ shortcut bias) of this channel block
                        __syncwarp();
                        for (int i = lane; i < BN; i += 32)
                            wbias[i] = (a.bias ? __ldg(a.bias + tl.n0 + i) : 0.f) + ((X2 && a.bias2) ? __ldg(a.bias2 + tl.n0 + i) : 0.f);
                        bias_n0 = tl.n0;
                        __syncwarp();
                    }
                    const uint32_t tacc = tmem_base + (uint32_t)((buf * PAIR + slot) * Cfg::ACC_COLS) + ((uint32_t)(ew * 32) << 16);
                    const bool last_tile = PH || slot == cnt - 1;
                    const int acc_bar = PH ? slot : buf;
                    // A TMEM read queues behind the MMAs already issued (measured: its latency grows with the number of
                    // weight stages the MMA warp is ahead), so the round trips are what a drain costs.  Where the drain
                    // is on the critical path (phase form: no second accumulator set) two passes are read per round trip;
                    // elsewhere the next pass is in flight while one is processed.
                    constexpr bool PAIRED = PH;
                    uint32_t ra[32], rb[32];
                    tmem_ld32(tacc, ra);
                    if (PAIRED) tmem_ld32(tacc + 32u, rb);
                    tmem_ld_wait();
#pragma unroll
                    for (int p = 0; p < NP; ++p) {
                        uint32_t (&rc)[32] = (p & 1) ? rb : ra;          // this pass
                        uint32_t (&rn)[32] = (p & 1) ? ra : rb;          // next pass, in flight while this one is processed
                        if (!PAIRED && p + 1 < NP) tmem_ld32(tacc + (uint32_t)((p + 1) * 32), rn);
                        const int sl = p / PPS, h = p % PPS;              // slice, half of the slice
                        // The CTA's last item has the weight stages to itself (every MMA has completed): its slices go
                        // through a longer ring of buffers there, so the stores of the tail are not paced by buffer reuse.
                        uint8_t* obuf = last_item ? smem_b + (ew * TAIL_BUFS + (int)((n_slice + sl) % TAIL_BUFS)) * WARP_SLICE_BYTES
                                                  : wout + (int)((n_slice + sl) % Cfg::OUT_BUFS) * WARP_SLICE_BYTES;
                        if (h == 0) {
                            if (lane == 0) {                              // the store that last read this buffer is done
                                if (last_item) bulk_wait_group_read<TAIL_BUFS - 1>();
                                else bulk_wait_group_read<Cfg::OUT_BUFS - 1>();
                            }
                            __syncwarp();
                        }
                        uint8_t* orow = obuf + lane * 128;
                        const float4* bp = (const float4*)(wbias + p * 32);
                        if (OUT_MODE == 0) {
                            if (has_bias) {
#pragma unroll
                                for (int c = 0; c < 8; ++c) {
                                    const float4 tb = bp[c];
                                    *(float4*)(orow + ((c ^ (lane & 7)) << 4)) =
                                        make_float4(__uint_as_float(rc[4 * c]) + tb.x, __uint_as_float(rc[4 * c + 1]) + tb.y,
                                                    __uint_as_float(rc[4 * c + 2]) + tb.z, __uint_as_float(rc[4 * c + 3]) + tb.w);
                                }
                            } else {                              // the accumulator as it is (the bias is accounted for downstream)
#pragma unroll
                                for (int c = 0; c < 8; ++c)
                                    *(uint4*)(orow + ((c ^ (lane & 7)) << 4)) = make_uint4(rc[4 * c], rc[4 * c + 1], rc[4 * c + 2], rc[4 * c + 3]);
                            }
                        } else if (!stats && !has_bias) {
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                *(uint4*)(orow + (((h * 4 + c) ^ (lane & 7)) << 4)) =
                                    make_uint4(pack_bf16(__uint_as_float(rc[8 * c]), __uint_as_float(rc[8 * c + 1])),
                                               pack_bf16(__uint_as_float(rc[8 * c + 2]), __uint_as_float(rc[8 * c + 3])),
                                               pack_bf16(__uint_as_float(rc[8 * c + 4]), __uint_as_float(rc[8 * c + 5])),
                                               pack_bf16(__uint_as_float(rc[8 * c + 6]), __uint_as_float(rc[8 * c + 7])));
                        } else {
                            float v[8];
                            const bool stat_hi = (lane & 16) != 0;
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float4 t0 = bp[2 * c], t1 = bp[2 * c + 1];
                                const float f[8] = {__uint_as_float(rc[8 * c]) + t0.x, __uint_as_float(rc[8 * c + 1]) + t0.y,
                                                    __uint_as_float(rc[8 * c + 2]) + t0.z, __uint_as_float(rc[8 * c + 3]) + t0.w,
                                                    __uint_as_float(rc[8 * c + 4]) + t1.x, __uint_as_float(rc[8 * c + 5]) + t1.y,
                                                    __uint_as_float(rc[8 * c + 6]) + t1.z, __uint_as_float(rc[8 * c + 7]) + t1.w};
                                *(uint4*)(orow + (((h * 4 + c) ^ (lane & 7)) << 4)) =
                                    make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                                if (stats) {
                                    v[2 * c] = stat_quad_first(f[0], f[1], f[2], f[3], stat_valid, stat_hi);
                                    v[2 * c + 1] = stat_quad_first(f[4], f[5], f[6], f[7], stat_valid, stat_hi);
                                }
                            }
                            if (stats) sacc[p] += stat_reduce(v, lane);
                        }
                        if (PAIRED && (p & 1) && p + 1 < NP) {           // both buffers are free again: the next two passes
                            tmem_ld32(tacc + (uint32_t)((p + 1) * 32), ra);
                            tmem_ld32(tacc + (uint32_t)((p + 2) * 32), rb);
                        }
                        if (p + 1 < NP) {
                            if (!PAIRED || (p & 1)) tmem_ld_wait();
                        }
                        // accumulators fully read (the last read has landed in registers): hand them back.  The arrival
                        // carries no data (the reads are complete), so it need not wait for this warp's shared-memory stores.
                        if (last_tile && (PAIRED ? p == NP - 3 : p == NP - 1)) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) {
                                if (PAIRED && CG == 2) mbar_arrive_cluster_relaxed(map_to_cta(smem_u32(&bars->acc_empty[acc_bar]), 0));
                                else arrive_leader(&bars->acc_empty[acc_bar]);
                            }
                        }
                        if (h == PPS - 1) {
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                constexpr int CS = 32 * PPS;
                                // phase form: the tile is one parity of a 32x16 output block: rows 2i + a through the map of
                                // row parity a (tmap_y, tmap2), columns 2j + b through the map's parity coordinate
                                if (PH) tma_store_5d((slot >> 1) ? &tmap2 : &tmap_y, smem_u32(obuf), tl.n0 + sl * CS, slot & 1, tl.tx0, tl.ty0 + 4 * ew, tl.b, pol_out);
                                else if (reduce_add) tma_reduce_add_4d(&tmap_y, smem_u32(obuf), tl.n0 + sl * CS, tl.tx0, tl.ty0 + 4 * ew, tl.b, pol_out);
                                else tma_store_4d(&tmap_y, smem_u32(obuf), tl.n0 + sl * CS, tl.tx0, tl.ty0 + 4 * ew, tl.b, pol_out);
                                bulk_commit_group();
                            }
                        }
                    }
                    n_slice += NP / PPS;
                }
                t += n;
            }
            if (stats && stat_b >= 0) stat_flush<NPS>(a, sacc, stat_b, stat_n0, lane);
            if (stats) __threadfence();
            if (lane == 0) bulk_wait_group<0>();             // all stores have landed before the CTA retires
        }
    } else if (warp == TMA_WARP) {
        // ------------------------------------------------ weight loads (TMA)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int t = sched.begin; t < sched.end && ok; t += sched.count(t)) {
                const Tile tl = sched.get(t, BN);
                if constexpr (PH) break;                 // the phase form streams its weights in PhaseSched order, below
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool second = X2 && kc >= kchunks;
                    const int ntap = second ? 1 : taps;
                    for (int tap = 0; tap < ntap; ++tap) {
                        if (stage % Cfg::B_GROUP == 0) {     // stages come back in groups (see the MMA thread)
                            ok = mbar_wait(smem_u32(&bars->b_empty[stage / Cfg::B_GROUP]), phase ^ 1, abort_flag);
                            if (!ok) break;
                        }
                        const uint32_t dst = smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES);
                        if (CG == 2) {       // this CTA's half of the rows; completion is reported to the leader's barrier
                            const uint32_t full = leader_bar(&bars->b_full[stage]);
                            const int row0 = tl.n0 + (int)rank * (BN / 2);
                            mbar_arrive_expect_tx_cluster(full, Cfg::B_STAGE_BYTES);
                            if (second) tma_load_2d_pair(dst, &tmap2, (kc - kchunks) * 32, row0, full);
                            else tma_load_2d_pair(dst, &tmap, kc * 64, tap * cout_pad + row0, full);
                        } else {
                            const uint32_t full = smem_u32(&bars->b_full[stage]);
                            mbar_arrive_expect_tx(full, Cfg::B_STAGE_BYTES);
                            if (second) tma_load_2d(dst, &tmap2, (kc - kchunks) * 32, tl.n0, full);
                            else tma_load_2d(dst, &tmap, kc * 64, tap * cout_pad + tl.n0, full);
                        }
                        ++issued;
                        if (++stage == Cfg::B_STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if constexpr (PH) {
                // two stages per (parity, chunk) block: dy = 0, 1, each with the taps dx = 0, 1 of this CTA's 64
                // output channels as one box of 128 rows (the packed layout keeps them adjacent)
                int nitems = 0;
                for (int t = sched.begin; t < sched.end; t += sched.count(t)) ++nitems;
                PhaseSched ps; ps.init(kchunks, nitems);
                int blk_of[2] = {0, 0};                      // channel block of the item (index & 1)
                int t_next = sched.begin;
                for (int s = 0; s < ps.steps() && ok; ++s) {
                    if (s < ps.S && s == ps.item_of(s) * ps.K) {         // a new item starts in this step
                        blk_of[ps.item_of(s) & 1] = sched.get(t_next, BN).n0 / BN;
                        t_next += sched.count(t_next);
                    }
                    const int r = ps.rot(s);
                    for (int j = 0; j < 4 && ok; ++j) {
                        const int p = (r + j) & 3, q = s - p * ps.lag;
                        if (q < 0 || q >= ps.S) continue;
                        const int it = ps.item_of(q), kc = q - it * ps.K;
                        for (int dy = 0; dy < 2; ++dy) {
                            ok = mbar_wait(smem_u32(&bars->b_empty[stage]), phase ^ 1, abort_flag);
                            if (!ok) break;
                            const uint32_t dst = smem_u32(smem_b + stage * Cfg::B_STAGE_BYTES);
                            const uint32_t full = leader_bar(&bars->b_full[stage]);
                            mbar_arrive_expect_tx_cluster(full, Cfg::B_STAGE_BYTES);
                            tma_load_2d_pair(dst, &tmap, kc * 64, (((2 * p + dy) * sched.nblk + blk_of[it & 1]) * 2 + (int)rank) * 128, full);
                            ++issued;
                            if (++stage == Cfg::B_STAGES) { stage = 0; phase ^= 1; }
                        }
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
    } else if (warp == MMA_WARP && rank == 0) {
        // ------------------------------------------------ MMA issue
        // The whole warp runs the loop and one elected lane issues: in warp-uniform code the
        // compiler keeps descriptors and counters in uniform registers, and the issue sequence of
        // wait / 4 x tcgen05.mma / commit costs about 300 cycles instead of about 480 from a
        // single-lane branch (measured), which a tap's 513 tensor cycles then hide.  Where an item
        // is two tiles the warp issues for both.
        {
            const bool leader = elect_one() != 0u;
            constexpr uint32_t idesc = PH ? make_idesc_f16(128 * CG, BN) : make_idesc_bf16(128 * CG, BN);
            const uint32_t a_hi = desc_hi(PW * 128, 2), b_hi = desc_hi(1024, 2);
            const uint32_t a_lo0 = desc_lo(smem_u32(smem_a)), b_lo0 = desc_lo(smem_u32(smem_b));
            // one MMA of the pair (M = 256 over both CTAs) or of this CTA; a commit to both CTAs or to this one
            auto mma = [&](uint32_t d, uint32_t alo, uint32_t blo, uint32_t accum) {
                if (CG == 2) umma2_bf16_split(d, alo, a_hi, blo, b_hi, idesc, accum);
                else umma_bf16_split(d, alo, a_hi, blo, b_hi, idesc, accum);
            };
            // the same, predicated on the elected lane (no branch: see umma_bf16_split_on)
            const uint32_t lead = leader ? 1u : 0u;
            auto mma_on = [&](uint32_t d, uint32_t alo, uint32_t blo, uint32_t accum) {
                if (CG == 2) umma2_bf16_split_on(d, alo, a_hi, blo, b_hi, idesc, accum, lead);
                else umma_bf16_split_on(d, alo, a_hi, blo, b_hi, idesc, accum, lead);
            };
            auto commit_on = [&](uint32_t bar) {
                if (CG == 2) umma2_commit_both_on(bar, lead);
                else umma_commit_on(bar, lead);
            };
            auto commit = [&](uint64_t* b) {
                if (CG == 2) umma2_commit_both(smem_u32(b));
                else umma_commit(smem_u32(b));
            };
            uint32_t as = 0, aph = 0, bs = 0, bph = 0;
            bool ok = true;
            int n_item = 0;
            // Where a tap's four (eight) MMAs take 512 tensor cycles, the issuing warp has about 100 cycles
            // to spare per tap (measured in isolation: wait + 8 MMAs + commit cost about 400), and none at
            // the chunk and item boundaries.  So the common form (one issuing warp, one weight stage per
            // commit; this CTA always has a tile then) runs a loop of its own: no votes (a wait that gave
            // up leaves garbage behind that nobody reads; the abort flag is looked at once per item), the
            // three taps of a kernel row unrolled so that their operand offsets are immediates, and every
            // running index an addition in uniform registers.
            constexpr bool FAST = Cfg::B_GROUP == 1;
            if constexpr (FAST) {
                const uint32_t b_full0 = smem_u32(&bars->b_full[0]), b_empty0 = smem_u32(&bars->b_empty[0]);
                auto wait_on = [&](uint32_t bar, uint32_t ph) {
                    if (!mbar_try_wait(bar, ph)) (void)mbar_wait(bar, ph, abort_flag);
                    tc_fence_after();
                };
                // one tap: its weight stage, the MMAs of the item's tile(s), the stage handed back
                auto tap_step = [&](auto two_c, uint32_t td, uint32_t a_lo, uint32_t acc0) {
                    constexpr bool TWO = decltype(two_c)::value;
                    wait_on(b_full0 + bs * 8u, bph);
                    const uint32_t b_lo = b_lo0 + bs * (uint32_t)(Cfg::B_STAGE_BYTES >> 4);
                    mma_on(td, a_lo, b_lo, acc0);
                    mma_on(td, a_lo + 2, b_lo + 2, 1u);
                    mma_on(td, a_lo + 4, b_lo + 4, 1u);
                    mma_on(td, a_lo + 6, b_lo + 6, 1u);
                    if (TWO) {
                        const uint32_t td2 = td + Cfg::ACC_COLS, a2 = a_lo + (A_TILE_BYTES >> 4);
                        mma_on(td2, a2, b_lo, acc0);
                        mma_on(td2, a2 + 2, b_lo + 2, 1u);
                        mma_on(td2, a2 + 4, b_lo + 4, 1u);
                        mma_on(td2, a2 + 6, b_lo + 6, 1u);
                    }
                    commit_on(b_empty0 + bs * 8u);
                    __syncwarp();
                    if (++bs == (uint32_t)Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                };
                // a shortcut sub-chunk: fp32 operands (dense 128-row tile, eight-row groups 1024 bytes apart; fp32 weight
                // stage), four kind::tf32 MMAs of K = 8 per tile
                auto shortcut_step = [&](auto two_c, uint32_t td, uint32_t a_lo) {
                    constexpr bool TWO = decltype(two_c)::value;
                    constexpr uint32_t idesc_tf32 = make_idesc_tf32(128, BN);
                    const uint32_t a_hi_dense = desc_hi(1024, 2);
                    wait_on(b_full0 + bs * 8u, bph);
                    const uint32_t b_lo = b_lo0 + bs * (uint32_t)(Cfg::B_STAGE_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_tf32_split_on(td, a_lo + 2 * k, a_hi_dense, b_lo + 2 * k, b_hi, idesc_tf32, 1u, lead);
                    if (TWO) {
                        const uint32_t td2 = td + Cfg::ACC_COLS, a2 = a_lo + (A_TILE_BYTES >> 4);
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_tf32_split_on(td2, a2 + 2 * k, a_hi_dense, b_lo + 2 * k, b_hi, idesc_tf32, 1u, lead);
                    }
                    commit_on(b_empty0 + bs * 8u);
                    __syncwarp();
                    if (++bs == (uint32_t)Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                };
                auto item = [&](auto two_c, uint32_t td, int buf) {
                    uint32_t acc = 0;                         // the first MMA of an item overwrites the accumulator
#pragma unroll 1
                    for (int kc = 0; kc < ktotal; ++kc) {
                        constexpr bool centre = KS == 1;                         // single centre tap
                        wait_on(smem_u32(&bars->a_full[as]), aph);
                        uint32_t a_row = a_lo0 + as * (A_STAGE_BYTES >> 4);
                        if (X2 && kc >= kchunks) {
                            if constexpr (CG == 1 && X2) shortcut_step(two_c, td, a_row);       // (always after the main chunks: accumulates)
                        } else if (!centre) {
#pragma unroll 1
                            for (int ky = 0; ky < 3; ++ky) {
                                tap_step(two_c, td, a_row, acc);
                                tap_step(two_c, td, a_row + 8, 1u);
                                tap_step(two_c, td, a_row + 16, 1u);
                                acc = 1u;
                                a_row += PW * 8;
                            }
                        } else {
                            tap_step(two_c, td, a_row + (PW + 1) * 8, acc);
                            acc = 1u;
                        }
                        commit_on(smem_u32(&bars->a_empty[as]));
                        __syncwarp();
                        if (++as == Cfg::A_STAGES) { as = 0; aph ^= 1; }
                    }
                    commit_on(smem_u32(&bars->acc_full[buf]));
                    __syncwarp();
                };
                // phase form: (parity, chunk) blocks in PhaseSched order.  Parity p = 2a + b accumulates in columns
                // [128p, 128p + 128), waits for its own "empty" barrier before an item's first chunk and reports
                // "full" after its last; an operand stage goes back once parity 3 (which lags most) has used it
                if constexpr (PH) {
                    int nitems = 0;
                    for (int t = sched.begin; t < sched.end; t += sched.count(t)) ++nitems;
                    PhaseSched ps; ps.init(kchunks, nitems);
#pragma unroll 1
                    for (int s = 0; s < ps.steps(); ++s) {
                        if (*abort_flag) break;
                        const int r = ps.rot(s);
#pragma unroll 1
                        for (int j = 0; j < 4; ++j) {
                            const int p = (r + j) & 3, q = s - p * ps.lag;
                            if (q < 0 || q >= ps.S) continue;
                            const int it = ps.item_of(q), kc = q - it * ps.K;
                            const uint32_t st = (uint32_t)q % (uint32_t)Cfg::A_STAGES;
                            if (p == 0) wait_on(smem_u32(&bars->a_full[st]), ((uint32_t)q / (uint32_t)Cfg::A_STAGES) & 1u);
                            const bool first = kc == 0, last = kc == ps.K - 1;
                            if (first) wait_on(smem_u32(&bars->acc_empty[p]), (uint32_t)((it & 1) ^ 1));
                            const uint32_t td = tmem_base + (uint32_t)(p * Cfg::ACC_COLS);
                            const uint32_t a_view = a_lo0 + st * (uint32_t)(A_STAGE_BYTES >> 4) + (uint32_t)(((p >> 1) * PW + (p & 1)) * 8);
#pragma unroll
                            for (int dy = 0; dy < 2; ++dy) {
                                wait_on(b_full0 + bs * 8u, bph);
                                const uint32_t b_lo = b_lo0 + bs * (uint32_t)(Cfg::B_STAGE_BYTES >> 4);
                                const uint32_t a_lo = a_view + (uint32_t)(dy * PW * 8);
                                mma_on(td, a_lo, b_lo, (first && dy == 0) ? 0u : 1u);
                                mma_on(td, a_lo + 2, b_lo + 2, 1u);
                                mma_on(td, a_lo + 4, b_lo + 4, 1u);
                                mma_on(td, a_lo + 6, b_lo + 6, 1u);
                                constexpr uint32_t B_TAP = (uint32_t)(Cfg::B_STAGE_BYTES >> 5);     // second tap of the stage
                                mma_on(td, a_lo + 8, b_lo + B_TAP, 1u);
                                mma_on(td, a_lo + 10, b_lo + B_TAP + 2, 1u);
                                mma_on(td, a_lo + 12, b_lo + B_TAP + 4, 1u);
                                mma_on(td, a_lo + 14, b_lo + B_TAP + 6, 1u);
                                commit_on(b_empty0 + bs * 8u);
                                __syncwarp();
                                if (++bs == (uint32_t)Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                            }
                            if (last) {
                                commit_on(smem_u32(&bars->acc_full[p]));
                                __syncwarp();
                            }
                            if (p == 3) {
                                commit_on(smem_u32(&bars->a_empty[st]));
                                __syncwarp();
                            }
                        }
                    }
                } else
                for (int t = sched.begin; t < sched.end; ++n_item) {
                    const int n = sched.count(t);
                    const int buf = n_item % NBUF;
                    wait_on(smem_u32(&bars->acc_empty[buf]), ((n_item / NBUF) & 1) ^ 1);
                    if (*abort_flag) break;
                    const uint32_t td = tmem_base + (uint32_t)(buf * PAIR * Cfg::ACC_COLS);
                    if (PAIR == 2 && sched.mine(n) == 2) item(std::true_type{}, td, buf);
                    else item(std::false_type{}, td, buf);
                    t += n;
                }
            } else
            for (int t = sched.begin; t < sched.end && ok; ++n_item) {
                const int n = sched.count(t);
                const int cnt = sched.mine(n);
                const bool active = cnt > 0;
                const int buf = n_item % NBUF;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->acc_empty[buf]), ((n_item / NBUF) & 1) ^ 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                const uint32_t td = tmem_base + (uint32_t)(buf * PAIR * Cfg::ACC_COLS);
                uint32_t acc = 0;                             // the first MMA of an item overwrites the accumulator
                for (int kc = 0; kc < ktotal && ok; ++kc) {
                    const bool centre = (X2 && kc >= kchunks) || KS == 1;            // single centre tap
                    const int ntap = centre ? 1 : 9;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->a_full[as]), aph, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    // tap view: rows start (ky*PW + kx) pixels into the halo tile; eight-row groups are
                    // one tile row (PW pixels) apart.  The tensor core applies the 128-byte swizzle to the
                    // absolute shared-memory address, so any 128-byte-aligned start works (base_offset 0).
                    uint32_t a_lo = a_lo0 + as * (A_STAGE_BYTES >> 4) + (centre ? (PW + 1) * 8 : 0);   // + (ky*PW + kx) * 128 B >> 4
                    int kx = 0;
                    for (int tap = 0; tap < ntap; ++tap) {
                        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->b_full[bs]), bph, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t b_lo = b_lo0 + bs * (Cfg::B_STAGE_BYTES >> 4);
                        if (leader) {
                            if (active) {
                                mma(td, a_lo, b_lo, acc);
                                mma(td, a_lo + 2, b_lo + 2, 1u);
                                mma(td, a_lo + 4, b_lo + 4, 1u);
                                mma(td, a_lo + 6, b_lo + 6, 1u);
                                if (PAIR == 2 && cnt == 2) {       // one warp issues for both tiles
                                    const uint32_t td2 = td + Cfg::ACC_COLS, a2 = a_lo + (A_TILE_BYTES >> 4);
                                    mma(td2, a2, b_lo, acc);
                                    mma(td2, a2 + 2, b_lo + 2, 1u);
                                    mma(td2, a2 + 4, b_lo + 4, 1u);
                                    mma(td2, a2 + 6, b_lo + 6, 1u);
                                }
                            }
                            // weight stages are handed back B_GROUP at a time (fewer commits)
                            if (bs % Cfg::B_GROUP == Cfg::B_GROUP - 1) {
                                if (active) commit(&bars->b_empty[bs / Cfg::B_GROUP]);
                                else mbar_arrive(smem_u32(&bars->b_empty[bs / Cfg::B_GROUP]));
                            }
                        }
                        __syncwarp();
                        acc = 1u;
                        if (++bs == Cfg::B_STAGES) { bs = 0; bph ^= 1; }
                        if (++kx == 3) { kx = 0; a_lo += (PW - 2) * 8; } else a_lo += 8;
                    }
                    if (leader) {
                        if (active) commit(&bars->a_empty[as]);
                        else mbar_arrive(smem_u32(&bars->a_empty[as]));
                    }
                    __syncwarp();
                    if (++as == Cfg::A_STAGES) { as = 0; aph ^= 1; }
                }
                if (ok && leader) {
                    if (active) commit(&bars->acc_full[buf]);
                    else mbar_arrive(smem_u32(&bars->acc_full[buf]));
                }
                __syncwarp();
                t += n;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                         // nobody leaves while the pair may still touch its memory
    if (tid == 0 && bars->abort_flag && status) {
        if (atomicCAS(status, 0u, kStatusConvTimeout) == 0u) {
            status[1] = blockIdx.x;
            status[2] = (uint32_t)BN;
        }
    }
    if (warp == MMA_WARP) {
        tc_fence_after();
        if (CG == 2) tmem_dealloc2(tmem_base, (uint32_t)Cfg::TMEM_COLS);
        else tmem_dealloc(tmem_base, (uint32_t)Cfg::TMEM_COLS);
    }
    if (STATS && OUT_MODE == 1) {
        // every sum of this CTA has been added (and fenced) before the barrier above
        if (tid == 0) {
            __threadfence();
            bars->stat_last = atomicAdd(a.stat_counter, 1u) == gridDim.x - 1u ? 1u : 0u;
        }
        __syncthreads();
        const bool last = bars->stat_last != 0u;
        __syncthreads();
        if (last) {
            __threadfence();
            stat_finalize(a, tid, smem);
            if (tid == 0) *a.stat_counter = 0u;              // ready for the next launch
        }
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

// Phase-collapsed upsampling convolution: OIHW 3x3 -> bf16 rows of Cin, ordered
// [stage = 2 * parity + dy][128-channel block][CTA rank][dx][64 channels], parity = 2a + b, so that the two
// column taps of one (parity, dy) for one CTA's half of a channel block are one box of 128 rows.
// The weight at (parity (a, b), dy, dx) is the sum of the 3x3 taps (ky, kx) that read the same source
// pixel: a = 0: dy 0 <- ky {0}, dy 1 <- ky {1, 2};  a = 1: dy 0 <- ky {0, 1}, dy 1 <- ky {2};  columns alike.
// The sum is formed in fp32 in a fixed order and rounded once, to FP16, and the kernel converts the
// activation operand of these layers to fp16 as well (same tensor rate as bf16): a sum of up to four bf16
// weights is not a bf16 number, and rounding it to bf16 would add a second 2^-9 error per product to these
// layers; fp16 rounds both operands eight times finer instead (magnitudes are far inside its range: weights
// below 1, activations saturate at 65504; a sum below 2^-14 is rounded with an absolute error of at most 2^-25).
// Both operands of one tcgen05.mma kind::f16 must have the same format: fp16 weights beside bf16 activations
// are an illegal instruction on this device.
template <typename T>
__global__ void pack_weight_phase_kernel(const T* w, __half* packed, int Cout, int Cin) {
    const int64_t total = (int64_t)16 * Cout * Cin;
    const int nblk = Cout / 128;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % Cin);
        const int o = (int)((i / Cin) % Cout);
        const int tap = (int)(i / ((int64_t)Cin * Cout));          // 0..15: parity * 4 + dy * 2 + dx
        const int par = tap >> 2, dy = (tap >> 1) & 1, dx = tap & 1;
        const int pa = par >> 1, pb = par & 1;
        const int ky0 = pa == 0 ? (dy == 0 ? 0 : 1) : (dy == 0 ? 0 : 2), ky1 = pa == 0 ? (dy == 0 ? 0 : 2) : (dy == 0 ? 1 : 2);
        const int kx0 = pb == 0 ? (dx == 0 ? 0 : 1) : (dx == 0 ? 0 : 2), kx1 = pb == 0 ? (dx == 0 ? 0 : 2) : (dx == 0 ? 1 : 2);
        float v = 0.f;
        for (int ky = ky0; ky <= ky1; ++ky)
            for (int kx = kx0; kx <= kx1; ++kx) {
                const size_t j = ((size_t)o * Cin + c) * 9 + ky * 3 + kx;
                v += sizeof(T) == 2 ? __bfloat162float(((const __nv_bfloat16*)w)[j]) : ((const float*)w)[j];
            }
        const int st = par * 2 + dy, blk = o / 128, rk = (o % 128) / 64, r = o % 64;
        const size_t row = ((((size_t)st * nblk + blk) * 2 + rk) * 2 + dx) * 64 + r;
        packed[row * Cin + c] = __float2half_rn(v);
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
int pick_bn(int Cout) {
    return (Cout % 128 != 0) ? 16 : ((Cout % 256 == 0) ? 256 : 128);
}

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

// clusters of two CTAs of this kernel that the device can hold at once (0: the form cannot run)
template <typename K>
int max_pairs(K kern, int smem) {
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
    if (cudaOccupancyMaxActiveClusters(&n, (const void*)kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

// Per-device launch state of one kernel instantiation (the shared-memory attribute is per device, and
// so is the number of CTA pairs that can be resident), looked up once per device under a lock.
constexpr int kMaxDevices = 64;
std::mutex g_launch_mu;
struct KernelState { bool configured[kMaxDevices]; int pairs[kMaxDevices]; int sms[kMaxDevices]; };

template <typename K>
cudaError_t kernel_state(K kern, int smem, int cg, KernelState& st, int* pairs, int* sms) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_launch_mu);
    if (!st.configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        st.sms[dev] = n;
        st.pairs[dev] = cg == 2 ? max_pairs(kern, smem) : 0;
        st.configured[dev] = true;
    }
    *pairs = st.pairs[dev];
    *sms = st.sms[dev];
    return cudaSuccess;
}

template <int BN, bool IB, int OM, int CG, bool PH = false, bool STATS = false, bool BIAS = true, bool X2 = false, int KS = 3>
cudaError_t launch_one(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    auto kern = conv_tc_kernel<BN, IB, OM, CG, PH, STATS, BIAS, X2, KS>;
    constexpr int SMEM = TileCfg<BN, CG, PH, IB>::SMEM_TOTAL;
    static KernelState state = {};
    int pairs = 0, sms = 0;
    cudaError_t e = kernel_state(kern, SMEM, CG, state, &pairs, &sms);
    if (e != cudaSuccess) return e;
    if (CG == 2 && pairs < 1) return cudaErrorInvalidConfiguration;
    // The phase form tiles the SOURCE grid (its four parities cover the 2x output): the kernel sees a
    // stride-1 convolution at the source resolution; only its output maps know about the 2x grid.
    ConvArgs ka = a;
    if (PH) { ka.H = a.Hs; ka.W = a.Ws; ka.upsample = 0; }
    const int tiles = ((ka.W + TILE_W - 1) / TILE_W) * ((ka.H + TILE_H - 1) / TILE_H);
    const long long total = (long long)tiles * (padded_cout(a.Cout) / BN) * a.B;
    int grid;
    if (CG == 2) grid = 2 * (int)std::min<long long>((total + 1) / 2, std::min(pairs, kConvMaxCtas / 2));
    else grid = (int)std::min<long long>(total, std::min(sms, kConvMaxCtas));
    // reciprocals for the kernel's tile numbering (see Sched)
    {
        const int tiles_x = (ka.W + TILE_W - 1) / TILE_W, nblk = padded_cout(a.Cout) / BN;
        const int dmax = std::max(tiles, std::max(tiles_x, nblk));
        if ((unsigned long long)total * (unsigned long long)std::max(dmax, grid + 1) >= (1ull << 32)) return cudaErrorInvalidValue;
        auto recip = [](int d) { return d == 1 ? 0u : (unsigned int)(((1ull << 32) + (unsigned long long)d - 1) / (unsigned long long)d); };
        ka.div_tiles = recip(tiles); ka.div_nblk = recip(nblk); ka.div_tx = recip(tiles_x);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (pdl_enabled()) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (CG == 2) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, ka, *(const CUtensorMap*)plan.tmap, *(const CUtensorMap*)plan.tmap2,
                              *(const CUtensorMap*)plan.tmap_y, *(const CUtensorMap*)plan.tmap_x2, status);
}

// can this device co-schedule the CTA pairs of the two-CTA kernels?  (looked up once per device)
bool pairs_available() {
    static KernelState state = {};
    int pairs = 0, sms = 0;
    auto k = conv_tc_kernel<256, false, 1, 2>;
    if (kernel_state(k, TileCfg<256, 2>::SMEM_TOTAL, 2, state, &pairs, &sms) != cudaSuccess) { cudaGetLastError(); return false; }
    return pairs >= 1;
}

}  // namespace

bool conv_tc_supported(const ConvArgs& a) {
    if (a.Cin % 64 != 0 || a.Cin < 64) return false;
    if (!a.bf16_operands) return false;
    if (a.ksize != 1 && a.ksize != 3) return false;
    if (a.ksize == 1 && (a.upsample || a.Cout % 128 != 0)) return false;       // 1x1: plain layers of 128-channel blocks
    if (a.x2 && (a.Cin2 % 32 != 0 || a.Cin2 < 32 || a.upsample || a.ksize != 3 || a.in_dtype != VD_BF16 || a.out_dtype != VD_F32 || a.Cout % 128 != 0)) return false;
    if (a.upsample == 2)     // phase-collapsed form: 3x3, 128-channel blocks, plain NHWC store
        return a.ksize == 3 && a.Cout % 128 == 0 && !a.out_nchw && !a.residual && !a.x2;
    if (a.Cout % 128 == 0) return !a.out_nchw && !a.out_u8;
    return a.Cout <= 16 && (a.out_nchw || a.out_u8) && !a.residual && !a.x2;      // the frame head: Cout padded to 16
}

// Layers whose epilogue can take the statistics of the following GroupNorm: the tile passes through the epilogue's
// registers as its final value (no residual added by the memory system), 32 groups at most, groups of 4, 8 or 16 channels.
bool conv_tc_stats_supported(const ConvArgs& a, int groups) {
    if (!conv_tc_supported(a) || a.Cout % 128 != 0 || a.upsample == 2 || a.residual) return false;
    if (a.out_dtype != VD_BF16) return false;
    if (groups < 1 || groups > 32 || a.Cout % groups != 0) return false;
    const int cpg = a.Cout / groups;
    return cpg == 4 || cpg == 8 || cpg == 16;
}

bool conv_tc_pairs_available() { return pairs_available(); }

size_t conv_tc_packed_bytes(int Cout, int Cin, int taps, bool phase) {
    return phase ? (size_t)16 * Cout * Cin * 2 : (size_t)taps * padded_cout(Cout) * Cin * 2;
}

cudaError_t launch_pack_weight_tc(const void* w, int w_dtype, void* packed, int Cout, int Cin, int taps, int cout_total,
                                  int cout_offset, bool phase, cudaStream_t s) {
    if (phase) {
        if (taps != 9 || cout_offset != 0 || cout_total != Cout || Cout % 128 != 0) return cudaErrorInvalidValue;
        const int64_t n = (int64_t)16 * Cout * Cin;
        const int grid = (int)std::min<int64_t>((n + 255) / 256, 148 * 16);
        if (w_dtype == VD_BF16) pack_weight_phase_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)w, (__half*)packed, Cout, Cin);
        else pack_weight_phase_kernel<float><<<grid, 256, 0, s>>>((const float*)w, (__half*)packed, Cout, Cin);
        return cudaGetLastError();
    }
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
    const bool phase = a.upsample == 2;
    const int bn = phase ? 128 : pick_bn(a.Cout);
    // 256-channel blocks of the folded upsampling form and the phase form run as two-CTA pairs (each CTA loads
    // half of the rows of a weight tile); the device must be able to co-schedule such pairs
    int cg = (phase || (bn == 256 && a.upsample)) ? 2 : 1;
    if (cg == 2 && !pairs_available()) {
        if (phase) return cudaErrorInvalidConfiguration;     // the phase form has no one-CTA variant
        cg = 1;
    }
    plan->cg = cg;
    plan->phase = phase ? 1 : 0;
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const bool ob = a.out_dtype == VD_BF16;
    const cuuint64_t es = ob ? 2 : 4;
    if (phase) {
        // weights: 16 * Cout rows in the order pack_weight_phase_kernel writes; one box = a stage of this CTA
        if (!encode_weights((CUtensorMap*)plan->tmap, a.w, a.Cin, 16 * a.Cout, 128)) return cudaErrorInvalidValue;
        // output [B][2 Hs][2 Ws][Cout] seen per row parity a as a 5-D tensor (channel, column parity b, source
        // column j, source row i, frame): element (c, b, j, i, n) is output pixel (2i + a, 2j + b).  A box is one
        // epilogue warp's four source rows x 8 source columns of one parity; the store clips the ragged edge.
        const cuuint64_t W = (cuuint64_t)a.W, C = (cuuint64_t)a.Cout;
        const cuuint64_t dims[5] = {C, 2, (cuuint64_t)a.Ws, (cuuint64_t)a.Hs, (cuuint64_t)std::max(a.B, 1)};
        const cuuint64_t strides[4] = {C * es, 2 * C * es, 2 * W * C * es, (cuuint64_t)a.H * W * C * es};
        const cuuint32_t box[5] = {ob ? 64u : 32u, 1, (cuuint32_t)TILE_W, 4, 1};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        for (int pa = 0; pa < 2; ++pa) {
            void* base = (char*)a.y + (size_t)pa * W * C * es;
            if (enc((CUtensorMap*)(pa ? plan->tmap2 : plan->tmap_y), ob ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                    5, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
        }
        memcpy(plan->tmap_x2, plan->tmap, sizeof(plan->tmap));
        plan->bn = bn;
        plan->batch = a.B;
        plan->y = a.y;
        plan->valid = 1;
        return cudaSuccess;
    }
    if (!encode_weights((CUtensorMap*)plan->tmap, a.w, a.Cin, taps * padded_cout(a.Cout), bn / cg)) return cudaErrorInvalidValue;
    memcpy(plan->tmap2, plan->tmap, sizeof(plan->tmap));
    memcpy(plan->tmap_x2, plan->tmap, sizeof(plan->tmap));
    if (a.x2) {
        if (cg != 1) return cudaErrorInvalidValue;           // the fused shortcut exists in the one-CTA forms
        // shortcut weights fp32 [Cout][Cin2] (one box = a weight stage: BN rows of 32 channels = 128 bytes)
        const cuuint64_t wd[2] = {(cuuint64_t)a.Cin2, (cuuint64_t)a.Cout};
        const cuuint64_t ws[1] = {(cuuint64_t)a.Cin2 * 4};
        const cuuint32_t wb[2] = {32, (cuuint32_t)bn};
        const cuuint32_t one2[2] = {1, 1};
        if (enc((CUtensorMap*)plan->tmap2, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(a.w2), wd, ws, wb, one2,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        // shortcut input fp32 NHWC [B][H][W][Cin2]; one box = a tile of 16 x 8 pixels x 32 channels, zero beyond the image
        const cuuint64_t xd[4] = {(cuuint64_t)a.Cin2, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)std::max(a.B, 1)};
        const cuuint64_t xs[3] = {(cuuint64_t)a.Cin2 * 4, (cuuint64_t)a.W * a.Cin2 * 4, (cuuint64_t)a.H * a.W * a.Cin2 * 4};
        const cuuint32_t xb[4] = {32, (cuuint32_t)TILE_W, (cuuint32_t)TILE_H, 1};
        const cuuint32_t one4[4] = {1, 1, 1, 1};
        if (enc((CUtensorMap*)plan->tmap_x2, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(a.x2), xd, xs, xb, one4,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        plan->x2 = a.x2;
    }
    if (!a.out_nchw && !a.out_u8) {
        // output [B][H][W][Cout] as a 4-D tensor (channels innermost); a box is one epilogue warp's quarter (4 rows) of a 128-byte-wide slice of a tile
        const cuuint64_t dims[4] = {(cuuint64_t)a.Cout, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)std::max(a.B, 1)};
        const cuuint64_t strides[3] = {(cuuint64_t)a.Cout * es, (cuuint64_t)a.W * a.Cout * es, (cuuint64_t)a.H * a.W * a.Cout * es};
        const cuuint32_t box[4] = {ob ? 64u : 32u, (cuuint32_t)TILE_W, 4, 1};      // one epilogue warp's rows
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

cudaError_t launch_conv_tc(const ConvArgs& a, const ConvTcPlan& plan, unsigned int* status, cudaStream_t s) {
    if (!plan.valid) return cudaErrorInvalidValue;
    if (!a.out_nchw && !a.out_u8 && (a.y != plan.y || a.B > plan.batch)) return cudaErrorInvalidValue;   // the output map is bound at prepare time
    if (a.residual && a.residual != a.y) return cudaErrorInvalidValue;                      // residual is accumulated in place
    if ((a.upsample == 2) != (plan.phase != 0)) return cudaErrorInvalidValue;
    if (a.x2 && a.x2 != plan.x2) return cudaErrorInvalidValue;                               // so is the shortcut's input map
    if (a.stat_sum && (!conv_tc_stats_supported(a, a.stat_G) || !a.stat_counter || !a.stat_scale || !a.stat_shift || !a.stat_gamma || !a.stat_beta))
        return cudaErrorInvalidValue;
    const bool ib = a.in_dtype == VD_BF16, ob = a.out_dtype == VD_BF16;
    const bool hb = a.bias != nullptr || a.bias2 != nullptr;
    const bool k1 = a.ksize == 1;
    if (a.stat_sum) {          // bf16 output with the statistics of the following GroupNorm (checked above)
        if (plan.bn == 256 && plan.cg == 2) return ib ? launch_one<256, true, 1, 2, false, true>(a, plan, status, s) : launch_one<256, false, 1, 2, false, true>(a, plan, status, s);
        if (plan.bn == 256) {
            if (k1) return ib ? launch_one<256, true, 1, 1, false, true, true, false, 1>(a, plan, status, s) : launch_one<256, false, 1, 1, false, true, true, false, 1>(a, plan, status, s);
            return ib ? launch_one<256, true, 1, 1, false, true>(a, plan, status, s) : launch_one<256, false, 1, 1, false, true>(a, plan, status, s);
        }
        if (k1) return ib ? launch_one<128, true, 1, 1, false, true, true, false, 1>(a, plan, status, s) : launch_one<128, false, 1, 1, false, true, true, false, 1>(a, plan, status, s);
        return ib ? launch_one<128, true, 1, 1, false, true>(a, plan, status, s) : launch_one<128, false, 1, 1, false, true>(a, plan, status, s);
    }
    if (plan.bn == 16) {
        if (k1) return cudaErrorInvalidValue;                  // the frame head is a 3x3 layer
        return ib ? launch_one<16, true, 2, 1>(a, plan, status, s) : launch_one<16, false, 2, 1>(a, plan, status, s);
    }
    if (a.x2) {                // fused shortcut: 3x3, bf16 intra-block input, fp32 output, one CTA per tile (conv_tc_supported)
        if (plan.bn == 256) return hb ? launch_one<256, true, 0, 1, false, false, true, true>(a, plan, status, s) : launch_one<256, true, 0, 1, false, false, false, true>(a, plan, status, s);
        return hb ? launch_one<128, true, 0, 1, false, false, true, true>(a, plan, status, s) : launch_one<128, true, 0, 1, false, false, false, true>(a, plan, status, s);
    }
#define VD_CONV_CASE(BN_, CG_, PH_, KS_)                                                                                    \
    do {                                                                                                                    \
        if (ib && ob) return hb ? launch_one<BN_, true, 1, CG_, PH_, false, true, false, KS_>(a, plan, status, s) : launch_one<BN_, true, 1, CG_, PH_, false, false, false, KS_>(a, plan, status, s);     \
        if (ib && !ob) return hb ? launch_one<BN_, true, 0, CG_, PH_, false, true, false, KS_>(a, plan, status, s) : launch_one<BN_, true, 0, CG_, PH_, false, false, false, KS_>(a, plan, status, s);    \
        if (!ib && ob) return hb ? launch_one<BN_, false, 1, CG_, PH_, false, true, false, KS_>(a, plan, status, s) : launch_one<BN_, false, 1, CG_, PH_, false, false, false, KS_>(a, plan, status, s);  \
        return hb ? launch_one<BN_, false, 0, CG_, PH_, false, true, false, KS_>(a, plan, status, s) : launch_one<BN_, false, 0, CG_, PH_, false, false, false, KS_>(a, plan, status, s);                 \
    } while (0)
    if (plan.phase) VD_CONV_CASE(128, 2, true, 3);
    if (plan.bn == 256 && plan.cg == 2) VD_CONV_CASE(256, 2, false, 3);          // (9-tap upsampling form: 3x3)
    if (plan.bn == 256) { if (k1) VD_CONV_CASE(256, 1, false, 1); VD_CONV_CASE(256, 1, false, 3); }
    if (k1) VD_CONV_CASE(128, 1, false, 1);
    VD_CONV_CASE(128, 1, false, 3);
#undef VD_CONV_CASE
}

}  // namespace vd
