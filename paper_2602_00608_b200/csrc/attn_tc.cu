// Fused single-head attention on tcgen05/TMEM for the decoder's mid block (C = 512 channels):
//   o[t,:] = sum_u softmax_u(scale * q[t,:].k[u,:]) v[u,:]
// One CTA owns 128 queries and one 256-channel half of the output.  Per 128-key tile:
//   S = Q K^T      streamed as eight 64-channel chunks of Q and K (TMA, 128B swizzle), fp32 in TMEM
//   softmax        four warps, one query row per thread: running maximum with lazy rescaling of
//                  the output accumulator, exp2 in fp32, row sums in fp32, P rounded to bf16 and
//                  written to shared memory in the swizzled K-major operand layout
//   O += P V       V is consumed transposed ([channel][token], produced by a small transpose
//                  kernel) so both operands of both products are K-major
// S is double-buffered in TMEM (2 x 128 columns next to the 256 columns of O), so the tensor
// core works on the next tile's scores while the softmax warps are busy.  The N x N score
// matrix never exists in memory.  Every wait is bounded (see tc_common.cuh).
#include <mutex>
#include <cuda.h>

#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

using namespace tc;

constexpr int BQ = 128, BKV = 128, DV = 256, DCHUNK = 64;
constexpr int QK_STAGES = 4, V_STAGES = 2;                   // as many Q/K stages as fit: the score product waits on this stream
constexpr int QK_STAGE_BYTES = 2 * BQ * DCHUNK * 2;          // Q chunk + K chunk: 16 KB + 16 KB
constexpr int V_STAGE_BYTES = DV * 64 * 2;                   // 256 channels x 64 keys: 32 KB
constexpr int P_BYTES = BQ * BKV * 2;                        // 32 KB (two 64-key halves)
constexpr int SMEM_TOTAL = QK_STAGES * QK_STAGE_BYTES + V_STAGES * V_STAGE_BYTES + P_BYTES + 256 + 1024;
constexpr int NUM_THREADS = 224;                             // 4 softmax warps, QK loader, V loader, MMA
constexpr float RESCALE_THRESHOLD = 8.0f;                    // log2 units: accumulators may grow by 2^8

struct Bars {
    uint64_t qk_full[QK_STAGES], qk_empty[QK_STAGES];
    uint64_t v_full[V_STAGES], v_empty[V_STAGES];
    uint64_t s_full[2], s_free[2];
    uint64_t p_full, pv_done;
    uint32_t tmem_base, abort_flag;
};

struct AttnTcParams {
    void* o;
    int B, T, C, ld_o;
    float scale_log2;        // scale * log2(e)
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_tc_kernel(const AttnTcParams a, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_vt, unsigned int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_qk = smem;
    uint8_t* smem_v = smem + QK_STAGES * QK_STAGE_BYTES;
    uint8_t* smem_p = smem_v + V_STAGES * V_STAGE_BYTES;
    Bars* bars = (Bars*)(smem_p + P_BYTES);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q0 = blockIdx.x * BQ;
    const int dv0 = blockIdx.y * DV;
    const int b = blockIdx.z;
    const int ntiles = (a.T + BKV - 1) / BKV;
    const int dchunks = a.C / DCHUNK;

    if (tid == 0) {
        for (int i = 0; i < QK_STAGES; ++i) { mbar_init(smem_u32(&bars->qk_full[i]), 1); mbar_init(smem_u32(&bars->qk_empty[i]), 1); }
        for (int i = 0; i < V_STAGES; ++i) { mbar_init(smem_u32(&bars->v_full[i]), 1); mbar_init(smem_u32(&bars->v_empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bars->s_full[i]), 1); mbar_init(smem_u32(&bars->s_free[i]), 128); }
        mbar_init(smem_u32(&bars->p_full), 128);
        mbar_init(smem_u32(&bars->pv_done), 1);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 4) tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    const uint32_t tmem_o = tmem + 256;
    griddep_launch();            // the next kernel may set itself up from here on
    if (warp != 6) griddep_wait();   // every role but the MMA issue loop touches activations of earlier kernels

    if (warp < 4) {
        // ------------------------------------------------------------ softmax warps
        const int row = tid;                                       // query row of the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < ntiles && ok; ++j) {
            const int buf = j & 1;
            ok = mbar_wait(smem_u32(&bars->s_full[buf]), (j >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ts = tmem + (uint32_t)(buf * 128) + lane_base;
            const int kvalid = min(BKV, a.T - j * BKV);            // keys of this tile that exist
            // pass 1: tile maximum (log2 units)
            float tmax = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < BKV; c += 32) {
                uint32_t r[32];
                tmem_ld32(ts + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 32; ++q)
                    if (c + q < kvalid) tmax = fmaxf(tmax, __uint_as_float(r[q]) * a.scale_log2);
            }
            // lazy rescale: keep the old reference unless the maximum grew by more than the threshold
            float factor = 1.f;
            const bool grow = tmax > m_ref + RESCALE_THRESHOLD;
            if (grow) {
                factor = ex2(m_ref - tmax);                        // 0 at the first tile (m_ref = -inf)
                m_ref = tmax;
                l *= factor;
            }
            const bool any_grow = __any_sync(0xffffffffu, grow) && j > 0;
            if (j > 0) {
                // P buffer and O are free once the previous tile's P.V product has completed
                ok = mbar_wait(smem_u32(&bars->pv_done), (j - 1) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
            }
            if (any_grow) {
#pragma unroll 1
                for (int c = 0; c < DV; c += 32) {
                    uint32_t r[32];
                    tmem_ld32(tmem_o + lane_base + c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) * factor);
                    tmem_st32(tmem_o + lane_base + c, r);
                }
                tmem_st_wait();
            }
            // pass 2: p = 2^(s - m_ref), row sum, bf16, swizzled store (row r, 16-byte chunk c -> c ^ (r & 7))
            uint8_t* prow = smem_p + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll 1
            for (int c = 0; c < BKV; c += 32) {
                uint32_t r[32];
                tmem_ld32(ts + c, r);
                tmem_ld_wait();
                float p[32];
#pragma unroll
                for (int q = 0; q < 32; ++q) {
                    const float e = ex2(fmaf(__uint_as_float(r[q]), a.scale_log2, -m_ref));
                    p[q] = (c + q < kvalid) ? e : 0.f;
                    l += p[q];
                }
                uint8_t* half = prow + (c >> 6) * (BQ * 128);
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int chunk = ((c & 63) >> 3) + g;
                    *(uint4*)(half + ((chunk ^ (row & 7)) << 4)) =
                        make_uint4(pack_bf16(p[8 * g], p[8 * g + 1]), pack_bf16(p[8 * g + 2], p[8 * g + 3]),
                                   pack_bf16(p[8 * g + 4], p[8 * g + 5]), pack_bf16(p[8 * g + 6], p[8 * g + 7]));
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars->s_free[buf]));             // scores consumed: buffer may be overwritten
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&bars->p_full));
        }
        if (ok) {
            ok = mbar_wait(smem_u32(&bars->pv_done), (ntiles - 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            const bool inside = q0 + row < a.T;
            __nv_bfloat16* orow = (__nv_bfloat16*)a.o + ((size_t)b * a.T + q0 + row) * a.ld_o + dv0;
#pragma unroll 1
            for (int c = 0; c < DV; c += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_o + lane_base + c, r);
                tmem_ld_wait();
                if (inside) {
#pragma unroll
                    for (int q = 0; q < 32; q += 8) {
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[q + e]) * inv;
                        *(uint4*)(orow + c + q) = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]),
                                                             pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                    }
                }
            }
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ Q/K chunk loads
        if (lane == 0) {
            uint32_t st = 0, ph = 0;
            bool ok = true;
            for (int j = 0; j < ntiles && ok; ++j) {
                for (int dc = 0; dc < dchunks; ++dc) {
                    ok = mbar_wait(smem_u32(&bars->qk_empty[st]), ph ^ 1, abort_flag);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&bars->qk_full[st]);
                    mbar_arrive_expect_tx(full, QK_STAGE_BYTES);
                    uint8_t* dst = smem_qk + st * QK_STAGE_BYTES;
                    tma_load_2d(smem_u32(dst), &tm_q, dc * DCHUNK, b * a.T + q0, full);
                    tma_load_2d(smem_u32(dst + BQ * DCHUNK * 2), &tm_k, dc * DCHUNK, b * a.T + j * BKV, full);
                    if (++st == QK_STAGES) { st = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ V^T loads
        if (lane == 0) {
            uint32_t st = 0, ph = 0;
            bool ok = true;
            for (int j = 0; j < ntiles && ok; ++j) {
                for (int h = 0; h < 2; ++h) {
                    ok = mbar_wait(smem_u32(&bars->v_empty[st]), ph ^ 1, abort_flag);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&bars->v_full[st]);
                    mbar_arrive_expect_tx(full, V_STAGE_BYTES);
                    tma_load_2d(smem_u32(smem_v + st * V_STAGE_BYTES), &tm_vt, j * BKV + h * 64, b * a.C + dv0, full);
                    if (++st == V_STAGES) { st = 0; ph ^= 1; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issue
        // The whole warp runs the loop and the tensor instructions are predicated on one elected lane
        // (no branch): warp-uniform code keeps the descriptors in uniform registers, which makes the
        // wait / 4 x MMA / commit sequence of a 64-channel chunk cheaper than the 256 tensor cycles it
        // feeds.  The waits are not voted on (a wait that gave up leaves garbage behind that nobody
        // reads); the abort flag is looked at once per key tile.
        {
            const uint32_t lead = elect_one();
            constexpr uint32_t idesc_s = make_idesc_bf16(128, BKV);
            constexpr uint32_t idesc_o = make_idesc_bf16(128, DV);
            const uint32_t hi = desc_hi(1024, 2);
            uint32_t qst = 0, qph = 0, vst = 0, vph = 0;
            auto wait_on = [&](uint64_t* bar, uint32_t ph) {
                const uint32_t b = smem_u32(bar);
                if (!mbar_try_wait(b, ph)) (void)mbar_wait(b, ph, abort_flag);
                tc_fence_after();
            };
            auto issue_qk = [&](int j) {
                const int buf = j & 1;
                wait_on(&bars->s_free[buf], ((j >> 1) & 1) ^ 1);
                for (int dc = 0; dc < dchunks; ++dc) {
                    wait_on(&bars->qk_full[qst], qph);
                    const uint32_t qa = desc_lo(smem_u32(smem_qk + qst * QK_STAGE_BYTES));
                    const uint32_t ka = qa + ((BQ * DCHUNK * 2) >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16_split_on(tmem + (uint32_t)(buf * 128), qa + k * 2, hi, ka + k * 2, hi, idesc_s, (dc | k) != 0 ? 1u : 0u, lead);
                    umma_commit_on(smem_u32(&bars->qk_empty[qst]), lead);
                    __syncwarp();
                    if (++qst == QK_STAGES) { qst = 0; qph ^= 1; }
                }
                umma_commit_on(smem_u32(&bars->s_full[buf]), lead);
                __syncwarp();
            };
            auto issue_pv = [&](int j) {
                wait_on(&bars->p_full, j & 1);
                for (int h = 0; h < 2; ++h) {
                    wait_on(&bars->v_full[vst], vph);
                    const uint32_t pa = desc_lo(smem_u32(smem_p + h * (BQ * 128)));
                    const uint32_t va = desc_lo(smem_u32(smem_v + vst * V_STAGE_BYTES));
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16_split_on(tmem_o, pa + k * 2, hi, va + k * 2, hi, idesc_o, (j | h | k) != 0 ? 1u : 0u, lead);
                    umma_commit_on(smem_u32(&bars->v_empty[vst]), lead);
                    __syncwarp();
                    if (++vst == V_STAGES) { vst = 0; vph ^= 1; }
                }
                umma_commit_on(smem_u32(&bars->pv_done), lead);
                __syncwarp();
            };
            issue_qk(0);
            for (int j = 0; j < ntiles; ++j) {
                if (*abort_flag) break;
                if (j + 1 < ntiles) issue_qk(j + 1);
                issue_pv(j);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && bars->abort_flag && status) {
        if (atomicCAS(status, 0u, kStatusAttnTimeout) == 0u) {
            status[1] = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
            status[2] = 0;
        }
    }
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

// v [B][T][ld] -> vt [B][C][Tp] (tokens contiguous, zero beyond T)
__global__ void transpose_v_kernel(const __nv_bfloat16* v, __nv_bfloat16* vt, int T, int Tp, int C, int ld) {
    __shared__ __nv_bfloat16 tile[32][33];
    griddep_launch();
    griddep_wait();
    const int b = blockIdx.z;
    const int t0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        const int t = t0 + i, c = c0 + threadIdx.x;
        tile[i][threadIdx.x] = (t < T) ? v[((size_t)b * T + t) * ld + c] : __float2bfloat16(0.f);
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        const int c = c0 + i, t = t0 + threadIdx.x;
        if (t < Tp) vt[((size_t)b * C + c) * Tp + t] = tile[threadIdx.x][i];
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

bool encode_2d(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes, uint32_t box_cols,
               uint32_t box_rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int padded_tokens(int T) { return (T + 63) / 64 * 64; }

}  // namespace

bool attn_tc_supported(const AttnArgs& a) {
    return a.dtype == VD_BF16 && a.C == 512 && a.ld_qkv % 8 == 0 && a.ld_o % 8 == 0 && a.T >= 1;
}

size_t attn_tc_scratch_bytes(int B, int T, int C) { return (size_t)B * C * padded_tokens(T) * 2; }

cudaError_t attn_tc_prepare(const AttnArgs& a, AttnTcPlan* plan) {
    plan->valid = 0;
    if (!a.vt) return cudaErrorInvalidValue;
    if (((uintptr_t)a.q | (uintptr_t)a.k | (uintptr_t)a.vt) & 15) return cudaErrorMisalignedAddress;
    const int Tp = padded_tokens(a.T);
    const uint64_t rows = (uint64_t)a.B * a.T;
    if (!encode_2d((CUtensorMap*)plan->tq, a.q, a.C, rows, (uint64_t)a.ld_qkv * 2, DCHUNK, BQ)) return cudaErrorInvalidValue;
    if (!encode_2d((CUtensorMap*)plan->tk, a.k, a.C, rows, (uint64_t)a.ld_qkv * 2, DCHUNK, BKV)) return cudaErrorInvalidValue;
    if (!encode_2d((CUtensorMap*)plan->tv, a.vt, Tp, (uint64_t)a.B * a.C, (uint64_t)Tp * 2, 64, DV)) return cudaErrorInvalidValue;
    plan->q = a.q; plan->k = a.k; plan->vt = a.vt;
    plan->batch = a.B; plan->tokens = a.T;
    plan->valid = 1;
    return cudaSuccess;
}

cudaError_t launch_attn_tc(const AttnArgs& a, const AttnTcPlan* plan, unsigned int* status, cudaStream_t s) {
    if (!a.vt) return cudaErrorInvalidValue;
    if (((uintptr_t)a.q | (uintptr_t)a.k | (uintptr_t)a.v | (uintptr_t)a.o | (uintptr_t)a.vt) & 15) return cudaErrorMisalignedAddress;
    const int Tp = padded_tokens(a.T);
    {
        dim3 grid(Tp / 32, a.C / 32, a.B), block(32, 8);
        cudaError_t e = launch_pdl(transpose_v_kernel, grid, block, 0, s, (const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.vt, a.T, Tp, a.C, a.ld_qkv);
        if (e != cudaSuccess) return e;
    }
    // The maps of a decoder's fixed workspace tensors are built once (attn_tc_prepare, for the largest batch: rows
    // beyond the batch in use are never addressed); a call on other tensors encodes its own.
    AttnTcPlan local;
    if (!(plan && plan->valid && plan->q == a.q && plan->k == a.k && plan->vt == a.vt && plan->tokens == a.T && a.B <= plan->batch)) {
        cudaError_t e = attn_tc_prepare(a, &local);
        if (e != cudaSuccess) return e;
        plan = &local;
    }
    const CUtensorMap &tq = *(const CUtensorMap*)plan->tq, &tk = *(const CUtensorMap*)plan->tk, &tv = *(const CUtensorMap*)plan->tv;
    {
        static std::mutex mu;
        static bool configured[64] = {};
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {              // the attribute is per device
            e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL);
            if (e != cudaSuccess) return e;
            configured[dev] = true;
        }
    }
    AttnTcParams p{a.o, a.B, a.T, a.C, a.ld_o, a.scale * 1.4426950408889634f};
    dim3 grid((a.T + BQ - 1) / BQ, a.C / DV, a.B);
    return launch_pdl(attn_tc_kernel, grid, dim3(NUM_THREADS), SMEM_TOTAL, s, p, tq, tk, tv, status);
}

}  // namespace vd
