// Pieces shared by the one-CTA and the two-CTA tensor-core convolution kernels: tile geometry,
// and the operand loader of the prologue.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {
namespace convtile {

constexpr int TILE_H = 16, TILE_W = 8;                               // one MMA tile: 128 output pixels
constexpr int PH = TILE_H + 2, PW = TILE_W + 2, NPIX = PH * PW;     // 18 x 10 = 180 halo pixels
constexpr int A_TILE_BYTES = (NPIX * 128 + 1023) / 1024 * 1024;      // one 64-channel chunk of one halo tile: 180 rows of 128 B
constexpr int ITEMS = NPIX * 8;                                      // (pixel, 8-channel group) pairs per tile chunk
constexpr int NUM_PRODUCER_WARPS = 15;
constexpr int NUM_PRODUCERS = NUM_PRODUCER_WARPS * 32;               // 480 = ITEMS / 3: three pairs per thread
constexpr int BATCH = ITEMS / NUM_PRODUCERS;                         // 3
static_assert(BATCH * NUM_PRODUCERS == ITEMS, "producer threads must tile the halo chunk exactly");
// Warps map to the four SM sub-partitions by (warp % 4), and a sub-partition's scheduler gives the
// MMA-issuing thread no priority: measured, fifteen warps of dense arithmetic stretch its
// wait / 4 x MMA / commit sequence from 513 to about 1800 cycles, while the same warps kept off its
// sub-partition cost nothing.  So sub-partition 0 carries only the MMA warp, the TMA warp and one
// epilogue warp (warps 8, 12 and 20 idle until the end), and the fifteen producer warps are the
// warps with warp % 4 != 0 outside the epilogue: five per remaining sub-partition.
constexpr int MMA_WARP = 0;
constexpr int TMA_WARP = 4;
constexpr int EPI_WARP0 = 16;                                        // warps 16-19 (warp % 4 = TMEM lane quarter)
constexpr int NUM_THREADS = 24 * 32;
__device__ __forceinline__ bool is_producer_warp(int warp) { return (warp & 3) != 0 && (warp < EPI_WARP0 || warp >= EPI_WARP0 + 4); }
// 0..14 over the producer warps
__device__ __forceinline__ int producer_index(int warp) { return (warp < EPI_WARP0 ? (warp >> 2) : 4) * 3 + (warp & 3) - 1; }
constexpr int OUT_SLICE_BYTES = 128 * 128;                           // 128 pixels x 128 B: one output slice in smem

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
// the same loads from the address of the thread's first channel.  The activations are streamed
// (no reuse within the SM): they bypass L1 allocation, which leaves the small L1 that remains beside
// the shared-memory tiles to the data that is reused.
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void load_raw_at(bool is_bf16, const char* p, Raw8& r) {
    r.lo = ldg_stream(p);
    if (!is_bf16) r.hi = ldg_stream(p + 128);
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

struct Tile { int tx0, ty0, n0, b; };

}  // namespace convtile
}  // namespace vd
