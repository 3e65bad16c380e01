// The centroid-side operand of the assign kernel's extra k-step, one 16-byte row per centroid:
// [1 1 1 h_hi h_mid h_lo 0 0] with h = ||c||^2 / 2 split into three bf16 terms (paper Section 5,
// "Flash-KMeans clean-start workload": the ||c||^2 term of the distance expansion).  Shared by the
// assign prologue and by the division kernel of the update, which writes the operand of the next
// iteration's centroids while it has them in registers: both sum the squares in the same order, so
// the operand does not depend on who wrote it.
#pragma once
#include <cstdint>

#include "internal.h"

namespace cake {
namespace aug {

__device__ __forceinline__ uint32_t bf16_rne_bits(float f) {
    uint32_t u = __float_as_uint(f);
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}
// h = hi + mid + lo with three bf16 terms (24 significand bits: nothing of the fp32 value is lost)
__device__ __forceinline__ void split3(float h, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
    hi = bf16_rne_bits(h);
    const float r1 = h - __uint_as_float(hi << 16);
    mid = bf16_rne_bits(r1);
    const float r2 = r1 - __uint_as_float(mid << 16);
    lo = bf16_rne_bits(r2);
}

// Four bf16 values (two packed words, columns 4j..4j+3 of the row) added to a lane's sum of squares.
// A row is summed as: lane l takes the column quads l, l+32, ... in ascending order, then the lanes
// are folded with xor-shuffles 16, 8, 4, 2, 1.
__device__ __forceinline__ float add_squares(float acc, uint32_t w0, uint32_t w1) {
    float v;
    v = __uint_as_float(w0 << 16); acc = fmaf(v, v, acc);
    v = __uint_as_float(w0 & 0xFFFF0000u); acc = fmaf(v, v, acc);
    v = __uint_as_float(w1 << 16); acc = fmaf(v, v, acc);
    v = __uint_as_float(w1 & 0xFFFF0000u); acc = fmaf(v, v, acc);
    return acc;
}
__device__ __forceinline__ float fold_lanes(float acc) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

// Lane 0 of the warp that holds ||c_k||^2 (`norm`) of centroid k of problem b writes the row.
// k >= K: a padded row [1 1 1 2^120 0 0 0 0], whose accumulator is about 2^120 and can never win
// (norms are assumed to stay below that).
__device__ __forceinline__ void write_row(uint8_t* caug, i64 b, int k, int K, int Kpad, float norm) {
    uint32_t hi = 0x7B80u, mid = 0, lo = 0;   // 2^120 as bf16
    if (k < K) split3(0.5f * norm, hi, mid, lo);
    const uint32_t one = 0x3F80u;
    const int tile = k / static_cast<int>(kAssignBlockN), rr = k % static_cast<int>(kAssignBlockN);
    uint8_t* blk = caug + (static_cast<size_t>(b) * (Kpad / static_cast<int>(kAssignBlockN)) + tile) * kAssignAugTileBytes;
    *reinterpret_cast<uint4*>(blk + rr * 16) = make_uint4(one | (one << 16), one | (hi << 16), mid | (lo << 16), 0u);
}

// The centroid rows are streamed by TMA once per row tile; rows whose pitch is not a multiple of 128
// bytes (D % 64 != 0) measured up to twice as slow to stream, so the kernel then reads a copy whose rows
// are padded with zeros to Dc columns (a multiple of 64).  One warp copies one row (src only 2-byte
// aligned when D is odd; dst 16-byte aligned).
__device__ __forceinline__ void copy_row_padded(const cake_bf16* __restrict__ src, int D, cake_bf16* __restrict__ dst,
                                                int Dc, int lane) {
    for (int g = lane; g < Dc / 8; g += 32) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = g * 8 + 2 * j;
            const uint32_t lo = c < D ? static_cast<uint32_t>(__ldg(src + c)) : 0u;
            const uint32_t hi = c + 1 < D ? static_cast<uint32_t>(__ldg(src + c + 1)) : 0u;
            w[j] = lo | (hi << 16);
        }
        reinterpret_cast<uint4*>(dst)[g] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace aug
}  // namespace cake
