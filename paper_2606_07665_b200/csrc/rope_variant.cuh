// Prelude variants of the rotary embedding for one head vector held by one warp: optional per-head
// RMSNorm, then rotation of the first rotary_dim elements with half-split or interleaved pairing.
// Shared by the stand-alone variant kernel and the single-launch step.
#pragma once

#include "ac_device.cuh"

namespace acdev {

// x[e] holds element lane * (D/32) + e of the vector (bf16 bits): the raw values on entry, the normalised
// and rotated ones on return.  `park` is D 16-bit words of shared memory private to the calling warp
// (every lane must be able to read the partner of each of its elements, wherever the pairing puts it);
// its contents on return are the normalised, un-rotated vector, and every lane is done reading it.
//
// RMSNorm arithmetic (norm_w != nullptr): sum of squares in fp64 (exact for bf16 inputs of moderate
// dynamic range), r = 1 / sqrt(sum / D + eps) with correctly rounded fp64 sqrt and division,
// y = bf16(x * r), then bf16(y * w): normalise, round to the model dtype, scale by the weight, round
// again.  Rotation: pair (i, i + rotary_dim/2) or (2i, 2i + 1), angle i = cos_row[i], sin_row[i], each
// result the nearest-even bf16 of the exact value (rope_first_half / rope_second_half); elements at or
// past rotary_dim pass through.
template <int D>
__device__ __forceinline__ void rope_variant_vector(uint16_t (&x)[D / 32], const uint16_t* norm_w,
                                                    float norm_eps, const float* cos_row,
                                                    const float* sin_row, int rotary_dim, int interleaved,
                                                    uint16_t* park, int lane) {
    constexpr int EPL = D / 32;                           // elements per lane: 4 (D=128) or 2 (D=64)
    if (norm_w != nullptr) {
        double ss = 0.0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const double v = static_cast<double>(bf16_bits_to_float(x[e]));
            ss = __dadd_rn(ss, __dmul_rn(v, v));
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) ss = __dadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, off));
        const double r = __ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(__ddiv_rn(ss, static_cast<double>(D)),
                                                             static_cast<double>(norm_eps))));
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const double v = static_cast<double>(bf16_bits_to_float(x[e]));
            const uint16_t y1 = f64_to_bf16_rne(__dmul_rn(v, r));
            const double w = static_cast<double>(bf16_bits_to_float(norm_w[lane * EPL + e]));
            x[e] = f64_to_bf16_rne(__dmul_rn(static_cast<double>(bf16_bits_to_float(y1)), w));
        }
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) park[lane * EPL + e] = x[e];
    __syncwarp();

    const int half = rotary_dim / 2;
    uint16_t out[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        const int j = lane * EPL + e;
        if (j >= rotary_dim) {
            out[e] = x[e];
            continue;
        }
        int i, partner;
        bool first;
        if (interleaved) {
            i = j >> 1;
            first = (j & 1) == 0;
            partner = first ? j + 1 : j - 1;
        } else {
            first = j < half;
            i = first ? j : j - half;
            partner = first ? j + half : j - half;
        }
        const float c = cos_row[i];
        const float sn = sin_row[i];
        const uint16_t other = park[partner];
        out[e] = first ? rope_first_half(x[e], other, c, sn) : rope_second_half(other, x[e], c, sn);
    }
    __syncwarp();                                         // every lane has read its partners
#pragma unroll
    for (int e = 0; e < EPL; ++e) x[e] = out[e];
}

}  // namespace acdev
