// Device side of sigma(. + b) with dropout, shared by the kernels that finish a layer (the forward equation of
// Section 3.3): the SpMM epilogue when a layer transforms first, the transform's epilogue when it aggregates first.
#pragma once

#include <stdint.h>

#include "gad_internal.h"

namespace gad {

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}

// Row part of the dropout hash: (seed, epoch, layer, row) -> 64 bits; the column is mixed in per element.
__device__ __forceinline__ uint64_t dropout_row_key(uint64_t seed, int64_t epoch, int layer, int64_t row) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    uint64_t h = mix64(seed + G * (uint64_t)(1 + epoch));
    h = mix64(h + G * (uint64_t)(1 + layer));
    return mix64(h + G * (uint64_t)(1 + row));
}
__device__ __forceinline__ bool dropout_keep(uint64_t row_key, int col, uint32_t thr24) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    uint64_t h = mix64(row_key + G * (uint64_t)(1 + col));
    return (uint32_t)(h >> 40) >= thr24;
}

// fp32 -> bfloat16 bits (round to nearest even; NaN stays a quiet NaN).
__device__ __forceinline__ uint32_t bf16_bits(float x) {
    const uint32_t b = __float_as_uint(x);
    if ((b & 0x7fffffffu) > 0x7f800000u) return (b >> 16) | 0x40u;
    return (b + 0x7fffu + ((b >> 16) & 1u)) >> 16;
}
// Four consecutive values as four bfloat16 (value i in bits 16 i .. 16 i + 15 of the 64 bits).
__device__ __forceinline__ uint2 bf16_pack4(float4 v) {
    return make_uint2(bf16_bits(v.x) | (bf16_bits(v.y) << 16), bf16_bits(v.z) | (bf16_bits(v.w) << 16));
}

// ReLU that lets NaN through (fmaxf would turn it into 0).
__device__ __forceinline__ float relu_nan(float x) { return x > 0.f ? x : (x <= 0.f ? 0.f : x); }

// The four biases of replica k for columns col .. col+3.
__device__ __forceinline__ float4 load_bias(const ActEpi& ep, int k, int col) {
    return __ldg(reinterpret_cast<const float4*>(ep.params + (long long)k * ep.pstride + ep.b_int + col));
}

// v = four consecutive pre-activation sums of `row`, columns col .. col+3 (before the bias b).
__device__ __forceinline__ float4 apply_act(float4 v, float4 b, const ActEpi& ep, long long row, int col) {
    float x[4] = {v.x + b.x, v.y + b.y, v.z + b.z, v.w + b.w};
    if (ep.relu) {
        const uint64_t key = ep.drop ? dropout_row_key(ep.seed, ep.epoch, ep.layer, row) : 0ull;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            x[t] = relu_nan(x[t]);
            if (ep.drop) x[t] = dropout_keep(key, ep.col0 + col + t, ep.thr) ? x[t] * ep.scale : 0.f;
        }
    }
    return make_float4(x[0], x[1], x[2], x[3]);
}
__device__ __forceinline__ float4 apply_act(float4 v, const ActEpi& ep, int k, long long row, int col) {
    return apply_act(v, load_bias(ep, k, col), ep, row, col);
}

}  // namespace gad
