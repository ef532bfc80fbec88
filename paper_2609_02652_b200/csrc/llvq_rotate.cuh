// Device pieces of the exact Walsh-Hadamard rotation, shared by the rotation kernel and by the GEMV whose
// prologue rotates x itself: integers in units of 2^-24, butterflies on 64-bit sums, one rounding to FP16.
#pragma once
#include <cstdint>

#include <cuda_fp16.h>

namespace llvq {

// R stages of the in-place butterfly on 2^R values: (a, b) -> (a + b, a - b) over every pair that differs in
// one index bit.  With the values taken at stride 2^s these are stages s .. s + R - 1 of the transform.
template <int R>
__device__ __forceinline__ void rot_butterflies(long long (&a)[8]) {
#pragma unroll
    for (int h = 1; h < (1 << R); h <<= 1) {
#pragma unroll
        for (int i = 0; i < (1 << R); i++) {
            if ((i & h) == 0) {
                const long long u = a[i], w = a[i + h];
                a[i] = u + w;
                a[i + h] = u - w;
            }
        }
    }
}

// One pass over `count` values in shared memory (a multiple of 2^R, made of whole blocks): stages s .. s + R - 1.
template <int R>
__device__ __forceinline__ void rot_pass(long long *v, int s, int count, int tid, int nthreads) {
    for (int g = tid; g < (count >> R); g += nthreads) {
        const int base = ((g >> s) << (s + R)) | (g & ((1 << s) - 1));
        long long a[8];
#pragma unroll
        for (int j = 0; j < (1 << R); j++) a[j] = v[base + (j << s)];
        rot_butterflies<R>(a);
#pragma unroll
        for (int j = 0; j < (1 << R); j++) v[base + (j << s)] = a[j];
    }
}
// the passes after the first: stages 3 .. block_log2 - 1, three at a time, a barrier after each
__device__ __forceinline__ void rot_later_passes(long long *v, int block_log2, int count, int tid, int nthreads) {
    for (int s = 3; s < block_log2; s += 3) {
        const int r = block_log2 - s;
        if (r >= 3) rot_pass<3>(v, s, count, tid, nthreads);
        else if (r == 2) rot_pass<2>(v, s, count, tid, nthreads);
        else rot_pass<1>(v, s, count, tid, nthreads);
        __syncthreads();
    }
}

// Eight consecutive FP16 coordinates -> integers in units of 2^-24 (exact: a power-of-two scaling of an 11-bit
// significand), sign flips applied (bit i of `flips` set = coordinate i negated).
__device__ __forceinline__ void rot_load8(const uint4 &raw, uint32_t flips, long long (&a)[8]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        const long long lo = __float2ll_rn(f.x * 16777216.f), hi = __float2ll_rn(f.y * 16777216.f);
        a[2 * i] = ((flips >> (2 * i)) & 1u) ? -lo : lo;
        a[2 * i + 1] = ((flips >> (2 * i + 1)) & 1u) ? -hi : hi;
    }
}

// The one rounding: eight exact sums -> f64 (exact below 2^53) -> times 2^-24 / sqrt(B) -> FP16, nearest even.
__device__ __forceinline__ uint4 rot_round8(const long long *v, double scale) {
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const __half lo = __double2half((double)v[2 * i] * scale);
        const __half hi = __double2half((double)v[2 * i + 1] * scale);
        out[i] = (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

}  // namespace llvq
