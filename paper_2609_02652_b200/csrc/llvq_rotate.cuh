// Device pieces of the exact Walsh-Hadamard rotation, shared by the rotation kernel and by the GEMV whose
// prologue rotates x itself: integers in units of 2^-24, butterflies on 64-bit sums, one rounding to FP16.
#pragma once
#include <cstdint>

#include <cuda_fp16.h>

namespace llvq {

// Where value i of the array lives in shared memory.  A thread of a pass touches eight values 2^s apart and its
// neighbours the values beside them; with the low four index bits XORed by the next four, every such access of a
// warp (32 values of 8 bytes) spreads evenly over the banks: two wavefronts, the least 256 bytes take.
__device__ __forceinline__ int rot_at(int i) { return i ^ ((i >> 4) & 15); }

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

// One pass over `count` values in shared memory (whole blocks): stages S .. S + R - 1.  S and R are compile-time
// so that the eight addresses of a thread come from one computed address and constants.
template <int R, int S>
__device__ __forceinline__ void rot_pass(long long *v, int count, int tid, int nthreads) {
    for (int g = tid; g < (count >> R); g += nthreads) {
        const int base = ((g >> S) << (S + R)) | (g & ((1 << S) - 1));
        long long a[8];
        if (S >= 8) {
            // the stride leaves the eight swizzled index bits alone
            long long *at = v + rot_at(base);
#pragma unroll
            for (int j = 0; j < (1 << R); j++) a[j] = at[j << S];
            rot_butterflies<R>(a);
#pragma unroll
            for (int j = 0; j < (1 << R); j++) at[j << S] = a[j];
        } else {
#pragma unroll
            for (int j = 0; j < (1 << R); j++) a[j] = v[rot_at(base + (j << S))];
            rot_butterflies<R>(a);
#pragma unroll
            for (int j = 0; j < (1 << R); j++) v[rot_at(base + (j << S))] = a[j];
        }
    }
}
template <int S>
__device__ __forceinline__ void rot_pass_from(long long *v, int block_log2, int count, int tid, int nthreads) {
    const int r = block_log2 - S;
    if (r >= 3) rot_pass<3, S>(v, count, tid, nthreads);
    else if (r == 2) rot_pass<2, S>(v, count, tid, nthreads);
    else rot_pass<1, S>(v, count, tid, nthreads);
    __syncthreads();
}
// the passes after the first: stages 3 .. block_log2 - 1 (block_log2 <= 14), three at a time, a barrier after each
__device__ __forceinline__ void rot_later_passes(long long *v, int block_log2, int count, int tid, int nthreads) {
    if (block_log2 > 3) rot_pass_from<3>(v, block_log2, count, tid, nthreads);
    if (block_log2 > 6) rot_pass_from<6>(v, block_log2, count, tid, nthreads);
    if (block_log2 > 9) rot_pass_from<9>(v, block_log2, count, tid, nthreads);
    if (block_log2 > 12) rot_pass_from<12>(v, block_log2, count, tid, nthreads);
}

// stores the eight values first .. first + 7 (first a multiple of eight)
__device__ __forceinline__ void rot_store8(long long *v, int first, const long long (&a)[8]) {
#pragma unroll
    for (int k = 0; k < 8; k++) v[rot_at(first + k)] = a[k];
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
// The sums are values first .. first + 7 of the array v (first a multiple of eight).
__device__ __forceinline__ uint4 rot_round8(const long long *v, int first, double scale) {
    uint32_t out[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const __half lo = __double2half((double)v[rot_at(first + 2 * i)] * scale);
        const __half hi = __double2half((double)v[rot_at(first + 2 * i + 1)] * scale);
        out[i] = (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

}  // namespace llvq
