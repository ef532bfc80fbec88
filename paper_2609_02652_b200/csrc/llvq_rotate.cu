// Activation rotation: the block-diagonal normalised Walsh-Hadamard transform applied to the activation ahead of
// every projection whose weights are stored in the incoherence-rotated basis (paper Sec. 2.3: the rotation is a
// kernel of its own, run by one thread block in its shared memory; Sec. 5, on the rotated basis: that block keeps
// the whole activation as f32, so the widest projection input of a model must fit one block's shared memory).
//
//     y[B c + k] = (1 / sqrt(B)) sum_{i < B} (-1)^popcount(i & k) s_i x[B c + i]      (natural order)
//
// What is done differently here:
//   - The transform is block diagonal, B a power of two that divides n, so a CTA holds one block (or a few short
//     ones), not the activation: the width of the model no longer meets a shared-memory bound, and the blocks of a
//     vector run on several multiprocessors.  16384 coordinates a block is the most a CTA takes (128 KiB).
//   - The butterflies run on integers.  An FP16 value is a multiple of 2^-24 below 2^16, so x 2^24 is an integer
//     below 2^40 and every partial sum of up to 2^14 of them fits 64 bits: the sums are exact, whatever the order.
//     The one rounding is the last step, (double)sum * 2^-24 / sqrt(B) -> FP16 to nearest even, so the output is
//     the correctly rounded value of the definition (while the block's sum of |x| stays below 2^29) and does not
//     depend on the launch.
//   - Three stages a pass in registers (radix 8), one barrier a pass: five barriers for 4096 coordinates instead
//     of a ladder of twelve.
//   - The kernel is a link of a programmatic-dependent-launch chain: it lets the next kernel (the GEMV) set up at
//     once and waits for the previous kernel before it touches x or y.
#include <cmath>

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "llvq_internal.cuh"
#include "llvq_rotate.cuh"

namespace llvq {
namespace {

constexpr int kRotThreads = 512;
constexpr int kRotMinChunkLog2 = 12;     // a CTA takes at least 4096 coordinates: eight a thread and pass

__global__ void __launch_bounds__(kRotThreads)
rotate_kernel(const __half *x, __half *y, const uint32_t *__restrict__ negate, long long n, int chunk_log2,
              int block_log2, double scale) {
    extern __shared__ __align__(16) unsigned char rot_smem[];
    long long *v = reinterpret_cast<long long *>(rot_smem);
    // x is not marked read-only: y may be x (each CTA reads its whole piece before it writes any of it)
    const int tid = threadIdx.x;
    const int chunk = 1 << chunk_log2;
    const long long first = (long long)blockIdx.x << chunk_log2;
    const long long left = n - first;
    const int count = left < chunk ? (int)left : chunk;          // whole blocks, a multiple of eight

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // Pass 0: eight consecutive coordinates a thread become integers in units of 2^-24 (exactly: a power-of-two
    // scaling of an 11-bit significand), take their sign flips and the stages 0..2 that stay inside the eight.
    for (int g = tid; g < (chunk >> 3); g += kRotThreads) {
        long long a[8];
        if (8 * g < count) {
            const long long at = first + 8 * g;
            const uint4 raw = *reinterpret_cast<const uint4 *>(x + at);
            const uint32_t flips = negate ? (negate[at >> 5] >> (at & 31)) & 0xffu : 0u;
            rot_load8(raw, flips, a);
            if (block_log2 >= 3) rot_butterflies<3>(a);
            else if (block_log2 == 2) {
                // two blocks of four: the butterflies of stages 0 and 1 never pair i with i + 4
                long long b[8] = {a[0], a[1], a[2], a[3], 0, 0, 0, 0}, c[8] = {a[4], a[5], a[6], a[7], 0, 0, 0, 0};
                rot_butterflies<2>(b);
                rot_butterflies<2>(c);
#pragma unroll
                for (int i = 0; i < 4; i++) { a[i] = b[i]; a[4 + i] = c[i]; }
            } else if (block_log2 == 1) {
#pragma unroll
                for (int i = 0; i < 8; i += 2) {
                    const long long u = a[i], w2 = a[i + 1];
                    a[i] = u + w2;
                    a[i + 1] = u - w2;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; i++) a[i] = 0;                // past the end of x: never mixed with a block of x
        }
        rot_store8(v, 8 * g, a);
    }
    __syncthreads();

    // Passes over the stages 3.., three at a time: a thread takes the eight (four, two) values that differ in
    // the pass's index bits.
    rot_later_passes(v, block_log2, chunk, tid, kRotThreads);

    // The one rounding: exact sum -> f64 (exact below 2^53) -> times 2^-24 / sqrt(B) -> FP16, nearest even.
    for (int g = tid; 8 * g < count; g += kRotThreads) {
        *reinterpret_cast<uint4 *>(y + first + 8 * g) = rot_round8(v, 8 * g, scale);
    }
}

}  // namespace

int rotate_block_log2(int64_t n, int64_t block) {
    if (n <= 0) return -1;
    if (block == 0) {
        int l = 0;
        while (l < kRotMaxBlockLog2 && n % ((int64_t)2 << l) == 0) l++;
        return l;
    }
    if (block < 1 || block > ((int64_t)1 << kRotMaxBlockLog2) || (block & (block - 1)) || n % block) return -1;
    int l = 0;
    while (((int64_t)1 << l) < block) l++;
    return l;
}

int rotate_configure() {
    return cudaFuncSetAttribute(rotate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(sizeof(long long) << kRotMaxBlockLog2)) == cudaSuccess ? 0 : -1;
}

cudaError_t launch_rotate(const __half *x, __half *y, const uint32_t *negate, int64_t n, int block_log2, bool pdl,
                          cudaStream_t s) {
    const int chunk_log2 = block_log2 > kRotMinChunkLog2 ? block_log2 : kRotMinChunkLog2;
    const long long chunk = 1ll << chunk_log2;
    const double scale = std::ldexp(1.0 / std::sqrt((double)(1ll << block_log2)), -24);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((n + chunk - 1) / chunk));
    cfg.blockDim = dim3(kRotThreads);
    cfg.dynamicSmemBytes = sizeof(long long) << chunk_log2;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    long long nn = n;
    return cudaLaunchKernelEx(&cfg, rotate_kernel, x, y, negate, nn, chunk_log2, block_log2, scale);
}

}  // namespace llvq
