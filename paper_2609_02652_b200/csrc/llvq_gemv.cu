// The fused dequantize-plus-matvec (paper Sec. 2.3, "The kernel"), re-designed for sm_100a.
//
// Geometry.  A lane owns a row: the 32 lanes of a warp work on the 32 rows of one row group and
// walk the same block columns together, so every read of x is a shared-memory broadcast and no
// shuffle reduction is needed.  The records of a launch form one sequence of units - a unit is a
// tile of four block columns of a row group, or the row group's last nb mod 4 columns - and the
// sequence is cut into equal contiguous ranges, one per warp of a grid of one CTA a
// multiprocessor, so every warp streams the same number of bytes (give or take one unit).
//
// Reduction.  The float sum of a unit (at most four blocks, fixed order) is converted to fixed
// point and from there on everything is integer: a warp adds its units of a row group in a
// 64-bit register and hands the sum, with the number of units it covers, to the row's 64-bit
// accumulator in the context's scratch by one atomic add.  Integer addition is exact and
// order-free, so a row's result does not depend on how the units were dealt or on which warp
// arrives last; the arrival that completes the unit count converts the total back to float,
// applies the row scale, writes y and clears the accumulator.  The quantum is 2^-39 of a bound on
// a unit's sum derived from max |x| and the gain, i.e. far below f32 resolution.
//
// Decode.  One rotate and one three-input logic op turn a payload word into a pair of fp16 bit
// patterns whose value is (+-)|x_i| * 2^-21 (a subnormal built in place: level bits at [6:4],
// the class parity or-ed in at bit 3, the sign at bit 15).  A mixed-precision fused multiply-add
// (fp16 x fp16 + f32, one instruction) accumulates the exact product with the fp16 activation.
// Per block one multiply applies gain[g] * 2^21 / (4 sqrt m), looked up by the class id.  Every
// lane runs the same instructions whatever its class.
//
// Memory.  Each warp streams its units through a private ring of 1792-byte shared-memory slots
// filled by bulk asynchronous copies (cp.async.bulk, completion on an mbarrier) that lane 0 issues
// kSlots units ahead.  The first copies go out before the kernel waits for its predecessor in the
// stream (records never depend on it), so under programmatic dependent launch the ring fills
// while the previous kernel drains.  Every wait is bounded.
#include <cmath>
#include <cstring>

#include "llvq_internal.cuh"

// Optional timeline (compiled in only with -DLLVQ_TRACE, never in the shipped library): lane 0 of
// every warp stores the global timer at a few points of the kernel.
#ifdef LLVQ_TRACE
#define LLVQ_TRACE_POINT(i)                                                                                       \
    if (p.trace && lane == 0) {                                                                                   \
        unsigned long long t_;                                                                                    \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                                    \
        p.trace[(((size_t)p.trace_launch * gridDim.x + blockIdx.x) * kWarps + warp) * 128 + (i)] = t_;            \
    }
// per-unit timeline of every warp: slot 8 + 3*n + {0: wait begins, 1: data there, 2: decoded}, n < 40
#define LLVQ_TRACE_UNIT(n, i)                                                                                     \
    if (p.trace && lane == 0 && (n) < 40) {                                                                       \
        unsigned long long t_;                                                                                    \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                                    \
        p.trace[(((size_t)p.trace_launch * gridDim.x + blockIdx.x) * kWarps + warp) * 128 + 8 + 3 * (n) + (i)] = t_; \
    }
// SM cycle counter into slots 120..127
#define LLVQ_TRACE_CLOCK(i)                                                                                       \
    if (p.trace && lane == 0)                                                                                     \
        p.trace[(((size_t)p.trace_launch * gridDim.x + blockIdx.x) * kWarps + warp) * 128 + 120 + (i)] = clock64();
#else
#define LLVQ_TRACE_POINT(i)
#define LLVQ_TRACE_UNIT(n, i)
#define LLVQ_TRACE_CLOCK(i)
#endif

namespace llvq {
namespace {

#ifndef LLVQ_WARPS
#define LLVQ_WARPS 16
#endif
#ifndef LLVQ_SLOTS
#define LLVQ_SLOTS 3
#endif
#ifndef LLVQ_MINB
#define LLVQ_MINB 1
#endif
constexpr int kWarps = LLVQ_WARPS;         // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kSlots = LLVQ_SLOTS;         // ring slots per warp
constexpr uint32_t kPairMask = 0x80708070u;

// fixed-point accumulator word: bits 53..63 count units, bits 0..52 sum the biased unit values
constexpr int kCountShift = 53;
constexpr unsigned long long kSumMask = (1ull << kCountShift) - 1;
constexpr long long kUnitBias = 1ll << 41;     // a unit's value is below 2^40 quanta in magnitude

__device__ __forceinline__ void fma_pair(float &lo, float &hi, uint32_t w, uint32_t x) {
    asm("{\n\t.reg .f16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %2;\n\t"
        "mov.b32 {xl, xh}, %3;\n\t"
        "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.f16 %1, wh, xh, %1;\n\t}"
        : "+f"(lo), "+f"(hi)
        : "r"(w), "r"(x));
}
// the same with a zero addend: starts the two chains without clearing registers first
__device__ __forceinline__ void mul_pair(float &lo, float &hi, uint32_t w, uint32_t x) {
    asm("{\n\t.reg .f16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %2;\n\t"
        "mov.b32 {xl, xh}, %3;\n\t"
        "fma.rn.f32.f16 %0, wl, xl, 0f00000000;\n\t"
        "fma.rn.f32.f16 %1, wh, xh, 0f00000000;\n\t}"
        : "=f"(lo), "=f"(hi)
        : "r"(w), "r"(x));
}

// sum over the 24 coordinates of one block of (+-|x_i| * 2^-21) * x[i]
__device__ __forceinline__ float block_dot(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t parity, const uint4 *xs) {
    float a0, a1;
    const uint32_t w[3] = {w0, w1, w2};
#pragma unroll
    for (int j = 0; j < 3; j++) {
        const uint4 xv = xs[j];                      // x[8j .. 8j+7] as four fp16 pairs (broadcast read)
        const uint32_t xp[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const uint32_t r = k ? __funnelshift_r(w[j], w[j], 4 * k) : w[j];
            const uint32_t v = (r & kPairMask) | parity;
            // two chains of twelve (measured faster than four of six)
            if (j == 0 && k == 0) mul_pair(a0, a1, v, xp[k]); else fma_pair(a0, a1, v, xp[k]);
        }
    }
    return a0 + a1;
}

// one-hot record: value = class table entry of the rank level, selected without indexing
__device__ __forceinline__ float onehot_dot(const uint32_t v[5], const float *__restrict__ val, const __half *xs) {
    const uint32_t smask = v[0], m1 = v[1], m2 = v[2], m3 = v[3], m4 = v[4];
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int i = 0; i < 24; i++) {
        float m = val[0];
        if ((m1 >> i) & 1) m = val[1];
        if ((m2 >> i) & 1) m = val[2];
        if ((m3 >> i) & 1) m = val[3];
        if ((m4 >> i) & 1) m = val[4];
        if ((smask >> i) & 1) m = -m;
        const float xv = __half2float(xs[i]);
        if (i & 1) a1 = fmaf(m, xv, a1); else a0 = fmaf(m, xv, a0);
    }
    return a0 + a1;
}

__device__ __forceinline__ int find_problem(const GemvParams &p, int group) {
    int q = 0;
#pragma unroll
    for (int i = 1; i < LLVQ_MAX_GROUP; i++)
        if (i < p.nprob && group >= p.prob[i].group_begin) q = i;
    return q;
}

// running maximum of |fp16| over both halves of a word, kept as two 15-bit patterns
__device__ __forceinline__ uint32_t max_abs_pair(uint32_t m, uint32_t x2) {
    const uint32_t a = x2 & 0x7fff7fffu;
    const __half2 r = __hmax2(*reinterpret_cast<const __half2 *>(&m), *reinterpret_cast<const __half2 *>(&a));
    return *reinterpret_cast<const uint32_t *>(&r);
}

// exact power of two as a float, |e| < 126
__device__ __forceinline__ float pow2f(int e) { return __int_as_float((127 + e) << 23); }

// The contiguous range of units [u0, u0 + n) of this warp; warps are numbered with the CTA index
// fastest, so the ranges that are one unit longer spread over all multiprocessors.  The host
// supplies total_units divided by the number of warps of the grid.
__device__ __forceinline__ void warp_range(const GemvParams &p, int warp, int &u0, int &n) {
    const int gw = warp * gridDim.x + blockIdx.x;
    u0 = gw * p.units_base + min(gw, p.units_rem);
    n = p.units_base + (gw < p.units_rem ? 1 : 0);
}

// Hands the warp's sum over `count` units of row group `group` to the row accumulators.
__device__ __forceinline__ void deliver(const GemvParams &p, const GemvProblemDev &pr, int group, int lane,
                                        long long sum, int count, int qexp, float row_scale) {
    const int row = (group - pr.group_begin) * kRowsPerGroup + lane;
    if (row >= pr.rows) return;                      // padding rows of the last row group
    const unsigned long long addend = (unsigned long long)(sum + (long long)count * kUnitBias) + ((unsigned long long)count << kCountShift);
    unsigned long long *slot = p.accum + (size_t)group * 32 + lane;
    const unsigned long long old = atomicAdd(slot, addend);
    if ((int)(old >> kCountShift) + count == p.units) {
        const long long total = (long long)((old + addend) & kSumMask) - (long long)p.units * kUnitBias;
        pr.y[row] = ((float)total * pow2f(qexp)) * row_scale;
        *slot = 0ull;                                // ready for the next launch on this context
    }
}

// ---- asynchronous copies: global -> shared, completion counted on an mbarrier in shared memory
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Every wait is bounded in time: a poll that fails starts a clock, and once kWaitLimitCycles SM cycles
// (about a second) have passed without the barrier completing, the caller records an error and winds
// down.  The first poll reads no clock, so a wait that is already satisfied costs one instruction.
constexpr long long kWaitLimitCycles = 2000000000ll;
__device__ __forceinline__ bool mbar_wait_for(uint32_t bar, uint32_t parity, long long limit_cycles) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    do {
        if (mbar_try(bar, parity)) return true;
    } while (clock64() - t0 < limit_cycles);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) { return mbar_wait_for(bar, parity, kWaitLimitCycles); }

// Ring reads through 32-bit shared-memory addresses.  Volatile: they must stay behind the wait on the
// slot's barrier and ahead of the copy that refills the slot.
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}

// Returns zero, but only once its operands are available: an address that adds this zero cannot be
// formed before the loads that produced them have completed.
__device__ __forceinline__ uint32_t settled(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t z;
    asm volatile("lop3.b32 %0, %1, %2, %3, 0x00;" : "=r"(z) : "r"(a), "r"(b), "r"(c));
    return z;
}

// First byte of a row group's records, and the matrix it belongs to.
__device__ __forceinline__ const uint8_t *group_base(const GemvParams &p, int group, int cell_bytes, int &q) {
    q = find_problem(p, group);
    return p.prob[q].layout + (size_t)(group - p.prob[q].group_begin) * (size_t)p.nb * cell_bytes;
}

template <bool NO_WEIGHTS>
__global__ void __launch_bounds__(kThreads, LLVQ_MINB) gemv_planes_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    // shared memory: ring | per-matrix block constants (1024 x {scale * gain, parity}) | x | barriers
    unsigned char *ring = smem;
    float2 *tab = reinterpret_cast<float2 *>(smem + kWarps * kSlots * kTileBytes);
    const uint4 *xs = reinterpret_cast<const uint4 *>(smem + kWarps * kSlots * kTileBytes + p.nprob * 8192);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kWarps * kSlots * kTileBytes + p.nprob * 8192 + ((p.nb * 48 + 127) / 128) * 128);
    uint32_t *warp_max = reinterpret_cast<uint32_t *>(bars + kWarps * kSlots);     // one slot a warp
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t my_ring = smem_addr(ring + warp * kSlots * kTileBytes);
    const uint32_t my_bar = smem_addr(bars + warp * kSlots);

    LLVQ_TRACE_POINT(0)
    // first the loads whose latency the rest of the prologue can cover: the class constants this
    // thread will turn into block constants, and x on its way into L2 (its values are read only after
    // the wait below, through L2, which is where the previous kernel's writes to x land)
    const int tab_entries = p.nprob * 1024;
    float2 cv[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int i = 0; i < 2; i++)
        if (tid + i * kThreads < tab_entries) cv[i] = __ldg(p.cls_pack + ((tid + i * kThreads) & 511));
    for (int e = tid * 128; e < p.nb * 48; e += kThreads * 128) {
        // a load whose value is thrown away: it brings the line into L2 and the translation into this
        // multiprocessor's TLB, which a prefetch hint does not promise
        uint32_t ignored;
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(ignored) : "l"(reinterpret_cast<const char *>(p.x) + e));
    }
    // a warp's barriers are used by that warp alone: no block-wide synchronisation is needed for them
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kSlots; s++) mbar_init(my_bar + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    int u0, n_units;
    warp_range(p, warp, u0, n_units);
    // consume side: row group and unit inside it; issue side: a running source pointer
    int group = u0 / p.units, k = u0 - group * p.units, q = 0;
    const uint8_t *src = nullptr;
    int ik = k, igroup = group, issued = 0;
    if (n_units > 0) src = group_base(p, group, kCellBytes, q) + (size_t)(k < p.tiles ? k : p.tiles) * kTileBytes;
    const uint32_t tail_bytes = (uint32_t)p.tail_cells * kCellBytes;

    // issue the copy of the next unit (lane 0 alone, by predicate) onto barrier `b` and buffer `dst`,
    // then step the source
    auto issue = [&](uint32_t b, uint32_t dst) {
        const uint32_t bytes = ik < p.tiles ? (uint32_t)kTileBytes : tail_bytes;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.eq.u32 p, %0, 0;\n\t"
            "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%1], %2;\n\t"
            "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%3], [%4], %2, [%1];\n\t}"
            ::"r"(lane), "r"(b), "r"(bytes), "r"(dst), "l"(src));
        // No "memory" clobber: the only memory the copy writes is the slot, whose last reads feed
        // `dst` through settled() and whose next reads follow the next wait on `b`; a clobber here
        // would pin every shared-memory read of the decode behind the copy.
        issued++;
        src += bytes;                                  // a row group's units are contiguous, and so are a matrix's row groups
        if (++ik == p.units) {
            ik = 0;
            igroup++;
            if (igroup < p.total_groups && issued < n_units) { int qi; src = group_base(p, igroup, kCellBytes, qi); }
        }
    };

    if (!NO_WEIGHTS) {
#pragma unroll
        for (int s = 0; s < kSlots; s++)
            if (issued < n_units) issue(my_bar + 8 * s, my_ring + s * kTileBytes);
    }
    // block constants of every matrix of the launch: (class | gain << 9) -> {gain * 2^21 / (4 sqrt m), parity pattern}
    for (int e = tid, i = 0; e < tab_entries; e += kThreads, i++) {
        const float2 v = i < 2 ? cv[i] : __ldg(p.cls_pack + (e & 511));
        const GemvProblemDev &pe = p.prob[e >> 10];
        tab[e] = make_float2(v.x * ((e & 512) ? pe.gain1 : pe.gain0), v.y);
    }
    // let the next kernel in the stream start its own prefetch, then wait for the previous one:
    // x, y and the reduction scratch may still be in use by it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    LLVQ_TRACE_POINT(1)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    LLVQ_TRACE_POINT(2)
    LLVQ_TRACE_CLOCK(0)
    // x into shared memory, every thread a 16-byte piece (L2 hits after the prefetch), and on the way
    // the largest |x|: every |x| is below 2^(e-14), e the biased exponent of the largest magnitude
    // (fp16 bit patterns of non-negative values order like integers)
    bool failed = false;
    int xexp;
    {
        uint32_t m = 0;
        const uint4 *xg = reinterpret_cast<const uint4 *>(p.x);
        uint4 *xw = const_cast<uint4 *>(xs);
        // all of a thread's loads go out before the first store, so their latencies overlap
        const int nx = p.nb * 3;
        for (int base = 0; base < nx; base += 4 * kThreads) {
            uint4 v[4];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int e = base + i * kThreads + tid;
                v[i] = e < nx ? __ldcg(xg + e) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int e = base + i * kThreads + tid;
                if (e < nx) xw[e] = v[i];
                m = max_abs_pair(max_abs_pair(max_abs_pair(max_abs_pair(m, v[i].x), v[i].y), v[i].z), v[i].w);
            }
        }
        LLVQ_TRACE_POINT(4)
        LLVQ_TRACE_CLOCK(1)
        m = __reduce_max_sync(0xffffffffu, max(m & 0xffffu, m >> 16));
        if (lane == 0) warp_max[warp] = m;             // plain stores: atomics on one word would serialise the warps
        __syncthreads();                               // publishes x, the maxima and the block constants
        m = warp_max[lane < kWarps ? lane : 0];
        xexp = max((int)(__reduce_max_sync(0xffffffffu, m) >> 10), 1) - 14;
    }
    LLVQ_TRACE_POINT(3)
    LLVQ_TRACE_CLOCK(2)

    int n = 0;
    uint32_t parity = 0;                               // every slot completes once a round of kSlots units
    uint32_t bar = my_bar;                             // barrier and buffer of the slot that is consumed next
    uint32_t sbuf = my_ring;
    const uint32_t sbuf_end = my_ring + kSlots * kTileBytes;
    const uint32_t lane16 = 16 * lane, lane8 = 8 * lane;
    const int tiles = p.tiles, units = p.units;

    // A run is the stretch of units of one row group inside this warp's range: its units are summed
    // in a register and handed over together.
    while (n < n_units && !failed) {
        const GemvProblemDev &pr = p.prob[q];
        const int qexp = xexp + pr.qexp_base;
        const float inv_q = pow2f(-qexp);
        const float2 *tq = tab + q * 1024;
        const int run = min(units - k, n_units - n);
        const int run_tiles = NO_WEIGHTS ? 0 : max(0, min(run, tiles - k));
        // the row's scale is needed only by the arrival that finishes the row, but loading it now
        // keeps a cold read off the tail of the kernel
        const int row = (group - pr.group_begin) * kRowsPerGroup + lane;
        const float row_scale = row < pr.rows ? __half2float(pr.row_scale[row]) : 0.f;
        const uint4 *xc = xs + 12 * k;
        long long sum = 0;

        for (int t = 0; t < run_tiles; t++, xc += 12) {
            LLVQ_TRACE_UNIT(n + t, 0)
            if (!mbar_wait(bar, parity)) { failed = true; break; }
            LLVQ_TRACE_UNIT(n + t, 1)
            const uint4 a0 = lds128(sbuf + lane16);
            const uint4 a1 = lds128(sbuf + lane16 + 512);
            const uint4 a2 = lds128(sbuf + lane16 + 1024);
            const uint2 hh = lds64(sbuf + lane8 + 1536);
            const uint32_t w0[4] = {a0.x, a0.y, a0.z, a0.w}, w1[4] = {a1.x, a1.y, a1.z, a1.w}, w2[4] = {a2.x, a2.y, a2.z, a2.w};
            const uint32_t hd[4] = {hh.x & 0xffffu, hh.x >> 16, hh.y & 0xffffu, hh.y >> 16};
            // The slot's words are in registers: refill it at once with the unit kSlots ahead, so
            // that every slot but the one just read is in flight while this unit is decoded.  The
            // copy's address is made to depend on the loaded words, which holds the copy back
            // until the four shared-memory reads of the whole warp have completed.
            if (issued < n_units) issue(bar, sbuf + (settled(a0.w, a1.w, a2.w) | settled(hh.y, hh.x, a0.x)));
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < 4; c++) {
#ifdef LLVQ_STREAM_ONLY
                s += __uint_as_float((w0[c] ^ w1[c] ^ w2[c] ^ hd[c]) & 0x007fffffu);   // debug: bytes only, no decode
#else
                const float2 kc = tq[hd[c]];           // header bits 10..15 are zero
                s = fmaf(kc.x, block_dot(w0[c], w1[c], w2[c], __float_as_uint(kc.y), xc + 3 * c), s);
#endif
            }
            sum += __float2ll_rn(s * inv_q);
            LLVQ_TRACE_UNIT(n + t, 2)
            bar += 8;
            sbuf += kTileBytes;
            const bool wrap = sbuf == sbuf_end;        // every slot completes once a round
            sbuf = wrap ? my_ring : sbuf;
            bar = wrap ? my_bar : bar;
            parity ^= wrap ? 1u : 0u;
        }
        if (failed) break;
        if (!NO_WEIGHTS && run_tiles < run) {
            // the run ends with the nb mod 4 last block columns of the row group: one cell at a time
            if (!mbar_wait(bar, parity)) { failed = true; break; }
            uint32_t guard = 0;
            const uint4 *xt = xs + 12 * tiles;
            float s = 0.f;
#pragma unroll 1
            for (int c = 0; c < p.tail_cells; c++) {
                const uint32_t cell = sbuf + c * kCellBytes;
                const uint32_t t0 = lds32(cell + 4 * lane);
                const uint32_t t1 = lds32(cell + 128 + 4 * lane);
                const uint32_t t2 = lds32(cell + 256 + 4 * lane);
                const uint32_t th = lds16(cell + 384 + 2 * lane);
                guard |= settled(t0, t1, t2) | settled(th, t0, t1);
                const float2 kc = tq[th];
                s = fmaf(kc.x, block_dot(t0, t1, t2, __float_as_uint(kc.y), xt + 3 * c), s);
            }
            if (issued < n_units) issue(bar, sbuf + guard);
            sum += __float2ll_rn(s * inv_q);
            bar += 8;
            sbuf += kTileBytes;
            if (sbuf == sbuf_end) { sbuf = my_ring; bar = my_bar; parity ^= 1u; }
        }
        // with no records read (the control launch) every unit contributes zero
        n += run;
        k += run;
        if (n == n_units) { LLVQ_TRACE_POINT(6) }
        deliver(p, pr, group, lane, sum, run, qexp, row_scale);
        if (k == units) {
            k = 0;
            group++;
            if (group < p.total_groups) q = find_problem(p, group);
        }
    }

    LLVQ_TRACE_POINT(5)
    if (failed) {
        // a wait ran out: report it, then give the copies still in flight a bounded chance to land
        // (a slot that is not pending returns at once or runs into the same bound)
        if (lane == 0) atomicExch(p.error, 1);
        for (int s = 0; s < kSlots && s < issued; s++) mbar_wait(my_bar + 8 * s, parity);
    }
}

// Exercises the wait limit without any fault: one warp waits, for about a millisecond, on a barrier
// that nothing will ever complete, then reports through the same error flag the GEMV uses.
__global__ void wait_limit_selftest_kernel(int *error) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_addr(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (!mbar_wait_for(b, 0, 2000000ll) && threadIdx.x == 0) atomicExch(error, 1);
}

// One-hot comparison arm: same unit sequence, same reduction, records read with plain loads.
__global__ void __launch_bounds__(kThreads, 1) gemv_onehot_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    uint4 *xs4 = reinterpret_cast<uint4 *>(smem);
    const __half *xs = reinterpret_cast<const __half *>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ uint32_t xor_word;
    if (tid == 0) xor_word = 0;
    const uint4 *xg = reinterpret_cast<const uint4 *>(p.x);
    uint32_t m = 0;
    for (int e = tid; e < 3 * p.nb; e += kThreads) {
        const uint4 v = __ldg(xg + e);
        xs4[e] = v;
        m = max_abs_pair(max_abs_pair(max_abs_pair(max_abs_pair(m, v.x), v.y), v.z), v.w);
    }
    __syncthreads();
    m = __reduce_max_sync(0xffffffffu, max(m & 0xffffu, m >> 16));
    if (lane == 0 && m) atomicMax(&xor_word, m);
    __syncthreads();
    const int xexp = max((int)(xor_word >> 10), 1) - 14;

    int u0, n_units;
    warp_range(p, warp, u0, n_units);
    int group = u0 / p.units, k = u0 - group * p.units, q = 0;
    const uint8_t *grp = n_units > 0 ? group_base(p, group, kOneHotCellBytes, q) : nullptr;
    long long sum = 0;
    int count = 0;
    for (int n = 0; n < n_units; n++) {
        const GemvProblemDev &pr = p.prob[q];
        const int qexp = xexp + pr.qexp_base;
        const int c0 = k * kTileCells, c1 = k < p.tiles ? c0 + kTileCells : p.nb;
        float s = 0.f;
        for (int c = c0; c < c1; c++) {
            const uint32_t *cell = reinterpret_cast<const uint32_t *>(grp + (size_t)c * kOneHotCellBytes);
            uint32_t v[5];
#pragma unroll
            for (int t = 0; t < 5; t++) v[t] = __ldcs(cell + 32 * t + lane);
            const int cid = (int)(v[0] >> 24) | (int)(((v[1] >> 24) & 1u) << 8);
            const float g = ((v[1] >> 25) & 1u) ? pr.gain1 : pr.gain0;
            const float4 lv = __ldg(reinterpret_cast<const float4 *>(p.cls_value + cid * 8));
            const float l4 = __ldg(p.cls_value + cid * 8 + 4);
            const float val[5] = {lv.x, lv.y, lv.z, lv.w, l4};
            s = fmaf(g, onehot_dot(v, val, xs + 24 * c), s);
        }
        sum += __float2ll_rn(s * pow2f(-qexp));
        count++;
        if (++k == p.units || n + 1 == n_units) {
            const int row = (group - pr.group_begin) * kRowsPerGroup + lane;
            deliver(p, pr, group, lane, sum, count, qexp, row < pr.rows ? __half2float(pr.row_scale[row]) : 0.f);
            sum = 0;
            count = 0;
            if (k == p.units) {
                k = 0;
                group++;
                if (group < p.total_groups) grp = group_base(p, group, kOneHotCellBytes, q);
            }
        }
    }
}

// FP16 control: one warp per row, 128-bit loads, f32 accumulation.
__global__ void __launch_bounds__(256) gemv_fp16_kernel(const __half *__restrict__ W, const __half *__restrict__ x, float *__restrict__ y,
                                                         int64_t rows, int64_t k) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const uint4 *wr = reinterpret_cast<const uint4 *>(W + row * k);
    const uint4 *xr = reinterpret_cast<const uint4 *>(x);
    const int64_t n = k / 8;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    for (int64_t i = lane; i < n; i += 32) {
        const uint4 wv = __ldcs(wr + i);
        const uint4 xv = __ldg(xr + i);
        fma_pair(a0, a1, wv.x, xv.x);
        fma_pair(a2, a3, wv.y, xv.y);
        fma_pair(a0, a1, wv.z, xv.z);
        fma_pair(a2, a3, wv.w, xv.w);
    }
    float s = (a0 + a1) + (a2 + a3);
#pragma unroll
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) y[row] = s;
}

// ---- helpers reading a record back: thread = (row group, block column, lane)
__device__ __forceinline__ void read_planes_record(const uint8_t *buf, int64_t nb, int64_t rg, int64_t b, int lane,
                                                   uint32_t w[3], uint32_t &hdr) {
    const int64_t tiles = nb / kTileCells;
    const uint8_t *grp = buf + (size_t)rg * (size_t)nb * kCellBytes;
    if (b < tiles * kTileCells) {
        const uint8_t *tile = grp + (size_t)(b / kTileCells) * kTileBytes;
        const int q = (int)(b % kTileCells);
        for (int j = 0; j < 3; j++) w[j] = *reinterpret_cast<const uint32_t *>(tile + 512 * j + 16 * lane + 4 * q);
        hdr = *reinterpret_cast<const uint16_t *>(tile + 1536 + 8 * lane + 2 * q);
    } else {
        const uint8_t *cell = grp + (size_t)tiles * kTileBytes + (size_t)(b - tiles * kTileCells) * kCellBytes;
        for (int j = 0; j < 3; j++) w[j] = *reinterpret_cast<const uint32_t *>(cell + 128 * j + 4 * lane);
        hdr = *reinterpret_cast<const uint16_t *>(cell + 384 + 2 * lane);
    }
}

// integer coordinates of one record, either layout
__device__ __forceinline__ void record_coords(int layout, const uint8_t *buf, int64_t nb, int64_t rg, int64_t b, int lane,
                                              const uint32_t *cls_parity, const uint8_t *cls_dist, int &cls, int &gain, int x[24]) {
    if (layout == LLVQ_PLANES) {
        uint32_t w[3], hdr;
        read_planes_record(buf, nb, rg, b, lane, w, hdr);
        cls = (int)(hdr & 511u); gain = (int)((hdr >> 9) & 1u);
        const int par = cls_parity[cls] ? 1 : 0;
        for (int i = 0; i < 24; i++) {
            const int j = i >> 3, k = (i & 7) >> 1, e = i & 1;
            const uint32_t r = __funnelshift_r(w[j], w[j], 4 * k);
            const int level = (int)((r >> (4 + 16 * e)) & 7u);
            const int a = (cls == kEmptyClass) ? 0 : 2 * level + par;
            x[i] = ((r >> (15 + 16 * e)) & 1u) ? -a : a;
        }
    } else {
        const uint32_t *cell = reinterpret_cast<const uint32_t *>(buf + ((size_t)rg * (size_t)nb + (size_t)b) * kOneHotCellBytes);
        uint32_t v[5];
        for (int t = 0; t < 5; t++) v[t] = cell[32 * t + lane];
        cls = (int)(v[0] >> 24) | (int)(((v[1] >> 24) & 1u) << 8);
        gain = (int)((v[1] >> 25) & 1u);
        const uint8_t *dist = cls_dist + cls * 8;
        for (int i = 0; i < 24; i++) {
            int level = 0;
            for (int t = 1; t <= 4; t++) if ((v[t] >> i) & 1u) level = t;
            const int a = dist[level];
            x[i] = ((v[0] >> i) & 1u) ? -a : a;
        }
    }
}

__global__ void __launch_bounds__(256) decode_i8_kernel(int layout, const uint8_t *__restrict__ buf, int8_t *__restrict__ coords,
                                                         uint16_t *__restrict__ class_ids, int64_t rows, int64_t nb,
                                                         const uint32_t *cls_parity, const uint8_t *cls_dist) {
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = (int)(gid & 31);
    const int64_t cell_id = gid >> 5, groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (cell_id >= groups * nb) return;
    const int64_t rg = cell_id / nb, b = cell_id % nb, row = rg * kRowsPerGroup + lane;
    if (row >= rows) return;
    int cls, gain, x[24];
    record_coords(layout, buf, nb, rg, b, lane, cls_parity, cls_dist, cls, gain, x);
    for (int i = 0; i < 24; i++) coords[(row * nb + b) * 24 + i] = (int8_t)x[i];
    class_ids[row * nb + b] = (uint16_t)cls;
}

__global__ void __launch_bounds__(256) dequant_kernel(int layout, const uint8_t *__restrict__ buf, const __half *__restrict__ row_scale,
                                                       float g0, float g1, __half *__restrict__ W, int64_t rows, int64_t nb,
                                                       const uint32_t *cls_parity, const uint8_t *cls_dist, const float *cls_scale) {
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = (int)(gid & 31);
    const int64_t cell_id = gid >> 5, groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (cell_id >= groups * nb) return;
    const int64_t rg = cell_id / nb, b = cell_id % nb, row = rg * kRowsPerGroup + lane;
    if (row >= rows) return;
    int cls, gain, x[24];
    record_coords(layout, buf, nb, rg, b, lane, cls_parity, cls_dist, cls, gain, x);
    // r * gain / (4 sqrt m): cls_scale carries 2^21 / (4 sqrt m)
    const float s = __half2float(row_scale[row]) * ((gain ? g1 : g0) * (cls_scale[cls] * (1.0f / 2097152.0f)));
    __half *dst = W + (row * nb + b) * 24;
    for (int i = 0; i < 24; i++) dst[i] = __float2half_rn(s * (float)x[i]);
}

}  // namespace

size_t gemv_smem_bytes(int layout, int nb, int nprob) {
    const size_t xbytes = ((size_t)nb * 48 + 127) / 128 * 128;
    if (layout != LLVQ_PLANES) return xbytes;
    return (size_t)kWarps * kSlots * kTileBytes + (size_t)nprob * 8192 + xbytes + kWarps * kSlots * 8 + kWarps * 4 + 16;
}

template <typename K>
static int allow_max_smem(K kernel, int optin) {
    cudaFuncAttributes a;
    if (cudaFuncGetAttributes(&a, kernel) != cudaSuccess) return -1;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)a.sharedSizeBytes) != cudaSuccess) return -1;
    // ask for the largest shared-memory carve-out, so that a CTA of the next kernel of the stream can
    // settle beside a running one (programmatic dependent launch) whenever two of them fit
    return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess ? 0 : -1;
}

int gemv_configure(const llvq_ctx *ctx) {
    const int bytes = ctx->max_smem_optin;
    if (allow_max_smem(gemv_planes_kernel<false>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<true>, bytes)) return -1;
    if (allow_max_smem(gemv_onehot_kernel, bytes)) return -1;
    return 0;
}

cudaError_t launch_gemv(const llvq_ctx *ctx, int layout, GemvParams &p, bool no_weights, cudaStream_t s) {
    const size_t smem = gemv_smem_bytes(layout, p.nb, p.nprob);
    // one CTA a multiprocessor (warps are numbered CTA-first, so a short launch spreads over all of them)
    int grid = p.total_units < ctx->sm_count ? p.total_units : ctx->sm_count;
    p.units_base = p.total_units / (grid * kWarps);
    p.units_rem = p.total_units % (grid * kWarps);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = ctx->use_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (layout == LLVQ_PLANES) {
        if (no_weights) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<true>, p);
        return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false>, p);
    }
    cfg.numAttrs = 0;
    return cudaLaunchKernelEx(&cfg, gemv_onehot_kernel, p);
}

cudaError_t launch_wait_limit_selftest(const llvq_ctx *ctx, cudaStream_t s) {
    wait_limit_selftest_kernel<<<1, 32, 0, s>>>(ctx->error);
    return cudaGetLastError();
}

cudaError_t launch_gemv_fp16(const __half *W, const __half *x, float *y, int64_t rows, int64_t k, cudaStream_t s) {
    const int64_t blocks = (rows + 7) / 8;
    gemv_fp16_kernel<<<(unsigned)blocks, 256, 0, s>>>(W, x, y, rows, k);
    return cudaGetLastError();
}

cudaError_t launch_dequant(const llvq_ctx *ctx, int layout, const uint8_t *buf, const __half *row_scale, float g0, float g1,
                           __half *W, int64_t rows, int64_t nb, cudaStream_t s) {
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    const int64_t blocks = (groups * nb * 32 + 255) / 256;
    dequant_kernel<<<(unsigned)blocks, 256, 0, s>>>(layout, buf, row_scale, g0, g1, W, rows, nb, ctx->dev.cls_parity, ctx->dev.cls_dist,
                                                   ctx->dev.cls_scale);
    return cudaGetLastError();
}

cudaError_t launch_decode_i8(const llvq_ctx *ctx, int layout, const uint8_t *buf, int8_t *coords, uint16_t *class_ids,
                             int64_t rows, int64_t nb, cudaStream_t s) {
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    const int64_t blocks = (groups * nb * 32 + 255) / 256;
    decode_i8_kernel<<<(unsigned)blocks, 256, 0, s>>>(layout, buf, coords, class_ids, rows, nb, ctx->dev.cls_parity, ctx->dev.cls_dist);
    return cudaGetLastError();
}

}  // namespace llvq

// ---------------------------------------------------------------------------------------------
// llvq_gemv_static: the bit-plane GEMV for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a matvec: a serving
// process whose memory pool already owns all of HBM, a plug-in that is handed buffers but no
// allocator, code that runs while a stream is being captured (allocation is not allowed there), or
// a real-time loop in which an allocation's implicit device synchronisation is not acceptable.
// Those callers cannot create a context either, because llvq_create allocates the tables and the
// reduction scratch.  For them everything the kernel needs besides the caller's own buffers lives
// in file-scope __device__ arrays that the module carries: the row accumulators (the scratch), the
// class table and the error flag.  Every GPU that loads the library holds these arrays (about
// 516 KiB) until the process exits.
//
// In host code the name of a __device__ array is only a host-side stand-in, not a device address;
// the kernel is therefore given the address that cudaGetSymbolAddress returns for the current
// device.  That, the upload of the class table and the kernel's shared-memory attribute are done
// by the first call on each device (synchronously), so make that first call before any stream
// capture begins.  All calls share the arrays: the accumulators are left at zero by every launch
// that completes, but two launches that overlap on the GPU (different streams) race on them.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRows = 65536;      // rows (rounded up to 32) one llvq_gemv_static call may have
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) unsigned long long g_static_accum[kStaticMaxRows];   // 512 KiB of scratch
static __device__ __align__(256) float2 g_static_cls_pack[llvq::kClassSlots];           // 4 KiB
static __device__ __align__(256) int g_static_error[64];

struct StaticDevice {
    bool ready = false;
    unsigned long long *accum = nullptr;
    float2 *cls_pack = nullptr;
    int *error = nullptr;
    int sm_count = 0, max_smem_optin = 0;
};
StaticDevice g_static_dev[kStaticMaxDevices];

// Once per device, with that device current: resolve the arrays' device addresses, fill the class
// table, zero the accumulators, raise the kernel's shared-memory limit.  Allocates no device memory.
int static_setup(int device, StaticDevice &d) {
    if (cudaGetSymbolAddress((void **)&d.accum, g_static_accum) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaGetSymbolAddress((void **)&d.cls_pack, g_static_cls_pack) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaGetSymbolAddress((void **)&d.error, g_static_error) != cudaSuccess) return LLVQ_ECUDA;
    llvq::HostTables host;                                   // host memory only
    if (!llvq::build_tables(host)) return LLVQ_EINVAL;
    if (cudaMemcpy(d.cls_pack, host.cls_pack.data(), llvq::kClassSlots * 8, cudaMemcpyHostToDevice) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemset(d.accum, 0, sizeof(unsigned long long) * kStaticMaxRows) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemset(d.error, 0, sizeof(int) * 64) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) return LLVQ_ECUDA;
    if (llvq::allow_max_smem(llvq::gemv_planes_kernel<false>, d.max_smem_optin)) return LLVQ_ECUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return LLVQ_ECUDA;
    d.ready = true;
    return LLVQ_OK;
}

}  // namespace

extern "C" int llvq_gemv_static(const void *layout_buf, const void *row_scale, const float *gain, const void *x, float *y,
                                int64_t rows, int64_t k_padded, void *stream) {
    using namespace llvq;
    if (!layout_buf || !row_scale || !gain || !x || !y || rows <= 0 || k_padded <= 0 || k_padded % 24 != 0) return LLVQ_EINVAL;
    if (k_padded > LLVQ_MAX_K) return LLVQ_ESIZE;
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (groups * kRowsPerGroup > kStaticMaxRows) return LLVQ_ESIZE;      // more rows than the built-in scratch holds
    if ((reinterpret_cast<uintptr_t>(layout_buf) & 127) || (reinterpret_cast<uintptr_t>(x) & 15) ||
        (reinterpret_cast<uintptr_t>(row_scale) & 1) || (reinterpret_cast<uintptr_t>(y) & 3))
        return LLVQ_EALIGN;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return LLVQ_ECUDA;
    if (device < 0 || device >= kStaticMaxDevices) return LLVQ_EINVAL;
    StaticDevice &d = g_static_dev[device];
    if (!d.ready) {
        const int rc = static_setup(device, d);
        if (rc != LLVQ_OK) return rc;
    }
    GemvParams p;
    memset(&p, 0, sizeof p);
    p.nprob = 1;
    p.prob[0].layout = (const uint8_t *)layout_buf;
    p.prob[0].row_scale = (const __half *)row_scale;
    p.prob[0].y = y;
    p.prob[0].rows = (int)rows;
    p.prob[0].group_begin = 0;
    p.prob[0].gain0 = gain[0];
    p.prob[0].gain1 = gain[1];
    {
        const float gm = fmaxf(fabsf(gain[0]), fabsf(gain[1]));
        if (!(gm < 3.0e38f)) return LLVQ_EINVAL;
        int ge = 0;
        frexpf(gm > 0.f ? gm : 1.f, &ge);
        p.prob[0].qexp_base = ge + 5 - 39;               // same quantum as llvq_gemv
    }
    p.x = (const __half *)x;
    p.nb = (int)(k_padded / 24);
    p.tiles = p.nb / kTileCells;
    p.tail_cells = p.nb % kTileCells;
    p.units = p.tiles + (p.tail_cells ? 1 : 0);
    if (p.units > 2047 || groups * p.units > 0x7fffffffll) return LLVQ_ESIZE;
    p.total_groups = (int)groups;
    p.total_units = (int)(groups * p.units);
    p.accum = d.accum;
    p.cls_pack = d.cls_pack;
    p.error = d.error;
    const size_t smem = gemv_smem_bytes(LLVQ_PLANES, p.nb, 1);
    if (smem + 1024 > (size_t)d.max_smem_optin) return LLVQ_ESIZE;
    int grid = p.total_units < d.sm_count ? p.total_units : d.sm_count;
    p.units_base = p.total_units / (grid * kWarps);
    p.units_rem = p.total_units % (grid * kWarps);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false>, p) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

