// The fused dequantize-plus-matvec (paper Sec. 2.3, "The kernel"), re-designed for sm_100a.
//
// Arithmetic.  A block contributes scale * sum_i x_i * x[24b+i] with x_i = 2 u_i + (parity - 16), u_i the
// four-bit code the record stores.  The activations are taken as fixed point, X_i = rint(x_i * 2^F) with F
// set by the largest |x| of the call, and 2 X_i is split into four balanced 8-bit limbs.  The inner sum then
// is an integer contraction that the tensor cores do exactly: mma.sync m16n8k32 / m16n8k16, u8 x s8 -> s32.
// A is 16 rows x 48 positions (two block slots of 24 coordinates) of codes, one byte each once the two nibbles
// of a payload byte are split (one shift, two ANDs a word: the whole decode); B is block-diagonal, its eight
// columns the four limbs of slot 0 and the four limbs of slot 1, so one accumulator tile holds, for 16 rows,
// the two blocks' sums limb by limb.  Per (row, block) the limbs are recombined in integers, the offset term
// (parity - 16) * sum_i X_i is added from a per-block sum prepared with x, and one float multiply-add applies
// gain[g] / (4 sqrt m), looked up by the header.  Every lane runs the same instructions whatever its class.
//
// Geometry.  A warp works on the 32 rows of a row group, 16 at a time; the records are stored as the
// instruction's operand fragments (include/llvq.h), so a lane's 128-bit shared-memory reads are its A
// registers.  The records of a launch form one sequence of units - a unit is a tile of four block columns of
// a row group, or the row group's last nb mod 4 columns - ordered panel by panel (a panel is about sixteen
// consecutive unit columns of every row group).  The sequence is cut into equal contiguous ranges, one per
// warp of a grid of one CTA a multiprocessor, warps numbered CTA by CTA: every warp streams the same number of
// bytes (give or take one unit), and a CTA's units lie in one or two panels, so it prepares only that part
// of x.
//
// Reduction.  After a unit the four lanes that share a row add their shares (two shuffles, fixed order), the
// float sum of the unit (at most four blocks) is converted to fixed point and from there on everything is
// integer: a warp adds its units of a row group in a 64-bit register and hands the sum, with the number of
// units it covers, to the row's 64-bit accumulator in the context's scratch by one atomic add.  Integer
// addition is exact and order-free, so a row's result does not depend on how the units were dealt or on which
// warp arrives last; the arrival that completes the unit count converts the total back to float, applies the
// row scale, writes y and clears the accumulator.  The quantum is 2^-39 of a bound on a unit's sum derived
// from max |x| and the gain, i.e. far below f32 resolution.
//
// Memory.  Each warp streams its units through a private ring of 1792-byte shared-memory slots filled by bulk
// asynchronous copies (cp.async.bulk, completion on an mbarrier) that lane 0 issues kSlots units ahead.  The
// first copies go out before the kernel waits for its predecessor in the stream (records never depend on
// it), so under programmatic dependent launch the ring fills while the previous kernel drains.  Every wait is
// bounded.
#include <cmath>
#include <cstring>
#include <mutex>

#include "llvq_internal.cuh"
#include "llvq_rotate.cuh"

namespace llvq {
namespace {

constexpr int kWarps = 16;                 // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kSlots = 2;                  // ring slots per warp
constexpr int kEarlySlots = 1;             // slots filled before the wait for the previous kernel; the rest once x is being prepared

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
    if (p.nprob == 1) return 0;                      // the common launch: one matrix
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

// The same in two halves, so that a warp does not sit out the atomic's round trip between two runs: hand_over
// sends the sum and remembers what the answer will mean, settle (called at the next hand-over, or at the end)
// reads the answer and, if this arrival completed the row, writes y and clears the accumulator.
struct Handed {
    unsigned long long old, addend;
    unsigned long long *slot;     // null: nothing is pending
    float *y;
    float yscale;
    int count;
};
__device__ __forceinline__ void settle(const GemvParams &p, Handed &h) {
    if (h.slot == nullptr) return;
    if ((int)(h.old >> kCountShift) + h.count == p.units) {
        const long long total = (long long)((h.old + h.addend) & kSumMask) - (long long)p.units * kUnitBias;
        *h.y = (float)total * h.yscale;
        *h.slot = 0ull;                              // ready for the next launch on this context
    }
    h.slot = nullptr;
}
// `accum` and `y` are the accumulators and the output of the activation vector the sum belongs to (a batched
// launch has one set a vector)
__device__ __forceinline__ void hand_over(const GemvParams &p, const GemvProblemDev &pr, unsigned long long *accum, float *y,
                                          int group, int lane, long long sum, int count, int qexp, float row_scale, Handed &h) {
    settle(p, h);
    const int row = (group - pr.group_begin) * kRowsPerGroup + lane;
    if (row >= pr.rows) return;                      // padding rows of the last row group
    h.addend = (unsigned long long)(sum + (long long)count * kUnitBias) + ((unsigned long long)count << kCountShift);
    h.slot = accum + (size_t)group * 32 + lane;
    h.old = atomicAdd(h.slot, h.addend);
    h.y = y + row;
    h.yscale = pow2f(qexp) * row_scale;
    h.count = count;
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
// Returns zero, but only once its operands are available: an address that adds this zero cannot be
// formed before the loads that produced them have completed.
__device__ __forceinline__ uint32_t settled(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t z;
    asm volatile("lop3.b32 %0, %1, %2, %3, 0x00;" : "=r"(z) : "r"(a), "r"(b), "r"(c));
    return z;
}

// First byte of a row group's records, and the matrix it belongs to.
__device__ __forceinline__ const uint8_t *group_base(const GemvParams &p, int group, int &q) {
    if (p.nprob == 1) {                              // the common launch: one matrix
        q = 0;
        return p.prob[0].layout + (size_t)(uint32_t)group * p.group_bytes;
    }
    q = find_problem(p, group);
    return p.prob[q].layout + (size_t)(uint32_t)(group - p.prob[q].group_begin) * p.group_bytes;
}

// ---- integer tensor-core contraction: D (16 rows x 8 columns, s32) = A (16 x k, u8) * B (k x 8, s8) [+ D]
__device__ __forceinline__ void mma_k32(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ void mma_k16(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm("mma.sync.aligned.m16n8k16.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}

// Bytes of x in shared memory, one record a block: four planes of 24 bytes (plane l = limb l of the 24
// fixed-point activations, doubled), a zero word at 96, and at 100 and 104 the two halves of the block's
// activation sum (see stage_x).
constexpr int kXRecBytes = 112;

// Offsets of this lane's operand words inside the two x records of a half-step (or, one = true, inside
// the single record both slots of the row group's last half-step share).  B is block-diagonal: column
// n = lane >> 2 carries limb n & 3 of slot n >> 2, and is zero at the positions of the other slot.
struct LaneOffsets { uint32_t b0, b1, b2, xs; };
__host__ __device__ __forceinline__ LaneOffsets lane_offsets(int lane, bool one) {
    const int g = lane >> 2, t = lane & 3, l = g & 3;
    const uint32_t zero = 96, second = one ? 0 : kXRecBytes;
    LaneOffsets o;
    if (g < 4) {
        o.b0 = 24 * l + 4 * t;                                  // positions 4t..4t+3: slot 0, coordinates 4t..
        o.b1 = t < 2 ? 24 * l + 16 + 4 * t : zero;              // positions 16+4t..: slot 0 up to 23, then slot 1
        o.b2 = zero;                                            // positions 32+4t..: slot 1
    } else {
        o.b0 = zero;
        o.b1 = t >= 2 ? second + 24 * l + 4 * (t - 2) : zero;
        o.b2 = second + 24 * l + 8 + 4 * t;
    }
    o.xs = (one ? 0 : kXRecBytes * (t >> 1)) + 100 + 4 * (t & 1);
    return o;
}

// Shared-memory reads with a constant byte offset folded into the instruction.  Volatile, so that the
// compiler never moves one out of the branch that guards it: an address formed for a unit this CTA does not
// own may lie outside its shared memory.
template <int OFF>
__device__ __forceinline__ uint32_t lds32_at(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
__device__ __forceinline__ float2 lds_f2(uint32_t a) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
}

// The B operand of one step (two block slots) for this lane, and its share of the slots' activation sum.
struct StepX { uint32_t b0, b1, b2; int xsum; };
// a.* are this lane's four addresses for the records at the start of a tile; OFF selects the step
template <int OFF>
__device__ __forceinline__ StepX load_step(const LaneOffsets &a) {
    StepX s;
    s.b0 = lds32_at<OFF>(a.b0); s.b1 = lds32_at<OFF>(a.b1); s.b2 = lds32_at<OFF>(a.b2);
    s.xsum = (int)lds32_at<OFF>(a.xs);
    return s;
}

// One half-step: 16 rows x 2 block slots.  wa, wb, wc are this lane's three payload words, hw the two
// headers of its rows for slot (lane & 3) >> 1, sx the step's operand.  Adds to r0 (row g of the 16) and r1
// (row g + 8) this lane's share of scale * sum_i x_i * X_i, X the fixed-point activations: its share is the
// limb pair (lane & 1) of slot (lane & 3) >> 1.  FIRST: r0 and r1 are written, not added to.
// (a & b) | c in one instruction
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

// The A operand of a half-step (the decode proper: one shift and two ANDs a word) and the block constants of
// its two rows; both are shared by every activation vector of a batched launch.
struct HalfA {
    uint32_t a0, a1, a2, a3, c0, c1;
    float2 k0, k1;
};
// COMPACT (13-byte layout): the two headers are the bytes at bit SHIFT and SHIFT + 8 of hw.
template <bool COMPACT = false, int SHIFT = 0>
__device__ __forceinline__ HalfA decode_half(uint32_t wa, uint32_t wb, uint32_t wc, uint32_t hw, uint32_t tq) {
    constexpr uint32_t kNib = 0x0f0f0f0fu;
    HalfA h;
    h.a0 = wa & kNib; h.a1 = wb & kNib; h.a2 = (wa >> 4) & kNib; h.a3 = (wb >> 4) & kNib;
    h.c0 = wc & kNib; h.c1 = (wc >> 4) & kNib;
    if (COMPACT) {
        // one byte a header, eight bytes an entry
        h.k0 = lds_f2(and_or(SHIFT >= 3 ? hw >> (SHIFT - 3) : hw << (3 - SHIFT), 0x7f8u, tq));
        h.k1 = lds_f2(and_or(hw >> (SHIFT + 5), 0x7f8u, tq));
    } else {
        // the headers of rows g (low half of hw) and g + 8 (high half), eight bytes an entry; tq is 8 KiB-aligned
        h.k0 = lds_f2(and_or(hw << 3, 0x1ff8u, tq));
        h.k1 = lds_f2(and_or(hw >> 13, 0x1ff8u, tq));
    }
    return h;
}
// The 10-byte layout's tile: nine words a lane (va = V0..V3, vb = V4..V7, v8), three bits a code.  Byte i of a word
// carries code i of two operand words in bits 0..2 and 3..5; bits 6, 7 carry the six operand words left over: the low
// two bits of Xk in Vk, its third bit in bit 6 + (k & 1) of V(6 + k / 2).  Two shifts and two ANDs a word pair as in the
// 14-byte layout, four instructions for each of the six.  hb = the eight header bytes of the lane's rows.
template <int K>
__device__ __forceinline__ uint32_t overlay_left_over(uint32_t vk, uint32_t vhigh) {
    // (vk >> 6 & 0x03030303) | (vhigh >> (4 + (K & 1)) & 0x04040404)
    return and_or(vhigh >> (4 + (K & 1)), 0x04040404u, (vk >> 6) & 0x03030303u);
}
template <int SHIFT>
__device__ __forceinline__ void header_consts(uint32_t hw, uint32_t tq, float2 &k0, float2 &k1) {
    k0 = lds_f2(and_or(SHIFT >= 3 ? hw >> (SHIFT - 3) : hw << (3 - SHIFT), 0x7f8u, tq));
    k1 = lds_f2(and_or(hw >> (SHIFT + 5), 0x7f8u, tq));
}
__device__ __forceinline__ void decode_overlay_tile(const uint4 &va, const uint4 &vb, uint32_t v8, const uint2 &hb, uint32_t tq,
                                                    HalfA &h0, HalfA &h1, HalfA &h2, HalfA &h3) {
    constexpr uint32_t k7 = 0x07070707u;
    h0.a0 = va.x & k7; h0.a2 = (va.x >> 3) & k7; h0.a1 = va.y & k7; h0.a3 = (va.y >> 3) & k7;
    h1.a0 = va.z & k7; h1.a2 = (va.z >> 3) & k7; h1.a1 = va.w & k7; h1.a3 = (va.w >> 3) & k7;
    h2.a0 = vb.x & k7; h2.a2 = (vb.x >> 3) & k7; h2.a1 = vb.y & k7; h2.a3 = (vb.y >> 3) & k7;
    h3.a0 = vb.z & k7; h3.a2 = (vb.z >> 3) & k7; h3.a1 = vb.w & k7; h3.a3 = (vb.w >> 3) & k7;
    h0.c0 = v8 & k7; h1.c0 = (v8 >> 3) & k7;
    h0.c1 = overlay_left_over<0>(va.x, vb.z);            // X0 = Group(0, 1, 2): low bits in V0, third bit in V6
    h1.c1 = overlay_left_over<1>(va.y, vb.z);            // X1 = Group(1, 1, 2)
    h2.c0 = overlay_left_over<2>(va.z, vb.w);            // X2 = Group(2, 0, 2): V2 and V7
    h2.c1 = overlay_left_over<3>(va.w, vb.w);            // X3 = Group(2, 1, 2)
    h3.c0 = overlay_left_over<4>(vb.x, v8);              // X4 = Group(3, 0, 2): V4 and V8
    h3.c1 = overlay_left_over<5>(vb.y, v8);              // X5 = Group(3, 1, 2)
    header_consts<0>(hb.x, tq, h0.k0, h0.k1);
    header_consts<16>(hb.x, tq, h1.k0, h1.k1);
    header_consts<0>(hb.y, tq, h2.k0, h2.k1);
    header_consts<16>(hb.y, tq, h3.k0, h3.k1);
}
// nibbles 0..3 of h to the low nibbles of bytes 0..3
__device__ __forceinline__ uint32_t spread_nibbles(uint32_t h) {
    h &= 0xffffu;
    h = (h | (h << 8)) & 0x00ff00ffu;
    return (h | (h << 4)) & 0x0f0f0f0fu;
}
// One entry of the exception table against the x record of its block (`rec`): the block's whole product, in the
// accumulator's quanta.  The arithmetic of the tile path for one block: integer sums limb pair by limb pair, the
// block's scale in f32.  `tail_tab` is the table of the four-bit records' headers (the entry's header byte indexes it).
__device__ __forceinline__ long long exception_value(const uint4 &ent, uint32_t rec, uint32_t tail_tab, float inv_q) {
    const float2 k = lds_f2(tail_tab + 8 * (ent.x & 63u));
    int d[4] = {0, 0, 0, 0};
    uint32_t cw = ent.y;
#pragma unroll
    for (int j = 0; j < 3; j++) {
        const uint32_t lo4 = spread_nibbles(cw), hi4 = spread_nibbles(cw >> 16);
#pragma unroll
        for (int l = 0; l < 4; l++) {
            const uint2 x8 = lds64(rec + 24 * l + 8 * j);
            d[l] = __dp4a((int)hi4, (int)x8.y, __dp4a((int)lo4, (int)x8.x, d[l]));
        }
        cw = j == 0 ? ent.z : ent.w;
    }
    const int off = __float_as_int(k.y);
    const int e_lo = off * (int)lds32(rec + 100) + (d[0] + 256 * d[1]);
    const int e_hi = off * (int)lds32(rec + 104) + (d[2] + 256 * d[3]);
    return __float2ll_rn(((float)e_lo * k.x + ((float)e_hi * k.x) * 65536.f) * inv_q);
}

template <bool FIRST>
__device__ __forceinline__ void contract_half(const HalfA &h, const StepX &sx, float &r0, float &r1) {
    int d[4];
    mma_k32(d, h.a0, h.a1, h.a2, h.a3, sx.b0, sx.b1);
    mma_k16(d, h.c0, h.c1, sx.b2);
    // sum_i x_i X_i = sum_i u_i (2 X_i) + (parity - 16) sum_i X_i, limb pair by limb pair, in integers
    const int e0 = __float_as_int(h.k0.y) * sx.xsum + (d[0] + 256 * d[1]);
    const int e1 = __float_as_int(h.k1.y) * sx.xsum + (d[2] + 256 * d[3]);
    if (FIRST) { r0 = (float)e0 * h.k0.x; r1 = (float)e1 * h.k1.x; }
    else { r0 = fmaf((float)e0, h.k0.x, r0); r1 = fmaf((float)e1, h.k1.x, r1); }
}
template <bool FIRST>
__device__ __forceinline__ void half_step(uint32_t wa, uint32_t wb, uint32_t wc, uint32_t hw, const StepX &sx, uint32_t tq,
                                          float &r0, float &r1) {
    contract_half<FIRST>(decode_half(wa, wb, wc, hw, tq), sx, r0, r1);
}

// x (fp16) -> records.  X_i = rint(x_i * 2^F) with F chosen from the largest |x| so that |X_i| < 2^29; the
// record of a block stores the four balanced limbs of 2 X_i (2 X_i = sum_l limb_l 256^l, limbs in -128..127)
// plane by plane, and the block's sum of the X_i split in two, sum = s0 + 65536 s1.  An item is eight coordinates (one 128-bit piece of x): item e belongs to block e / 3.
// The three items of a block add their shares of s0 and s1 with shared-memory atomics; the words were zeroed
// before.  `rec` is the shared-memory address of the block's record.
__device__ __forceinline__ void convert_item(const uint4 &v, int third, uint32_t rec, float scale) {
    const uint32_t hv[4] = {v.x, v.y, v.z, v.w};
    uint32_t w[8];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&hv[i]));
        const int z0 = __float2int_rn(f.x * scale), z1 = __float2int_rn(f.y * scale);
        w[2 * i] = ((uint32_t)(2 * z0) + 0x80808080u) ^ 0x80808080u;       // bytes = balanced limbs of 2 X
        w[2 * i + 1] = ((uint32_t)(2 * z1) + 0x80808080u) ^ 0x80808080u;
    }
    uint32_t pl[4][2];
    int limb_sum[4] = {0, 0, 0, 0};
#pragma unroll
    for (int hlf = 0; hlf < 2; hlf++) {
        const uint32_t a = w[4 * hlf], b = w[4 * hlf + 1], c = w[4 * hlf + 2], dd = w[4 * hlf + 3];
        const uint32_t t0 = __byte_perm(a, b, 0x5140), t1 = __byte_perm(c, dd, 0x5140);   // limbs 0,1 of a,b / c,d
        const uint32_t t2 = __byte_perm(a, b, 0x7362), t3 = __byte_perm(c, dd, 0x7362);   // limbs 2,3
        pl[0][hlf] = __byte_perm(t0, t1, 0x5410); pl[1][hlf] = __byte_perm(t0, t1, 0x7632);
        pl[2][hlf] = __byte_perm(t2, t3, 0x5410); pl[3][hlf] = __byte_perm(t2, t3, 0x7632);
#pragma unroll
        for (int l = 0; l < 4; l++) limb_sum[l] = __dp4a((int)pl[l][hlf], 0x01010101, limb_sum[l]);
    }
#pragma unroll
    for (int l = 0; l < 4; l++)
        asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(rec + 24 * l + 8 * third), "r"(pl[l][0]), "r"(pl[l][1]) : "memory");
    // this item's sum of 2 X is a0 + 65536 a1; it is even, and so is a0; if a1 is odd one unit of it moves to
    // a0, and then both halve exactly: the item adds a0 / 2 and a1 / 2 to the block's s0 and s1
    int a0 = limb_sum[0] + 256 * limb_sum[1], a1 = limb_sum[2] + 256 * limb_sum[3];
    a0 += (a1 & 1) << 16;
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(rec + 100), "r"(a0 >> 1) : "memory");
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(rec + 104), "r"(a1 >> 1) : "memory");
}

// ---- the order of work.  A unit is a tile of a row group or its leftover blocks (column p.tiles).  Units
// are numbered panel by panel: a panel is p.panel consecutive unit columns (the last panel may be narrower)
// of every row group; inside a panel row group by row group, inside a row group by column.  The sequence is
// cut into equal contiguous ranges, one per warp, warps numbered CTA by CTA: a CTA's range then lies in one
// or two panels, so it needs only those panels' part of x, while a warp still meets several consecutive
// units of one row group (a run), which it sums in registers.
struct Cursor {
    int panel, group, col, end;      // end = first column past the panel
};
__host__ __device__ inline int fast_div(int n, const FastDiv &f, int d) {
#ifdef __CUDA_ARCH__
    (void)d;
    return f.mul ? (int)(__umulhi((uint32_t)n, f.mul) >> f.shift) : n;
#else
    (void)f;
    return n / d;
#endif
}
__host__ __device__ inline int panel_of_unit(const GemvParams &p, int f) {
    const int j = fast_div(f, p.div_panel_units, p.total_groups * p.panel);
    return j < p.npanels ? j : p.npanels - 1;
}
// steps over n units of the current row group's stretch; true if the row group changed
__device__ __forceinline__ bool advance(const GemvParams &p, Cursor &c, int n) {
    c.col += n;
    if (c.col < c.end) return false;
    c.group++;
    if (c.group == p.total_groups) {
        c.group = 0;
        c.panel++;
        c.end = min(c.end + p.panel, p.units);
    }
    c.col = c.panel * p.panel;
    return true;
}
// BATCH activation vectors share one pass over the records: the decode of a half-step and its block constants
// are computed once, the contraction, the scaling and the reduction once a vector.  x is BATCH vectors of
// 24 nb halves one after the other, y BATCH vectors of rows floats (p.prob[].y is vector 0's), the accumulators
// BATCH sets of total_groups * 32.
// ROTATE: x is rotated on its way into the records (llvq_gemv_rotated): every CTA rotates the Walsh-Hadamard
// blocks of x that its share of the matrix touches, exactly as the rotation kernel does, and rounds them to FP16.
// LAYOUT: LLVQ_PLANES; LLVQ_PLANES13 (one header byte a block; the code words are where the 14-byte layout has them);
// LLVQ_PLANES10X (tiles of three-bit codes, leftover blocks as in the 13-byte layout, and after each run the exact
// records of the run's exception blocks, whose short records are empty and add nothing).
template <bool NO_WEIGHTS, int BATCH, bool ROTATE = false, int LAYOUT = LLVQ_PLANES>
__global__ void __launch_bounds__(kThreads, 1) gemv_planes_kernel(const __grid_constant__ GemvParams p) {
    constexpr bool COMPACT = LAYOUT != LLVQ_PLANES, OVERLAY = LAYOUT == LLVQ_PLANES10X;
    static_assert(!OVERLAY || (BATCH == 1 && !ROTATE && !NO_WEIGHTS), "the 10-byte layout: one vector, as it is");
    constexpr int kSrcCell = COMPACT ? kCell13Bytes : kCellBytes;        // bytes of a leftover block column of a row group
    constexpr int kSrcTile = OVERLAY ? kTile10Bytes : (COMPACT ? kTile13Bytes : kTileBytes);   // bytes of a tile in memory (a ring slot always has kTileBytes)
    extern __shared__ __align__(128) unsigned char smem[];
    // shared memory: ring | per-matrix block constants (1024 x {gain / (4 sqrt m), parity - 16}) | x records | barriers
    unsigned char *ring = smem;
    // the block constants start on an 8 KiB boundary of the shared window, so that a matrix's table base and
    // an entry's offset combine by OR (half_step)
    const uint32_t tab_pad = (0u - (smem_addr(smem) + kWarps * kSlots * kTileBytes)) & 8191u;
    float2 *tab = reinterpret_cast<float2 *>(smem + kWarps * kSlots * kTileBytes + tab_pad);
    unsigned char *xrec = smem + kWarps * kSlots * kTileBytes + tab_pad + p.nprob * 8192;
    const uint32_t xrec_stride = ((p.xblocks * kXRecBytes + 127) / 128) * 128;     // a vector's records
    uint64_t *bars = reinterpret_cast<uint64_t *>(xrec + BATCH * xrec_stride);
    uint32_t *warp_max = reinterpret_cast<uint32_t *>(bars + kWarps * kSlots);     // one slot a warp and vector
    long long *rot = reinterpret_cast<long long *>(warp_max + BATCH * kWarps);     // ROTATE: the exact sums of this CTA's blocks of x
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t my_ring = smem_addr(ring + warp * kSlots * kTileBytes);
    const uint32_t my_bar = smem_addr(bars + warp * kSlots);

    // The parameters the start of a CTA needs are read up front, all at once: a parameter line's first read by a
    // multiprocessor costs some two hundred cycles, and the chain below would otherwise meet them one by one.
    const CtaShare me = p.cta[blockIdx.x];
    const int next_first = p.cta[blockIdx.x + 1].first;
    const int h_nprob = p.nprob, h_units = p.units, h_groups = p.total_groups, h_panel = p.panel, h_npanels = p.npanels, h_tiles = p.tiles;
    const FastDiv h_div_panel = p.div_panel, h_div_last = p.div_last;
    const uint32_t h_group_bytes = p.group_bytes, h_tail_cells = (uint32_t)p.tail_cells;
    const uint8_t *h_layout0 = p.prob[0].layout;
    const float2 *h_cls_block = p.cls_block;
    const uint4 *h_lane_table = p.lane_table;
    asm volatile("" ::"r"(me.first), "r"(next_first), "r"(h_nprob), "r"(h_units), "r"(h_groups), "r"(h_panel), "r"(h_npanels), "r"(h_tiles),
                 "r"(h_div_panel.mul), "r"(h_div_last.mul), "r"(h_group_bytes), "r"(h_tail_cells), "l"(h_layout0), "l"(h_cls_block), "l"(h_lane_table));
    // a warp's barriers are used by that warp alone: no block-wide synchronisation is needed for them; they
    // are set up before any load is in flight, so that the fence has nothing to wait for
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kSlots; s++) mbar_init(my_bar + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    // The CTA's units come from the host's plan; its warps share them evenly (the odd ones spread over the
    // warps).  The blocks of x the CTA's units touch, [blk_lo, blk_hi), are those of the panels its range lies in.
    const int cta_u0 = me.first, cta_n = next_first - cta_u0;
    const int u0 = cta_u0 + (warp * cta_n + kWarps - 1) / kWarps;
    const int n_units = cta_u0 + ((warp + 1) * cta_n + kWarps - 1) / kWarps - u0;
    const int blk_lo = me.blk_lo, blk_hi = me.blk_hi;
    const uint32_t xs0 = smem_addr(xrec) - (uint32_t)blk_lo * kXRecBytes;     // address of block 0's record, were it there

    // consume side and issue side walk the same sequence of units.  The warp's first unit lies in the panel of
    // the CTA's first unit (the plan names it) or, seldom, in a later one.
    Cursor cc;
    {
        int panel = me.panel, first = panel * h_panel, w = min(h_panel, h_units - first), r = u0 - me.panel_first;
        while (r >= h_groups * w && panel < h_npanels - 1) {
            r -= h_groups * w;
            panel++;
            first += h_panel;
            w = min(h_panel, h_units - first);
        }
        cc.panel = panel;
        cc.end = first + w;
        cc.group = panel == h_npanels - 1 ? fast_div(r, h_div_last, w) : fast_div(r, h_div_panel, w);
        cc.col = first + (r - cc.group * w);
    }
    Cursor ic = cc;
    int q = 0;
    const uint8_t *isrc = nullptr;                     // first byte of the issue side's row group
    if (n_units > 0) isrc = h_nprob == 1 ? h_layout0 + (size_t)(uint32_t)ic.group * h_group_bytes : group_base(p, ic.group, q);
    const uint32_t tail_bytes = h_tail_cells * kSrcCell;

    // The issue side's walk.  A stretch is a row group's columns inside one panel; its units are consecutive in memory.
    // `next` is the next unit's first byte, `left` the units left in the stretch; next() hands out the unit's source and
    // size and steps on.  At the end of a stretch the same columns of the next row group follow, group_bytes further on,
    // as long as that row group belongs to the same matrix and panel (`spans` counts those stretches down); at the end of
    // a span the next matrix's first row group follows, or the next panel's first stretch.
    struct Walk {
        const uint8_t *next;
        int left, done;
        int first, width;     // the current panel's first unit column, and the units of a stretch in it
        int spans;            // stretches the short step still reaches, this one included
        int span_end;         // first row group past the span
        int q;                // the span's matrix
        int turn_at;          // 1 while the stretch ends with the leftover blocks (a unit of another size), else 0
        uint32_t bytes;       // size of the next unit
    };
    const int n_tiles_total = h_tiles;
    Walk iw;
    iw.next = isrc + (size_t)ic.col * kSrcTile;      // the leftover blocks follow the last tile
    iw.left = ic.end - ic.col;
    iw.done = 0;
    iw.first = ic.panel * h_panel;
    iw.width = ic.end - iw.first;
    iw.q = q;
    iw.span_end = (h_nprob == 1 || q + 1 == h_nprob) ? h_groups : p.prob[q + 1].group_begin;
    iw.spans = iw.span_end - ic.group;
    iw.turn_at = (h_tail_cells != 0 && ic.end == h_units) ? 1 : 0;
    iw.bytes = ic.col < n_tiles_total ? (uint32_t)kSrcTile : tail_bytes;
    auto walk_next = [&](Walk &w, const uint8_t *&src, uint32_t &bytes) {
        src = w.next;
        bytes = w.bytes;
        w.done++;
        w.next += kSrcTile;
        if (--w.left <= w.turn_at && w.done < n_units) {     // once a stretch (twice where it ends with the leftover unit)
            if (w.left == 0) {
                if (--w.spans > 0) {
                    // from the end of this stretch (counted in whole tiles) to the same columns of the next row group:
                    // negative where a row group is shorter than its units counted as whole tiles
                    w.next += (long long)h_group_bytes - (long long)w.width * kSrcTile;
                } else {
                    int g = w.span_end;
                    if (g == h_groups) {               // the panel is done: the next one's first stretch
                        g = 0;
                        w.q = -1;
                        w.first += h_panel;
                        w.width = min(h_panel, h_units - w.first);
                        w.turn_at = (h_tail_cells != 0 && w.first + w.width == h_units) ? 1 : 0;
                    }
                    const uint8_t *base = h_layout0;
                    w.span_end = h_groups;
                    if (h_nprob != 1) {                // the next matrix (they follow each other in the order of row groups)
                        w.q++;
                        base = p.prob[w.q].layout - (size_t)(uint32_t)p.prob[w.q].group_begin * h_group_bytes;
                        if (w.q + 1 < h_nprob) w.span_end = p.prob[w.q + 1].group_begin;
                    }
                    w.spans = w.span_end - g;
                    w.next = base + (size_t)(uint32_t)g * h_group_bytes + (size_t)w.first * kSrcTile;
                }
                w.left = w.width;
                w.bytes = (w.turn_at && w.left == 1) ? tail_bytes : (uint32_t)kSrcTile;
            } else {
                w.bytes = tail_bytes;                  // one unit left, and it is the leftover one
            }
        }
    };
    // issue the copy of the next unit onto barrier `b` and buffer `dst`: by one elected lane under a condition that
    // is the same for the whole warp, or (the four-vector build, where that form costs a register too many) by
    // lane 0 under its own predicate
    const int my_issues = lane == 0 ? n_units : 0;
    auto issue = [&](uint32_t b, uint32_t dst) {
        const int done = iw.done;
        const uint8_t *src;
        uint32_t bytes;
        walk_next(iw, src, bytes);
        if constexpr (BATCH >= 4) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.lt.s32 p, %0, %1;\n\t"
                "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%2], %3;\n\t"
                "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%4], [%5], %3, [%2];\n\t}"
                ::"r"(done), "r"(my_issues), "r"(b), "r"(bytes), "r"(dst), "l"(src));
        } else if (done < n_units) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "elect.sync _|p, 0xffffffff;\n\t"
                "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t"
                "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%2], [%3], %1, [%0];\n\t}"
                ::"r"(b), "r"(bytes), "r"(dst), "l"(src));
        }
        // No "memory" clobber: the only memory the copy writes is the slot, whose last reads feed
        // `dst` through settled() and whose next reads follow the next wait on `b`; a clobber here
        // would pin every shared-memory read of the decode behind the copy.
    };

    // Loads of the caller's constants and of the library's tables go out now and are used after the wait: this
    // thread's class constants {1 / (4 sqrt m), parity - 16} (class = thread index), this lane's operand offsets,
    // the first run's row scale, the rotation's sign flips; and x on its way into L2 with its translation into
    // this multiprocessor's TLB (its values are read only after the wait, through L2, which is where the previous
    // kernel's writes to x land).
    static_assert(kThreads == 512, "one thread a class slot");
    float2 my_class = make_float2(0.f, 0.f);
    if (!COMPACT) asm volatile("ld.global.nc.v2.f32 {%0, %1}, [%2];" : "=f"(my_class.x), "=f"(my_class.y) : "l"(h_cls_block + tid));
    uint4 lane_consts;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(lane_consts.x), "=r"(lane_consts.y), "=r"(lane_consts.z), "=r"(lane_consts.w) : "l"(h_lane_table + lane));
    const int my_row = (lane >> 2) + 8 * (lane & 3);       // the row of the group this lane ends up with
    uint16_t first_scale_bits = 0;
    if (n_units > 0) {
        const GemvProblemDev &p0 = p.prob[q];
        const int row0 = (cc.group - p0.group_begin) * kRowsPerGroup + my_row;
        if (row0 < p0.rows) asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(first_scale_bits) : "l"(p0.row_scale + row0));
    }
    // 10-byte layout: a slot a row for the products of exception blocks (this warp's 32, where a rotation would keep its sums)
    unsigned long long *exc_scratch = reinterpret_cast<unsigned long long *>(rot) + warp * 32;
    if constexpr (OVERLAY) {
        exc_scratch[lane] = 0ull;
        __syncwarp();
    }
    // 10-byte layout: the first run's range of the exception table (the caller's constants, like the records)
    uint32_t exc_first0 = 0, exc_first1 = 0;
    if constexpr (OVERLAY) {
        if (n_units > 0) {
            // the tiles [col, col + run) of the run's row group: index entries col and col + run of that row group
            const GemvProblemDev &p0 = p.prob[q];
            const int run0 = min(cc.end - cc.col, n_units);
            const uint32_t *ix = p0.exc_index + (size_t)(cc.group - p0.group_begin) * h_tiles;
            asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(exc_first0) : "l"(ix + min(cc.col, h_tiles)));
            asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(exc_first1) : "l"(ix + min(cc.col + run0, h_tiles)));
        }
    }
    uint32_t warm = 0;
    for (int e = tid * 128; e < p.nb * 48 * p.batch; e += kThreads * 128) {
        // a load whose value is not used: the register stays claimed until after the wait (settled() below), so
        // nothing stalls on the load's return before then
        uint32_t w;
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(w) : "l"(reinterpret_cast<const char *>(p.x) + e));
        warm |= w;
    }
    // ROTATE: the coordinates [c_lo, c_hi) this CTA rotates are the whole rotation blocks that meet its blocks of x
    int c_lo = 0, c_hi = 0;
    if (ROTATE) {
        const int mask = (1 << p.rot_log2) - 1;
        c_lo = min(p.rot_n, (24 * blk_lo) & ~mask);
        c_hi = min(p.rot_n, (24 * blk_hi + mask) & ~mask);
        if (p.rot_negate)       // the sign flips are the caller's constants: on their way before the wait
            for (int w = (c_lo >> 5) + tid; w < ((c_hi + 31) >> 5); w += kThreads) warm |= __ldg(p.rot_negate + w);
    }
    if (!NO_WEIGHTS) {
#pragma unroll
        for (int s = 0; s < kEarlySlots; s++) issue(my_bar + 8 * s, my_ring + s * kTileBytes);
    }
    const uint32_t lane16 = 16 * lane, lane4 = 4 * lane, pair16 = 16 * (lane >> 1);
    const int tiles = p.tiles;
    const bool odd_lane = lane & 1, high_lane = lane & 2;
    const float limb_scale = odd_lane ? 65536.f : 1.f;     // this lane's limb pair: 256^0,1 or 256^2,3
    const uint32_t tab0 = smem_addr(tab);
    // the block constants of every matrix of the launch: (class | gain << 9) -> {gain / (4 sqrt m), parity - 16}
    // (13-byte layout: the header byte is shell | parity << 4 | gain << 5 - 64 entries a matrix)
    auto build_tables = [&]() {
        if (COMPACT) {
            // 10-byte layout: 256 entries for the short records' header bytes ((f ^ shell) | shell << 4, f = window base - 3 |
            // parity << 2 | gain << 3; the base shifts the codes: x = 2 (v + base - 8) + parity), then the 64 of the four-bit records
            constexpr int kEntries = OVERLAY ? 320 : 64;
            for (int e = tid; e < p.nprob * kEntries; e += kThreads) {
                const int m = e / kEntries, h = e - m * kEntries;
                const bool window = OVERLAY && h < 256;
                const uint32_t shell = window ? h >> 4 : h & 15;
                const int f = (h ^ (h >> 4)) & 15;
                const int parity = window ? (f >> 2) & 1 : (h >> 4) & 1, gain = window ? (f >> 3) & 1 : (h >> 5) & 1;
                const int base = window ? 2 * (3 + (f & 3)) : 0;
                const GemvProblemDev &pe = p.prob[m];
                tab[m * 1024 + h] = make_float2(p.shell_inv_norm[shell] * (gain ? pe.gain1 : pe.gain0), __int_as_float(shell ? parity - 16 + base : 0));
            }
        } else {
            for (int m = 0; m < p.nprob; m++) {
                tab[m * 1024 + tid] = make_float2(my_class.x * p.prob[m].gain0, my_class.y);
                tab[m * 1024 + 512 + tid] = make_float2(my_class.x * p.prob[m].gain1, my_class.y);
            }
        }
    };
    // let the next kernel in the stream start its own prefetch, then wait for the previous one:
    // x, y and the reduction scratch may still be in use by it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // One pass over x finds the largest |x| (fp16 bit patterns of non-negative values order like integers):
    // every |x| is below 2^xexp, xexp = e - 14 with e the biased exponent of the largest magnitude.  The
    // pieces of x this CTA needs stay in registers meanwhile and then become fixed-point records on the scale
    // 2^(29 - xexp).
    bool failed = false;
    int xexp[BATCH];
    if constexpr (ROTATE) {
        // The rotated vector's largest magnitude is not known before it is rotated, but every rotated coordinate is
        // a unit-norm combination of its block, so |x'_k| <= ||x||_2: the scan sums the squares instead of taking
        // the maximum, and the fixed-point scale follows from that bound (a few bits coarser than the maximum
        // would give, of 29).  In the same pass the pieces of this CTA's rotation blocks become integers, take
        // their first three stages in registers and go to shared memory; the later stages follow there; the
        // rounded FP16 values - bit for bit those of the rotation kernel - become the fixed-point records.
        const int nx = p.nb * 3, e_lo = 3 * blk_lo, e_hi = 3 * blk_hi;
        const bool one_each = e_hi - e_lo <= kThreads;
        const uint4 *xg = reinterpret_cast<const uint4 *>(p.x);
        uint4 mine = make_uint4(0u, 0u, 0u, 0u);               // a piece of this CTA's share past the rotated length
        int mine_e = -1;
        float ss = __uint_as_float(settled(warm, warm, warm));
        for (int base = 0; base < nx; base += 4 * kThreads) {
            uint4 v[4];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int e = base + i * kThreads + tid;
                v[i] = e < nx ? __ldcg(xg + e) : make_uint4(0u, 0u, 0u, 0u);
            }
            if (base == 0) {
                for (int b = tid; b < blk_hi - blk_lo; b += kThreads)
                    asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(smem_addr(xrec) + b * kXRecBytes + 96), "r"(0) : "memory");
                build_tables();
            }
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int e = base + i * kThreads + tid;
                const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[k]));
                    ss = fmaf(f.x, f.x, ss);
                    ss = fmaf(f.y, f.y, ss);
                }
                if (8 * e >= c_lo && 8 * e < c_hi) {
                    long long a[8];
                    const uint32_t flips = p.rot_negate ? (__ldg(p.rot_negate + (e >> 2)) >> (8 * (e & 3))) & 0xffu : 0u;
                    rot_load8(v[i], flips, a);
                    rot_butterflies<3>(a);
                    rot_store8(rot, 8 * e - c_lo, a);
                } else if (e >= e_lo && e < e_hi) {
                    mine = v[i];
                    mine_e = e;
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if (lane == 0) warp_max[warp] = __float_as_uint(ss);
        __syncthreads();                               // publishes the sums of squares, the first stages, the block constants
        rot_later_passes(rot, p.rot_log2, c_hi - c_lo, tid, kThreads);
        {
            // every thread of every CTA adds the sixteen sums in the same order
            float total = __uint_as_float(warp_max[lane & (kWarps - 1)]);
#pragma unroll
            for (int off = kWarps / 2; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
            // total * 1.0625 covers the rounding of the sum and of the FP16 results: it is below 2^e2, so
            // every |x'| is below 2^ceil(e2 / 2)
            const int e2 = (int)((__float_as_uint(total * 1.0625f) >> 23) & 255u) - 126;
            xexp[0] = max((e2 + 1) >> 1, -13);
        }
        const float scale = pow2f(29 - xexp[0]);
        // rotated pieces: from the exact sums; pieces past the rotated length: as they are (the one this thread
        // met in the scan, or read again when the share is too wide for that)
        for (int e = e_lo + tid; e < e_hi; e += kThreads) {
            if (8 * e < c_hi) convert_item(rot_round8(rot, 8 * e - c_lo, p.rot_scale), e % 3, xs0 + (uint32_t)(e / 3) * kXRecBytes, scale);
            else if (!one_each) convert_item(__ldcg(xg + e), e % 3, xs0 + (uint32_t)(e / 3) * kXRecBytes, scale);
        }
        if (one_each && mine_e >= 0) convert_item(mine, mine_e % 3, xs0 + (uint32_t)(mine_e / 3) * kXRecBytes, scale);
        if (!NO_WEIGHTS) {
#pragma unroll
            for (int s = kEarlySlots; s < kSlots; s++) issue(my_bar + 8 * s, my_ring + s * kTileBytes);
        }
        __syncthreads();                               // publishes the x records
    } else {
        const int nx = p.nb * 3, e_lo = 3 * blk_lo, e_hi = 3 * blk_hi;
        const bool one_each = e_hi - e_lo <= kThreads;         // then no thread meets two of the pieces wanted
        uint4 mine[BATCH];
        int mine_e = -1;
#pragma unroll
        for (int j = 0; j < BATCH; j++) {
            uint32_t m = j == 0 ? settled(warm, warm, warm) : 0u;
            const uint4 *xg = reinterpret_cast<const uint4 *>(p.x) + (size_t)j * nx;
            mine[j] = make_uint4(0u, 0u, 0u, 0u);
            for (int base = 0; base < nx; base += 4 * kThreads) {
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const int e = base + i * kThreads + tid;
                    v[i] = (e < nx && j < p.batch) ? __ldcg(xg + e) : make_uint4(0u, 0u, 0u, 0u);
                }
                if (j == 0 && base == 0) {
                    // while the first loads are on their way: what the loop needs besides x.
                    // The zero word and the two sums of every x record this CTA will fill
                    for (int b = tid; b < BATCH * (blk_hi - blk_lo); b += kThreads) {
                        const int jj = BATCH == 1 ? 0 : b / (blk_hi - blk_lo), bb = b - jj * (blk_hi - blk_lo);
                        asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(smem_addr(xrec) + jj * xrec_stride + bb * kXRecBytes + 96), "r"(0) : "memory");
                    }
                    build_tables();
                }
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const int e = base + i * kThreads + tid;
                    m = max_abs_pair(max_abs_pair(max_abs_pair(max_abs_pair(m, v[i].x), v[i].y), v[i].z), v[i].w);
                    if (e >= e_lo && e < e_hi) { mine[j] = v[i]; mine_e = e; }
                }
            }
            m = __reduce_max_sync(0xffffffffu, max(m & 0xffffu, m >> 16));
            if (lane == 0) warp_max[j * kWarps + warp] = m;    // plain stores: atomics on one word would serialise the warps
        }
        __syncthreads();                               // publishes the maxima, the block constants and the zeroed sums
        // the second copy of records goes out now that the loads of x have returned: ahead of the conversion, whose
        // arithmetic hides its issue
        if (!NO_WEIGHTS) {
#pragma unroll
            for (int s = kEarlySlots; s < kSlots; s++) issue(my_bar + 8 * s, my_ring + s * kTileBytes);
        }
#pragma unroll
        for (int j = 0; j < BATCH; j++) {
            const uint32_t m = warp_max[j * kWarps + (lane < kWarps ? lane : 0)];
            xexp[j] = max((int)(__reduce_max_sync(0xffffffffu, m) >> 10), 1) - 14;
            const float scale = pow2f(29 - xexp[j]);
            const uint4 *xg = reinterpret_cast<const uint4 *>(p.x) + (size_t)j * nx;
            const uint32_t xsj = xs0 + j * xrec_stride;
            if (one_each) {
                if (mine_e >= 0) convert_item(mine[j], mine_e % 3, xsj + (uint32_t)(mine_e / 3) * kXRecBytes, scale);
            } else {
                for (int e = e_lo + tid; e < e_hi; e += kThreads)
                    convert_item(j < p.batch ? __ldcg(xg + e) : make_uint4(0u, 0u, 0u, 0u), e % 3, xsj + (uint32_t)(e / 3) * kXRecBytes, scale);
            }
        }
        __syncthreads();                               // publishes the x records
    }
    const LaneOffsets lo = {lane_consts.x, lane_consts.y, lane_consts.z, lane_consts.w};
    float first_row_scale;
    asm volatile("cvt.f32.f16 %0, %1;" : "=f"(first_row_scale) : "h"(first_scale_bits));

    int n = 0;
    uint32_t parity = 0;                               // every slot completes once a round of kSlots units
    uint32_t bar = my_bar;                             // barrier and buffer of the slot that is consumed next
    uint32_t sbuf = my_ring;
    const uint32_t sbuf_end = my_ring + kSlots * kTileBytes;

    // Sums the quad's shares: acc[r] of lane 4g+t is the share of row g + 8r; afterwards lane 4g+t
    // holds the whole sum of row g + 8t.  Fixed order, so the result does not depend on the launch.
    auto quad_sum = [&](const float (&acc)[4]) -> float {
        const float send0 = high_lane ? acc[0] : acc[2], send1 = high_lane ? acc[1] : acc[3];
        const float keep0 = high_lane ? acc[2] : acc[0], keep1 = high_lane ? acc[3] : acc[1];
        const float r0 = (keep0 + __shfl_xor_sync(0xffffffffu, send0, 2)) * limb_scale;
        const float r1 = (keep1 + __shfl_xor_sync(0xffffffffu, send1, 2)) * limb_scale;
        return (odd_lane ? r1 : r0) + __shfl_xor_sync(0xffffffffu, odd_lane ? r0 : r1, 1);
    };

    Handed handed;                                      // BATCH == 1: the hand-over waits for its answer a run later
    handed.slot = nullptr;
    // A run is the stretch of units of one row group inside this warp's range: its units are summed
    // in a register and handed over together.
    while (n < n_units) {
        const GemvProblemDev &pr = p.prob[q];
        // quantum of a row accumulator: 2^(xexp + qexp_base) in units of y / row_scale, xexp that of the vector;
        // a lane's sums are in units of 2^(xexp - 29)
        const float inv_q = pow2f(-29 - pr.qexp_base);
        const uint32_t tq = tab0 + q * 8192;
        const uint32_t tq_tail = OVERLAY ? tq + 2048 : tq;          // the table the four-bit records' header bytes index
        const int run = min(cc.end - cc.col, n_units - n);
        // 10-byte layout: the run's range [exc_begin, exc_end) of the exception table (the index has an entry a tile, and
        // the table follows the order of the tiles).  The first run's was loaded at the start of the CTA, a later run's
        // is read here; this lane's entry of the range goes out now, to be used when the run's tiles are summed.
        uint32_t exc_begin = exc_first0, exc_end = exc_first1;
        uint4 exc_entry = make_uint4(~0u, 0u, 0u, 0u);          // a block column no run contains
        if constexpr (OVERLAY) {
            if (n != 0) {
                const uint32_t *ix = pr.exc_index + (size_t)(cc.group - pr.group_begin) * tiles;
                asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(exc_begin) : "l"(ix + min(cc.col, tiles)));
                asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(exc_end) : "l"(ix + min(cc.col + run, tiles)));
            }
            // a run of `run` tiles holds at most 128 * run blocks: whatever the index says, the loop over the range ends
            exc_end = exc_begin + min(exc_end - exc_begin, (uint32_t)run * 128u);
            if (lane < exc_end - exc_begin) exc_entry = __ldg(pr.exc_table + exc_begin + lane);
        }
        const int run_tiles = NO_WEIGHTS ? 0 : max(0, min(run, tiles - cc.col));
        // the row's scale is needed only by the arrival that finishes the row, but loading it now
        // keeps a cold read off the tail of the kernel
        const int row = (cc.group - pr.group_begin) * kRowsPerGroup + my_row;
        const float row_scale = n == 0 ? first_row_scale : (row < pr.rows ? __half2float(pr.row_scale[row]) : 0.f);
        // this lane's addresses in the x records of the run's first tile
        const uint32_t xk = xs0 + (uint32_t)cc.col * (4 * kXRecBytes);
        LaneOffsets xa = {xk + lo.b0, xk + lo.b1, xk + lo.b2, xk + lo.xs};
        long long sum[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; j++) sum[j] = 0;

#pragma unroll 1
        for (int t = 0; t < run_tiles; t++) {
            if (!mbar_try(bar, parity)) {
                if (!mbar_wait(bar, parity)) { failed = true; break; }
            }
            // 10-byte layout: nine words a lane (two 128-bit reads and one word) and the eight header bytes of its pair
            const uint4 a0 = lds128(sbuf + lane16);
            const uint4 a1 = lds128(sbuf + lane16 + 512);
            const uint4 a2 = OVERLAY ? make_uint4(lds32(sbuf + lane4 + 1024), 0u, 0u, 0u) : lds128(sbuf + lane16 + 1024);
            // headers: four words a lane pair (14-byte layout) or two (one byte a header: hh.x serves half-steps 0, 1, hh.y 2, 3)
            uint4 hh;
            if (COMPACT) { const uint2 h2 = lds64(sbuf + (pair16 >> 1) + (OVERLAY ? 1152 : 1536)); hh = make_uint4(h2.x, h2.y, h2.y, h2.x); }
            else hh = lds128(sbuf + pair16 + 1536);
            // The slot's words are in registers: refill it at once with the unit kSlots ahead, so
            // that every slot but the one just read is in flight while this unit is decoded.  The
            // copy's address is made to depend on the loaded words, which holds the copy back
            // until the four shared-memory reads of the whole warp have completed.
            issue(bar, sbuf + (settled(a0.w, a1.w, OVERLAY ? a2.x : a2.w) | settled(hh.w, hh.x, a0.x)));
            float acc[BATCH][4];
            if constexpr (BATCH == 1) {
                // one vector: every shared-memory load first, then the eight contractions back to back (four independent
                // accumulator tiles in the tensor pipe at once), then the eight scale steps
                const StepX s1 = load_step<0>(xa), s2 = load_step<2 * kXRecBytes>(xa);
                HalfA h0, h1, h2, h3;
                if constexpr (OVERLAY) {
                    decode_overlay_tile(a0, a1, a2.x, make_uint2(hh.x, hh.y), tq, h0, h1, h2, h3);
                } else {
                    h0 = decode_half<COMPACT, 0>(a0.x, a0.y, a0.z, hh.x, tq);
                    h1 = decode_half<COMPACT, 16>(a0.w, a1.x, a1.y, COMPACT ? hh.x : hh.y, tq);
                    h2 = decode_half<COMPACT, 0>(a1.z, a1.w, a2.x, COMPACT ? hh.y : hh.z, tq);
                    h3 = decode_half<COMPACT, 16>(a2.y, a2.z, a2.w, COMPACT ? hh.y : hh.w, tq);
                }
                int d0[4], d1[4], d2[4], d3[4];
                mma_k32(d0, h0.a0, h0.a1, h0.a2, h0.a3, s1.b0, s1.b1);
                mma_k32(d1, h1.a0, h1.a1, h1.a2, h1.a3, s1.b0, s1.b1);
                mma_k32(d2, h2.a0, h2.a1, h2.a2, h2.a3, s2.b0, s2.b1);
                mma_k32(d3, h3.a0, h3.a1, h3.a2, h3.a3, s2.b0, s2.b1);
                mma_k16(d0, h0.c0, h0.c1, s1.b2);
                mma_k16(d1, h1.c0, h1.c1, s1.b2);
                mma_k16(d2, h2.c0, h2.c1, s2.b2);
                mma_k16(d3, h3.c0, h3.c1, s2.b2);
                auto e = [](const int (&d)[4], float ky, int xsum, int r) { return __float_as_int(ky) * xsum + (d[2 * r] + 256 * d[2 * r + 1]); };
                acc[0][0] = (float)e(d0, h0.k0.y, s1.xsum, 0) * h0.k0.x;
                acc[0][1] = (float)e(d0, h0.k1.y, s1.xsum, 1) * h0.k1.x;
                acc[0][2] = (float)e(d1, h1.k0.y, s1.xsum, 0) * h1.k0.x;
                acc[0][3] = (float)e(d1, h1.k1.y, s1.xsum, 1) * h1.k1.x;
                acc[0][0] = fmaf((float)e(d2, h2.k0.y, s2.xsum, 0), h2.k0.x, acc[0][0]);
                acc[0][1] = fmaf((float)e(d2, h2.k1.y, s2.xsum, 1), h2.k1.x, acc[0][1]);
                acc[0][2] = fmaf((float)e(d3, h3.k0.y, s2.xsum, 0), h3.k0.x, acc[0][2]);
                acc[0][3] = fmaf((float)e(d3, h3.k1.y, s2.xsum, 1), h3.k1.x, acc[0][3]);
            } else {
                StepX sx[BATCH];
#pragma unroll
                for (int j = 0; j < BATCH; j++) {
                    const LaneOffsets xj = {xa.b0 + j * xrec_stride, xa.b1 + j * xrec_stride, xa.b2 + j * xrec_stride, xa.xs + j * xrec_stride};
                    sx[j] = load_step<0>(xj);
                }
                const HalfA h0 = decode_half<COMPACT, 0>(a0.x, a0.y, a0.z, hh.x, tq);
#pragma unroll
                for (int j = 0; j < BATCH; j++) contract_half<true>(h0, sx[j], acc[j][0], acc[j][1]);
                const HalfA h1 = decode_half<COMPACT, 16>(a0.w, a1.x, a1.y, COMPACT ? hh.x : hh.y, tq);
#pragma unroll
                for (int j = 0; j < BATCH; j++) contract_half<true>(h1, sx[j], acc[j][2], acc[j][3]);
#pragma unroll
                for (int j = 0; j < BATCH; j++) {
                    const LaneOffsets xj = {xa.b0 + j * xrec_stride, xa.b1 + j * xrec_stride, xa.b2 + j * xrec_stride, xa.xs + j * xrec_stride};
                    sx[j] = load_step<2 * kXRecBytes>(xj);
                }
                const HalfA h2 = decode_half<COMPACT, 0>(a1.z, a1.w, a2.x, COMPACT ? hh.y : hh.z, tq);
#pragma unroll
                for (int j = 0; j < BATCH; j++) contract_half<false>(h2, sx[j], acc[j][0], acc[j][1]);
                const HalfA h3 = decode_half<COMPACT, 16>(a2.y, a2.z, a2.w, COMPACT ? hh.y : hh.w, tq);
#pragma unroll
                for (int j = 0; j < BATCH; j++) contract_half<false>(h3, sx[j], acc[j][2], acc[j][3]);
            }
#pragma unroll
            for (int j = 0; j < BATCH; j++) sum[j] += __float2ll_rn(quad_sum(acc[j]) * inv_q);
            xa.b0 += 4 * kXRecBytes; xa.b1 += 4 * kXRecBytes; xa.b2 += 4 * kXRecBytes; xa.xs += 4 * kXRecBytes;
            bar += 8;
            sbuf += kTileBytes;
            const bool wrap = sbuf == sbuf_end;        // every slot completes once a round
            sbuf = wrap ? my_ring : sbuf;
            bar = wrap ? my_bar : bar;
            parity ^= wrap ? 1u : 0u;
        }
        if (failed) break;
        if (!NO_WEIGHTS && run_tiles < run) {
            // the run ends with the nb mod 4 last block columns of the row group: a pair, a single, or both
            if (!mbar_wait(bar, parity)) { failed = true; break; }
            uint32_t guard = 0, piece = sbuf;
            float acc[BATCH][4];
#pragma unroll
            for (int j = 0; j < BATCH; j++) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
            const uint32_t xt = xs0 + (uint32_t)tiles * (4 * kXRecBytes);
            if (p.tail_cells >= 2) {
#pragma unroll
                for (int m = 0; m < 2; m++) {
                    const uint32_t wa = lds32(piece + 128 * (3 * m) + lane4), wb = lds32(piece + 128 * (3 * m + 1) + lane4);
                    const uint32_t wc = lds32(piece + 128 * (3 * m + 2) + lane4);
                    const uint32_t hw = COMPACT ? lds32(piece + 768 + 4 * (lane >> 1)) : lds32(piece + 768 + 8 * (lane >> 1) + 4 * m);
                    guard |= settled(wa, wb, wc) | settled(hw, wa, wb);
                    const HalfA h = m == 0 ? decode_half<COMPACT, 0>(wa, wb, wc, hw, tq_tail) : decode_half<COMPACT, 16>(wa, wb, wc, hw, tq_tail);
#pragma unroll
                    for (int j = 0; j < BATCH; j++) {
                        const uint32_t xj = xt + j * xrec_stride;
                        const LaneOffsets ta = {xj + lo.b0, xj + lo.b1, xj + lo.b2, xj + lo.xs};
                        contract_half<false>(h, load_step<0>(ta), acc[j][2 * m], acc[j][2 * m + 1]);
                    }
                }
                piece += 2 * kSrcCell;
            }
            if (p.tail_cells & 1) {
                // one block: the slots of this half-step are the two halves of the row group
                const uint32_t xl = xs0 + (uint32_t)(p.nb - 1) * kXRecBytes;
                const LaneOffsets l1 = lane_offsets(lane, true);
                const uint32_t wa = lds32(piece + lane4), wb = lds32(piece + 128 + lane4);
                const uint32_t wc = lds32(piece + 256 + lane4);
                // 13-byte layout: two bytes a lane pair, the pairs two to a word
                const uint32_t hw = COMPACT ? lds32(piece + 384 + 4 * (lane >> 2)) >> (8 * (lane & 2)) : lds32(piece + 384 + 4 * (lane >> 1));
                guard |= settled(wa, wb, wc) | settled(hw, wa, wb);
                const HalfA h = decode_half<COMPACT, 0>(wa, wb, wc, hw, tq_tail);
#pragma unroll
                for (int j = 0; j < BATCH; j++) {
                    const uint32_t xj = xl + j * xrec_stride;
                    const LaneOffsets ta = {xj + l1.b0, xj + l1.b1, xj + l1.b2, xj + l1.xs};
                    float c0, c1;
                    contract_half<true>(h, load_step<0>(ta), c0, c1);
                    acc[j][0] += high_lane ? 0.f : c0; acc[j][1] += high_lane ? 0.f : c1;
                    acc[j][2] += high_lane ? c0 : 0.f; acc[j][3] += high_lane ? c1 : 0.f;
                }
            }
            issue(bar, sbuf + guard);
#pragma unroll
            for (int j = 0; j < BATCH; j++) sum[j] += __float2ll_rn(quad_sum(acc[j]) * inv_q);
            bar += 8;
            sbuf += kTileBytes;
            if (sbuf == sbuf_end) { sbuf = my_ring; bar = my_bar; parity ^= 1u; }
        }
        if constexpr (OVERLAY) {
            // The exact records of this run's exception blocks: every lane takes an entry of the run's range and adds
            // the product to its row's slot of the warp's scratch (integer additions, so the order does not matter);
            // then every lane collects its own row's slot.
            const uint32_t exc_count = exc_end - exc_begin;          // at most 2048 (bounded where the range was read)
            const bool any = exc_count != 0;
#pragma unroll 1
            for (uint32_t done = 0; done < exc_count; done += 32) {
                if (done != 0) exc_entry = done + lane < exc_count ? __ldg(pr.exc_table + exc_begin + done + lane) : make_uint4(~0u, 0u, 0u, 0u);
                if (exc_entry.x != ~0u) {
                    const long long v = exception_value(exc_entry, xs0 + (exc_entry.x >> 13) * kXRecBytes, tq_tail, inv_q);
                    // in two 32-bit halves, v = hi * 2^24 + lo with lo in [0, 2^24): a row meets at most 64 entries
                    // a run and |v| < 2^40, so neither half overflows its word
                    uint32_t *half = reinterpret_cast<uint32_t *>(exc_scratch + ((exc_entry.x >> 8) & 31u));
                    atomicAdd(half, (uint32_t)(v & 0xffffff));
                    atomicAdd(reinterpret_cast<int *>(half + 1), (int)(v >> 24));
                }
            }
            if (any) {
                __syncwarp();
                const uint2 halves = *reinterpret_cast<const uint2 *>(exc_scratch + my_row);
                sum[0] += ((long long)(int)halves.y << 24) + (long long)halves.x;
                __syncwarp();
                exc_scratch[my_row] = 0ull;
                __syncwarp();                          // the slots are clear before any lane adds to them again
            }
        }
        // with no records read (the control launch) every unit contributes zero
        n += run;
        if (BATCH == 1) {
            hand_over(p, pr, p.accum, pr.y, cc.group, my_row, sum[0], run, xexp[0] + pr.qexp_base, row_scale, handed);
        } else {
            // one hand-over a vector; each waits for its answer (a batched launch has arithmetic to hide behind)
#pragma unroll
            for (int j = 0; j < BATCH; j++) {
                if (j >= p.batch) break;               // a launch may carry fewer vectors than the kernel is built for
                Handed hj;
                hj.slot = nullptr;
                hand_over(p, pr, p.accum + (size_t)j * p.total_groups * 32, pr.y + (size_t)j * p.y_stride, cc.group, my_row, sum[j], run,
                          xexp[j] + pr.qexp_base, row_scale, hj);
                settle(p, hj);
            }
        }
        if (advance(p, cc, run) && cc.panel < p.npanels) q = find_problem(p, cc.group);
    }
    settle(p, handed);

    if (failed) {
        // a wait ran out: report it, then give the copies still in flight a bounded chance to land
        // (a slot that is not pending returns at once or runs into the same bound)
        if (lane == 0) atomicExch(p.error, 1);
        for (int s = 0; s < kSlots && s < min(iw.done, n_units); s++) mbar_wait(my_bar + 8 * s, parity);
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
    const uint8_t *grp = n_units > 0 ? group_base(p, group, q) : nullptr;
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
                if (group < p.total_groups) grp = group_base(p, group, q);
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

// ---- helpers reading a record back: thread = (row group, block column, row of the group)
// The 24 codes (c[j] = codes of coordinates 8j..8j+7, a nibble each) and the header of one block of one row,
// found from the layout's description in include/llvq.h: which piece, half-step, lane, word and nibble.
// kTile: bytes of a tile in this buffer (the 10-byte layout's leftover blocks are read with COMPACT and its own tile size)
template <bool COMPACT, int kTile = COMPACT ? kTile13Bytes : kTileBytes>
__device__ __forceinline__ void read_planes_record(const uint8_t *buf, int64_t nb, int64_t rg, int64_t b, int r,
                                                   uint32_t c[3], uint32_t &hdr) {
    const int64_t tiles = nb / kTileCells, left = nb % kTileCells;
    constexpr int kCell = COMPACT ? kCell13Bytes : kCellBytes;
    const uint8_t *grp = buf + (size_t)rg * ((size_t)tiles * kTile + (size_t)left * kCell);
    const int m = r >> 4, e = (r >> 3) & 1, g = r & 7;
    const int64_t j = b - tiles * kTileCells;
    const uint8_t *base;
    int slot, kind, h = 0;                         // kind 0 tile, 1 pair, 2 single
    if (j < 0) {
        base = grp + (size_t)(b / kTileCells) * kTile;
        slot = (int)(b & 1); h = 2 * (int)((b % kTileCells) >> 1) + m; kind = 0;
    } else if (left >= 2 && j < 2) {
        base = grp + (size_t)tiles * kTile; slot = (int)j; kind = 1;
    } else {
        base = grp + (size_t)tiles * kTile + (left == 3 ? 2 * kCell : 0); slot = m; kind = 2;
    }
    auto word = [&](int q, int lane) -> uint32_t {
        const int k = 3 * h + q;
        const uint8_t *a = kind == 0 ? base + 512 * (k >> 2) + 16 * lane + 4 * (k & 3)
                         : kind == 1 ? base + 128 * (3 * m + q) + 4 * lane
                                     : base + 128 * q + 4 * lane;
        return *reinterpret_cast<const uint32_t *>(a);
    };
    const int pair = 2 * g + slot;
    if (COMPACT) {
        hdr = kind == 0 ? base[1536 + 8 * pair + 2 * h + e] : kind == 1 ? base[768 + 4 * pair + 2 * m + e] : base[384 + 2 * pair + e];
    } else {
        const uint32_t hw = *reinterpret_cast<const uint32_t *>(kind == 0 ? base + 1536 + 16 * pair + 4 * h
                                                                : kind == 1 ? base + 768 + 8 * pair + 4 * m
                                                                            : base + 384 + 4 * pair);
        hdr = (hw >> (16 * e)) & 0xffffu;
    }
    c[0] = c[1] = c[2] = 0;
    for (int i = 0; i < 24; i++) {
        const int kappa = 24 * slot + i;
        uint32_t w; int nib;
        if (kappa < 32) { w = word(e, 4 * g + ((kappa & 15) >> 2)); nib = 2 * (kappa & 3) + (kappa >> 4); }
        else { w = word(2, 4 * g + ((kappa - 32) >> 2)); nib = 2 * (kappa & 3) + e; }
        c[i >> 3] |= ((w >> (4 * nib)) & 15u) << (4 * (i & 7));
    }
}

// 10-byte layout: the four-bit codes and the header byte (shell | parity << 4 | gain << 5) of one block of one row -
// from the short record (three-bit codes plus the window base), from the exception table when the short record is
// empty and the table lists the block, else the empty record.
__device__ __forceinline__ void read_overlay_record(const uint8_t *buf, int64_t rows, int64_t nb, int64_t rg, int64_t b, int r,
                                                    uint32_t c[3], uint32_t &hdr) {
    const int64_t tiles = nb / kTileCells;
    if (b >= tiles * kTileCells) {                 // a leftover block: a four-bit record
        read_planes_record<true, kTile10Bytes>(buf, nb, rg, b, r, c, hdr);
        return;
    }
    const uint8_t *tile = buf + (size_t)rg * overlay_group_bytes(nb) + (size_t)(b / kTileCells) * kTile10Bytes;
    const int m = r >> 4, e = (r >> 3) & 1, g = r & 7;
    const int slot = (int)(b & 1), h = 2 * (int)((b % kTileCells) >> 1) + m;
    auto V = [&](int k, int lane) -> uint32_t {
        return *reinterpret_cast<const uint32_t *>(tile + (k < 4 ? 16 * lane + 4 * k : (k < 8 ? 512 + 16 * lane + 4 * (k - 4) : 1024 + 4 * lane)));
    };
    const uint32_t hb = tile[1152 + 8 * (2 * g + slot) + 2 * h + e];
    if (hb == 0) {
        // empty: an exception (then the table has the block), a row past the end or a code that named no point
        const uint32_t *index = reinterpret_cast<const uint32_t *>(buf + overlay_index_offset(rows, nb));
        const uint4 *table = reinterpret_cast<const uint4 *>(buf + overlay_table_offset(rows, nb));
        hdr = 0; c[0] = c[1] = c[2] = 0x88888888u;
        const int64_t tile_id = rg * tiles + b / kTileCells;
        const uint32_t first = index[tile_id], count = min(index[tile_id + 1] - first, 128u);      // a tile has 128 blocks
        for (uint32_t i = first; i < first + count; i++) {
            const uint4 ent = table[i];
            if ((ent.x >> 13) == (uint32_t)b && ((ent.x >> 8) & 31u) == (uint32_t)r) { hdr = ent.x & 63u; c[0] = ent.y; c[1] = ent.z; c[2] = ent.w; }
        }
        return;
    }
    const uint32_t f = (hb ^ (hb >> 4)) & 15u;         // window base - 3 | parity << 2 | gain << 3
    hdr = (hb >> 4) | (f >> 2) << 4;                   // as the 13-byte layout writes it: shell | parity << 4 | gain << 5
    const uint32_t base = 3u + (f & 3u);
    c[0] = c[1] = c[2] = 0;
    for (int i = 0; i < 24; i++) {
        const int kappa = 24 * slot + i;
        uint32_t v;
        if (kappa < 32) {
            v = (V(2 * h + e, 4 * g + ((kappa & 15) >> 2)) >> (8 * (kappa & 3) + 3 * (kappa >> 4))) & 7u;
        } else {
            const int lane = 4 * g + ((kappa - 32) >> 2), sh = 8 * (kappa & 3);
            if (e == 0 && h < 2) {
                v = (V(8, lane) >> (sh + 3 * h)) & 7u;
            } else {
                const int k = h == 0 ? 0 : (h == 1 ? 1 : 2 * h - 2 + e);          // X0..X5 = (0,1) (1,1) (2,0) (2,1) (3,0) (3,1)
                v = ((V(k, lane) >> (sh + 6)) & 3u) | (((V(6 + (k >> 1), lane) >> (sh + 6 + (k & 1))) & 1u) << 2);
            }
        }
        c[i >> 3] |= (v + base) << (4 * (i & 7));
    }
}

// integer coordinates of one record, any layout
__device__ __forceinline__ void record_coords(int layout, const uint8_t *buf, int64_t rows, int64_t nb, int64_t rg, int64_t b, int lane,
                                              const uint32_t *cls_parity, const uint8_t *cls_dist, int &cls, int &gain, int x[24]) {
    if (layout == LLVQ_PLANES) {
        uint32_t c[3], hdr;
        read_planes_record<false>(buf, nb, rg, b, lane, c, hdr);
        cls = (int)(hdr & 511u); gain = (int)((hdr >> 9) & 1u);
        const int par = cls_parity[cls] ? 1 : 0;
        for (int i = 0; i < 24; i++) x[i] = 2 * ((int)((c[i >> 3] >> (4 * (i & 7))) & 15u) - 8) + par;
    } else if (layout == LLVQ_PLANES13 || layout == LLVQ_PLANES10X) {
        // no class id in these layouts: `cls` returns the header byte (shell | parity << 4 | gain << 5)
        uint32_t c[3], hdr;
        if (layout == LLVQ_PLANES13) read_planes_record<true>(buf, nb, rg, b, lane, c, hdr);
        else read_overlay_record(buf, rows, nb, rg, b, lane, c, hdr);
        cls = (int)hdr; gain = (int)((hdr >> 5) & 1u);
        const int par = (int)((hdr >> 4) & 1u);
        for (int i = 0; i < 24; i++) x[i] = 2 * ((int)((c[i >> 3] >> (4 * (i & 7))) & 15u) - 8) + par;
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
    record_coords(layout, buf, rows, nb, rg, b, lane, cls_parity, cls_dist, cls, gain, x);
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
    record_coords(layout, buf, rows, nb, rg, b, lane, cls_parity, cls_dist, cls, gain, x);
    // r * gain / (4 sqrt m): cls_scale carries 2^21 / (4 sqrt m)
    const float s = __half2float(row_scale[row]) * ((gain ? g1 : g0) * (cls_scale[cls] * (1.0f / 2097152.0f)));
    __half *dst = W + (row * nb + b) * 24;
    for (int i = 0; i < 24; i++) dst[i] = __float2half_rn(s * (float)x[i]);
}

}  // namespace

void gemv_lane_table(uint32_t (*out)[4]) {
    for (int lane = 0; lane < 32; lane++) {
        const LaneOffsets o = lane_offsets(lane, false);
        out[lane][0] = o.b0; out[lane][1] = o.b1; out[lane][2] = o.b2; out[lane][3] = o.xs;
    }
}

GemvLaunch gemv_plan(int layout, GemvParams &p, int sm_count) {
    GemvLaunch g;
    // one CTA a multiprocessor
    g.grid = p.total_units < sm_count ? p.total_units : sm_count;
    p.units_base = p.total_units / (g.grid * kWarps);
    p.units_rem = p.total_units % (g.grid * kWarps);
    p.group_bytes = layout == LLVQ_PLANES10X ? (uint32_t)overlay_group_bytes(p.nb)
                                             : (uint32_t)p.nb * (uint32_t)(layout == LLVQ_ONEHOT ? kOneHotCellBytes : (layout == LLVQ_PLANES13 ? kCell13Bytes : kCellBytes));
    if (layout == LLVQ_ONEHOT) {
        g.smem = ((size_t)p.nb * 48 + 127) / 128 * 128;
        return g;
    }
    // panels of about sixteen unit columns, as equal as they come
    constexpr int kPanelColumns = 16;
    const int want = (p.units + kPanelColumns / 2) / kPanelColumns > 1 ? (p.units + kPanelColumns / 2) / kPanelColumns : 1;
    p.panel = (p.units + want - 1) / want;
    p.npanels = (p.units + p.panel - 1) / p.panel;
    p.div_panel_units = make_fastdiv((uint32_t)(p.total_groups * p.panel));
    p.div_panel = make_fastdiv((uint32_t)p.panel);
    p.div_last = make_fastdiv((uint32_t)(p.units - (p.npanels - 1) * p.panel));
    // Shares of the CTAs.  CTAs start in index order as multiprocessors come free, the first ones while the
    // previous kernel of the stream is still finishing, so the first CTAs can afford more units than the last:
    // the share falls linearly from mean + lead to mean - lead.
    if (g.grid > kMaxGridCtas) g.grid = kMaxGridCtas;
    {
        const double mean = (double)p.total_units / g.grid;
        double lead = 10.0;                            // units: about half a microsecond of a multiprocessor's streaming (measured optimum 9-12)
        if (lead > 0.6 * mean) lead = 0.6 * mean;
        const double skew = mean > 0 ? lead / mean : 0.0;
        double acc = 0.0;
        p.cta[0].first = 0;
        for (int c = 0; c < g.grid; c++) {
            const double w = g.grid > 1 ? 1.0 + skew * (1.0 - 2.0 * c / (g.grid - 1)) : 1.0;
            acc += mean * w;
            int f = (int)(acc + 0.5);
            if (f < p.cta[c].first) f = p.cta[c].first;
            if (f > p.total_units) f = p.total_units;
            p.cta[c + 1].first = f;
        }
        p.cta[g.grid].first = p.total_units;
        p.cta[g.grid].blk_lo = p.cta[g.grid].blk_hi = p.cta[g.grid].panel = 0;
        p.cta[g.grid].panel_first = 0;
    }
    // the stretch of x a CTA meets: the whole panels its units lie in (consecutive ones)
    p.xblocks = 0;
    p.rot_span = 0;
    for (int c = 0; c < g.grid; c++) {
        const int f0 = p.cta[c].first, f1 = p.cta[c + 1].first;
        const int lo = panel_of_unit(p, f0) * p.panel * kTileCells;
        int hi = (panel_of_unit(p, f1 - 1 > f0 ? f1 - 1 : f0) + 1) * p.panel * kTileCells;
        if (hi > p.nb) hi = p.nb;
        p.cta[c].blk_lo = (uint16_t)lo;
        p.cta[c].blk_hi = (uint16_t)hi;
        p.cta[c].panel = (uint16_t)panel_of_unit(p, f0);
        p.cta[c].panel_first = p.cta[c].panel * (p.total_groups * p.panel);
        if (hi - lo > p.xblocks) p.xblocks = hi - lo;
        if (p.rot_log2 > 0) {
            // the whole rotation blocks that meet the CTA's blocks of x (the kernel computes the same)
            const int mask = (1 << p.rot_log2) - 1;
            int c_lo = (24 * lo) & ~mask, c_hi = (24 * hi + mask) & ~mask;
            if (c_lo > p.rot_n) c_lo = p.rot_n;
            if (c_hi > p.rot_n) c_hi = p.rot_n;
            if (c_hi - c_lo > p.rot_span) p.rot_span = c_hi - c_lo;
        }
    }
    const int vectors = p.batch <= 1 ? 1 : (p.batch == 2 ? 2 : 4);             // the kernel is built for 1, 2 and 4
    const size_t xbytes = ((size_t)p.xblocks * kXRecBytes + 127) / 128 * 128 * vectors;
    g.smem = (size_t)kWarps * kSlots * kTileBytes + 8192 /* alignment of the tables */ + (size_t)p.nprob * 8192 + xbytes + kWarps * kSlots * 8 + kWarps * 4 * vectors + 16 + (size_t)p.rot_span * 8;
    if (layout == LLVQ_PLANES10X) g.smem += (size_t)kWarps * 32 * 8;        // the warps' slots for the products of exception blocks
    return g;
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
    if (allow_max_smem(gemv_planes_kernel<false, 1>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<true, 1>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<false, 2>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<false, 4>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<false, 1, true>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<false, 1, false, LLVQ_PLANES13>, bytes)) return -1;
    if (allow_max_smem(gemv_planes_kernel<false, 1, false, LLVQ_PLANES10X>, bytes)) return -1;
    if (allow_max_smem(gemv_onehot_kernel, bytes)) return -1;
    return 0;
}

cudaError_t launch_gemv(int layout, const GemvParams &p, const GemvLaunch &g, bool no_weights, bool pdl, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)g.grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (layout == LLVQ_PLANES13) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 1, false, LLVQ_PLANES13>, p);
    if (layout == LLVQ_PLANES10X) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 1, false, LLVQ_PLANES10X>, p);
    if (layout == LLVQ_PLANES) {
        if (no_weights) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<true, 1>, p);
        if (p.rot_log2 > 0) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 1, true>, p);
        if (p.batch <= 1) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 1>, p);
        if (p.batch == 2) return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 2>, p);
        return cudaLaunchKernelEx(&cfg, gemv_planes_kernel<false, 4>, p);
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
// llvq_gemv_static: the 14-byte-layout GEMV for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a matvec: a serving
// process whose memory pool already owns all of HBM, a plug-in that is handed buffers but no
// allocator, code that runs while a stream is being captured (allocation is not allowed there), or
// a real-time loop in which an allocation's implicit device synchronisation is not acceptable.
// Those callers cannot create a context either, because llvq_create allocates the tables and the
// reduction scratch.  For them everything the kernel needs besides the caller's own buffers lives
// in file-scope __device__ arrays that the module carries: the row accumulators (the scratch) and
// the error flag; the class constants travel in the kernel's parameters.  Every GPU that loads the
// library holds these arrays (about 512 KiB) until the process exits.
//
// In host code the name of a __device__ array is only a host-side stand-in, not a device address;
// the kernel is therefore given the address that cudaGetSymbolAddress returns for the current
// device.  That, the zeroing of the scratch and the kernel's shared-memory attribute are done
// by the first call on each device (synchronously), so make that first call before any stream
// capture begins.  All calls share the arrays: the accumulators are left at zero by every launch
// that completes, but two launches that overlap on the GPU (different streams) race on them.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRows = 65536;      // rows (rounded up to 32) one llvq_gemv_static call may have
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) unsigned long long g_static_accum[kStaticMaxRows];   // 512 KiB of scratch
static __device__ __align__(256) int g_static_error[64];
static __device__ __align__(256) float2 g_static_cls_block[llvq::kClassSlots];   // {1 / (4 sqrt m), parity - 16} of every class slot
static __device__ __align__(256) uint4 g_static_lane_table[32];                  // a lane's operand offsets

struct StaticDevice {
    bool ready = false;
    unsigned long long *accum = nullptr;
    float2 *cls_block = nullptr;
    uint4 *lane_table = nullptr;
    uint32_t cls_shell_nibbles[64], cls_odd_bits[16];      // class constants (host copies, handed to every launch)
    float shell_inv_norm[16];
    int *error = nullptr;
    int sm_count = 0, max_smem_optin = 0;
};
StaticDevice g_static_dev[kStaticMaxDevices];
std::mutex g_static_mutex;                 // guards the first call's set-up on a device

// Once per device, with that device current: resolve the arrays' device addresses, build the class
// constants on the host, zero the accumulators, raise the kernel's shared-memory limit.  Allocates no device memory.
int static_setup(int device, StaticDevice &d) {
    if (cudaGetSymbolAddress((void **)&d.accum, g_static_accum) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaGetSymbolAddress((void **)&d.error, g_static_error) != cudaSuccess) return LLVQ_ECUDA;
    llvq::HostTables host;                                   // host memory only
    if (!llvq::build_tables(host)) return LLVQ_EINVAL;
    memcpy(d.cls_shell_nibbles, host.cls_shell_nibbles, sizeof d.cls_shell_nibbles);
    memcpy(d.cls_odd_bits, host.cls_odd_bits, sizeof d.cls_odd_bits);
    memcpy(d.shell_inv_norm, host.shell_inv_norm, sizeof d.shell_inv_norm);
    uint32_t lanes[32][4];
    llvq::gemv_lane_table(lanes);
    if (cudaGetSymbolAddress((void **)&d.cls_block, g_static_cls_block) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaGetSymbolAddress((void **)&d.lane_table, g_static_lane_table) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemcpy(d.cls_block, host.cls_block.data(), sizeof(float2) * llvq::kClassSlots, cudaMemcpyHostToDevice) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemcpy(d.lane_table, lanes, sizeof lanes, cudaMemcpyHostToDevice) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemset(d.accum, 0, sizeof(unsigned long long) * kStaticMaxRows) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemset(d.error, 0, sizeof(int) * 64) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) return LLVQ_ECUDA;
    if (llvq::allow_max_smem(llvq::gemv_planes_kernel<false, 1>, d.max_smem_optin)) return LLVQ_ECUDA;
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
    {
        // two host threads may make the first call on a device at once: one of them sets up, the other waits
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!d.ready) {
            const int rc = static_setup(device, d);
            if (rc != LLVQ_OK) return rc;
        }
    }
    GemvParams p;
    memset(&p, 0, sizeof p);
    p.nprob = 1;
    p.batch = 1;
    p.y_stride = (int)rows;
    p.prob[0].layout = (const uint8_t *)layout_buf;
    p.prob[0].row_scale = (const __half *)row_scale;
    p.prob[0].y = y;
    p.prob[0].rows = (int)rows;
    p.prob[0].group_begin = 0;
    p.prob[0].gain0 = gain[0];
    p.prob[0].gain1 = gain[1];
    {
        const float gm = fmaxf(fabsf(gain[0]), fabsf(gain[1]));
        if (!(gm == 0.f || (gm >= 8.673617379884035e-19f && gm < 1.152921504606847e18f))) return LLVQ_EINVAL;   // as llvq_gemv
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
    memcpy(p.cls_shell_nibbles, d.cls_shell_nibbles, sizeof p.cls_shell_nibbles);
    memcpy(p.cls_odd_bits, d.cls_odd_bits, sizeof p.cls_odd_bits);
    memcpy(p.shell_inv_norm, d.shell_inv_norm, sizeof p.shell_inv_norm);
    p.error = d.error;
    p.cls_block = d.cls_block;
    p.lane_table = d.lane_table;
    const llvq::GemvLaunch g = llvq::gemv_plan(LLVQ_PLANES, p, d.sm_count);
    if (g.smem + 1024 > (size_t)d.max_smem_optin) return LLVQ_ESIZE;
    return llvq::launch_gemv(LLVQ_PLANES, p, g, false, true, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}


// Reports and repairs what a llvq_gemv_static launch that gave up on a bounded wait leaves behind.  Without a
// context there is no llvq_status to do it: the flag such a launch raises and the partial sums it abandons live in
// the library's own arrays, and an unreported time-out would spoil every later call on the device.
extern "C" int llvq_static_status(void *stream) {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return LLVQ_ECUDA;
    if (device < 0 || device >= kStaticMaxDevices) return LLVQ_EINVAL;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LLVQ_ECUDA;
    StaticDevice &d = g_static_dev[device];
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!d.ready) return LLVQ_OK;                  // no call was made on this device yet
    }
    int flag = 0;
    if (cudaMemcpy(&flag, d.error, sizeof flag, cudaMemcpyDeviceToHost) != cudaSuccess) return LLVQ_ECUDA;
    if (!flag) return LLVQ_OK;
    // no allocation here either: both arrays are the library's own
    if (cudaMemset(d.error, 0, sizeof(int) * 64) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemset(d.accum, 0, sizeof(unsigned long long) * kStaticMaxRows) != cudaSuccess) return LLVQ_ECUDA;
    return LLVQ_ETIMEOUT;
}

// Points the wait-limit self-test at the static entry point's error flag, so that the path above can be exercised
// without any fault on the GPU.
extern "C" int llvq_static_selftest_wait_limit(void *stream) {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return LLVQ_ECUDA;
    if (device < 0 || device >= kStaticMaxDevices) return LLVQ_EINVAL;
    StaticDevice &d = g_static_dev[device];
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!d.ready) {
            const int rc = static_setup(device, d);
            if (rc != LLVQ_OK) return rc;
        }
    }
    llvq::wait_limit_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d.error);
    return cudaGetLastError() == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}
