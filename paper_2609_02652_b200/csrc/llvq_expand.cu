// The expander (paper Sec. 2.2, "Unfolding at load time"): one pass that turns every 48-bit code
// word into its decoded-field record - class id, gain bit, sign mask, per-coordinate level - in
// the 14-byte or the one-hot layout.  Integer arithmetic only, so the output is bit-exact.
//
// The index splits as the paper states it (Sec. 2.1: classes first, then arrangements and signs
// inside a class, as a mixed-radix number).  The digit order used here:
//   even type:  ((codeword rank * perm_a + rank_a) * perm_b + rank_b) << sign_bits | signs
//   odd type:   arrangement rank * 4096 + message bits of the codeword
// Arrangement ranks are lexicographic over the distinct orderings, smaller magnitude first; sign
// bits run over the non-zero off-support coordinates first, then the support coordinates but the
// last, whose sign restores the sum condition mod 8.
#include "llvq_internal.cuh"

namespace llvq {
namespace {

struct Unranker {
    uint64_t rank, total;
    int left;
    int cnt[7];
};

// Next value index (0..NV-1) of the lexicographically rank-th ordering.
template <int NV>
__device__ __forceinline__ int unrank_step(Unranker &u) {
    int pick = 0;
    bool done = false;
#pragma unroll
    for (int v = 0; v < NV; v++) {
        if (!done && u.cnt[v] > 0) {
            uint64_t sub = u.total * (uint64_t)u.cnt[v] / (uint64_t)u.left;   // orderings starting with v
            if (u.rank < sub) {
                pick = v; u.total = sub; u.cnt[v]--; done = true;
            } else {
                u.rank -= sub;
            }
        }
    }
    u.left--;
    return pick;
}

struct Decoded {
    int cls, gain;
    uint32_t smask;
    uint32_t mag[3];   // magnitude of coordinate i in nibble i%8 of word i/8
};

__device__ __forceinline__ void set_mag(Decoded &d, int i, int a) { d.mag[i >> 3] |= (uint32_t)a << (4 * (i & 7)); }

__device__ bool decode_code(uint64_t code, const DeviceTables &T, Decoded &d) {
    d.cls = kEmptyClass; d.gain = 0; d.smask = 0; d.mag[0] = d.mag[1] = d.mag[2] = 0;
    const uint64_t idx = code & ((1ull << kIndexBits) - 1);
    if ((code >> 48) != 0 || idx >= T.num_points) return false;
    // class: last c with base[c] <= idx
    int lo = 0, hi = T.num_classes;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(&T.base[mid]) <= idx) lo = mid; else hi = mid;
    }
    const ClassDesc c = T.desc[lo];
    uint64_t r = idx - __ldg(&T.base[lo]);
    d.cls = lo;
    d.gain = (int)((code >> kIndexBits) & 1);

    if (c.odd) {
        const uint32_t cw = __ldg(&T.golay_by_message[(uint32_t)r & 4095u]);
        Unranker u;
        u.rank = r >> 12; u.total = c.perm_a; u.left = 24;
#pragma unroll
        for (int v = 0; v < 7; v++) u.cnt[v] = c.cnt[v];
#pragma unroll
        for (int i = 0; i < 24; i++) {
            const int a = 1 + 2 * unrank_step<7>(u);
            const int want = 1 + 2 * (int)((cw >> i) & 1);     // residue of x_i mod 4
            if ((a & 3) != want) d.smask |= 1u << i;
            set_mag(d, i, a);
        }
        return true;
    }

    const uint64_t sigma = r & ((1ull << c.sign_bits) - 1);
    r >>= c.sign_bits;
    const uint64_t rank_b = r % c.perm_b; r /= c.perm_b;
    const uint64_t rank_a = r % c.perm_a; r /= c.perm_a;
    const uint32_t cw = __ldg(&T.golay_by_weight[T.weight_offset[c.w] + (int)r]);
    Unranker ua, ub;
    ua.rank = rank_a; ua.total = c.perm_a; ua.left = c.w;
    ub.rank = rank_b; ub.total = c.perm_b; ub.left = 24 - c.w;
#pragma unroll
    for (int v = 0; v < 4; v++) { ua.cnt[v] = c.cnt[v]; ub.cnt[v] = c.cnt[4 + v]; }
    int off_bit = 0, sup_seen = 0, last = -1, sum = 0;
#pragma unroll
    for (int i = 0; i < 24; i++) {
        int a; bool neg = false;
        if ((cw >> i) & 1) {
            a = 2 + 4 * unrank_step<4>(ua);
            sup_seen++;
            if (sup_seen < c.w) neg = (sigma >> (c.nz_b + sup_seen - 1)) & 1; else last = i;
        } else {
            a = 4 * unrank_step<4>(ub);
            if (a) { neg = (sigma >> off_bit) & 1; off_bit++; }
        }
        set_mag(d, i, a);
        if (neg) d.smask |= 1u << i;
        sum += neg ? -a : a;
    }
    if (last >= 0 && (sum & 7) != 0) d.smask |= 1u << last;     // the repair sign
    return true;
}

// word j of a block's codes in coordinate order: nibble n = code of coordinate 8j+n, u = 8 + floor(x / 2)
__device__ __forceinline__ uint32_t code_word(const Decoded &d, int j) {
    uint32_t w = 0;
#pragma unroll
    for (int n = 0; n < 8; n++) {
        const uint32_t a = (d.mag[j] >> (4 * n)) & 15u;
        const bool neg = (d.smask >> (8 * j + n)) & 1u;
        const uint32_t u = neg ? 8u - (a >> 1) - (a & 1u) : 8u + (a >> 1);
        w |= u << (4 * n);
    }
    return w;
}

// nibbles 0..3 of h go to nibbles 0, 2, 4, 6
__device__ __forceinline__ uint32_t spread4(uint32_t h) {
    h &= 0xffffu;
    h = (h | (h << 8)) & 0x00ff00ffu;
    return (h | (h << 4)) & 0x0f0f0f0fu;
}

// One warp writes one piece of a row group: a tile (four blocks), the pair after the tiles or the
// single at the end (see include/llvq.h).  First every lane decodes the blocks of its own row into
// shared memory in coordinate order, then lane 4g+t gathers the words it owns in the layout.
// two header pairs (each two 16-bit fields of which the low byte counts) -> four bytes
__device__ __forceinline__ uint32_t bytes4(uint32_t a, uint32_t b) {
    return (a & 0xffu) | ((a >> 8) & 0xff00u) | ((b & 0xffu) << 16) | ((b << 8) & 0xff000000u);
}

// The window base of the 10-byte layout for a block's 24 four-bit codes (three words of eight nibbles): the
// smallest o in 3..6 with o <= the smallest code and the largest code <= o + 7; 0 if there is none.
__device__ __forceinline__ uint32_t window_base(const uint32_t cw[3]) {
    uint32_t lo = 15u, hi = 0u;
#pragma unroll
    for (int j = 0; j < 3; j++)
#pragma unroll
        for (int n = 0; n < 8; n++) {
            const uint32_t u = (cw[j] >> (4 * n)) & 15u;
            lo = min(lo, u);
            hi = max(hi, u);
        }
    const uint32_t o = max(3u, hi > 7u ? hi - 7u : 0u);
    return o <= min(6u, lo) ? o : 0u;
}

// header byte of the 13-byte layout: shell | parity << 4 | gain << 5 (0 for the empty record)
__device__ __forceinline__ uint32_t header_byte(const DeviceTables &T, const Decoded &d) {
    return d.cls == kEmptyClass ? 0u : ((uint32_t)T.desc[d.cls].shell | ((uint32_t)T.desc[d.cls].odd << 4) | ((uint32_t)d.gain << 5));
}

// LAYOUT = LLVQ_PLANES, LLVQ_PLANES13 (the same code words, the header one byte) or LLVQ_PLANES10X (tiles of
// three-bit window codes, the blocks a window cannot hold listed in the exception table; the leftover blocks as in
// LLVQ_PLANES13).  For LLVQ_PLANES10X `index` holds, on entry, every tile's first entry in the table, and `capacity`
// is the number of entries the table has room for.
template <int LAYOUT>
__global__ void __launch_bounds__(256) expand_planes_kernel(DeviceTables T, const uint64_t *__restrict__ codes, int64_t rows, int64_t nb,
                                                            uint8_t *__restrict__ out, uint32_t *bad_count, uint32_t *ctx_bad,
                                                            const uint32_t *index, uint4 *table, uint32_t capacity) {
    constexpr bool COMPACT = LAYOUT != LLVQ_PLANES, OVERLAY = LAYOUT == LLVQ_PLANES10X;
    __shared__ uint32_t nat_all[8][4][4][32];              // [warp][block of the piece][word 0..2, header][row]
    const int64_t tiles = nb / kTileCells, left = nb % kTileCells;
    const int64_t pieces = tiles + (left >= 2 ? 1 : 0) + (left & 1);
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = (int)(gid & 31);
    const int64_t piece_id = gid >> 5;
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (piece_id >= groups * pieces) return;               // whole warps leave together
    uint32_t (*nat)[4][32] = nat_all[threadIdx.x >> 5];
    const int64_t rg = piece_id / pieces, u = piece_id % pieces;
    const int64_t row = rg * kRowsPerGroup + lane;
    constexpr int kCell = COMPACT ? kCell13Bytes : kCellBytes, kTile = OVERLAY ? kTile10Bytes : (COMPACT ? kTile13Bytes : kTileBytes);
    uint8_t *grp = out + (size_t)rg * ((size_t)tiles * kTile + (size_t)left * kCell);
    const bool is_tile = u < tiles;
    const bool is_pair = !is_tile && left >= 2 && u == tiles;
    const int ncell = is_tile ? 4 : (is_pair ? 2 : 1);
    const int64_t b0 = is_tile ? u * kTileCells : (is_pair ? tiles * kTileCells : nb - 1);
    uint32_t next_entry = 0;                               // OVERLAY: where this tile's next exception goes
    if (OVERLAY && is_tile) next_entry = index[rg * tiles + u];
    int bad = 0;
#pragma unroll 1
    for (int q = 0; q < ncell; q++) {
        Decoded d;
        if (row < rows) {
            if (!decode_code(codes[row * nb + b0 + q], T, d)) bad++;
        } else {
            d.cls = kEmptyClass; d.gain = 0; d.smask = 0; d.mag[0] = d.mag[1] = d.mag[2] = 0;
        }
        uint32_t cw[3] = {code_word(d, 0), code_word(d, 1), code_word(d, 2)};
        uint32_t hdr = COMPACT ? header_byte(T, d) : ((uint32_t)d.cls | ((uint32_t)d.gain << 9));
        if (OVERLAY && is_tile) {
            const uint32_t o = d.cls == kEmptyClass ? 0u : window_base(cw);
            const bool exception = d.cls != kEmptyClass && o == 0u;
            // the tile's exceptions in the order block, row: this block's follow those of the blocks before
            const uint32_t votes = __ballot_sync(0xffffffffu, exception);
            if (exception) {
                const uint32_t at = next_entry + __popc(votes & ((1u << lane) - 1u));
                if (at < capacity) table[at] = make_uint4(hdr | (uint32_t)lane << 8 | (uint32_t)(b0 + q) << 13, cw[0], cw[1], cw[2]);
            }
            next_entry += __popc(votes);
            // no borrow between nibbles: every code is at least o
#pragma unroll
            for (int j = 0; j < 3; j++) cw[j] = o ? cw[j] - o * 0x11111111u : 0u;
            // the short record's header byte: the shell above, and below it window, parity and gain mixed with the shell
            hdr = o ? (((o - 3u) | ((hdr >> 4) & 3u) << 2) ^ (hdr & 15u)) | (hdr & 15u) << 4 : 0u;
        }
        nat[q][0][lane] = cw[0]; nat[q][1][lane] = cw[1]; nat[q][2][lane] = cw[2];
        nat[q][3][lane] = hdr;
    }
    __syncwarp();
    const int g = lane >> 2, t = lane & 3;
    const bool single = !is_tile && !is_pair;
    // four codes of row (m, e, g) starting at position kappa0 (a multiple of 4) of the half-step whose slots are blocks q0, q0+1
    auto quad = [&](int q0, int m, int e, int kappa0) -> uint32_t {
        const int slot = kappa0 / 24, i0 = kappa0 % 24;
        const int r = single ? 16 * slot + 8 * e + g : 16 * m + 8 * e + g;
        const int q = single ? q0 : q0 + slot;
        return nat[q][i0 >> 3][r] >> (16 * ((i0 >> 2) & 1));
    };
    auto header = [&](int q0, int m, int e, int slot) -> uint32_t {
        const int r = single ? 16 * slot + 8 * e + g : 16 * m + 8 * e + g;
        return nat[single ? q0 : q0 + slot][3][r];
    };
    auto half_step = [&](int q0, int m, uint32_t w[3], uint32_t &hw) {
        w[0] = spread4(quad(q0, m, 0, 4 * t)) | spread4(quad(q0, m, 0, 16 + 4 * t)) << 4;
        w[1] = spread4(quad(q0, m, 1, 4 * t)) | spread4(quad(q0, m, 1, 16 + 4 * t)) << 4;
        w[2] = spread4(quad(q0, m, 0, 32 + 4 * t)) | spread4(quad(q0, m, 1, 32 + 4 * t)) << 4;
        hw = header(q0, m, 0, t >> 1) | header(q0, m, 1, t >> 1) << 16;
    };
    if (OVERLAY && is_tile) {
        // Group(h, e, c): byte i = code i of row (m, e, g) at positions 16c + 4t + i (c < 2) or 32 + 4t + i of half-step h
        auto group = [&](int h, int e, int c) -> uint32_t { return spread4(quad(2 * (h >> 1), h & 1, e, (c < 2 ? 16 * c : 32) + 4 * t)); };
        uint32_t V[9], hw[4];
#pragma unroll
        for (int k = 0; k < 8; k++) V[k] = group(k >> 1, k & 1, 0) | group(k >> 1, k & 1, 1) << 3;
        V[8] = group(0, 0, 2) | group(1, 0, 2) << 3;
        // the six groups left go to bits 6, 7: the low two bits of Xk to Vk, its third bit to V(6 + k / 2)
        const uint32_t X[6] = {group(0, 1, 2), group(1, 1, 2), group(2, 0, 2), group(2, 1, 2), group(3, 0, 2), group(3, 1, 2)};
#pragma unroll
        for (int k = 0; k < 6; k++) {
            V[k] |= (X[k] & 0x03030303u) << 6;
            V[6 + (k >> 1)] |= ((X[k] >> 2) & 0x01010101u) << (6 + (k & 1));
        }
#pragma unroll
        for (int h = 0; h < 4; h++) hw[h] = header(2 * (h >> 1), h & 1, 0, t >> 1) | header(2 * (h >> 1), h & 1, 1, t >> 1) << 16;
        uint8_t *tile = grp + (size_t)u * kTile;
        *reinterpret_cast<uint4 *>(tile + 16 * lane) = make_uint4(V[0], V[1], V[2], V[3]);
        *reinterpret_cast<uint4 *>(tile + 512 + 16 * lane) = make_uint4(V[4], V[5], V[6], V[7]);
        *reinterpret_cast<uint32_t *>(tile + 1024 + 4 * lane) = V[8];
        if ((t & 1) == 0) *reinterpret_cast<uint2 *>(tile + 1152 + 8 * (lane >> 1)) = make_uint2(bytes4(hw[0], hw[1]), bytes4(hw[2], hw[3]));
    } else if (is_tile) {
        uint32_t w[12], hw[4];
#pragma unroll
        for (int h = 0; h < 4; h++) half_step(2 * (h >> 1), h & 1, w + 3 * h, hw[h]);
        uint8_t *tile = grp + (size_t)u * kTile;
#pragma unroll
        for (int j = 0; j < 3; j++)
            *reinterpret_cast<uint4 *>(tile + 512 * j + 16 * lane) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        if ((t & 1) == 0) {
            if (COMPACT) *reinterpret_cast<uint2 *>(tile + 1536 + 8 * (lane >> 1)) = make_uint2(bytes4(hw[0], hw[1]), bytes4(hw[2], hw[3]));
            else *reinterpret_cast<uint4 *>(tile + 1536 + 16 * (lane >> 1)) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        }
    } else if (is_pair) {
        uint8_t *pair = grp + (size_t)tiles * kTile;
        uint32_t hw[2];
#pragma unroll
        for (int m = 0; m < 2; m++) {
            uint32_t w[3];
            half_step(0, m, w, hw[m]);
#pragma unroll
            for (int q = 0; q < 3; q++) *reinterpret_cast<uint32_t *>(pair + 128 * (3 * m + q) + 4 * lane) = w[q];
            if (!COMPACT && (t & 1) == 0) *reinterpret_cast<uint32_t *>(pair + 768 + 8 * (lane >> 1) + 4 * m) = hw[m];
        }
        if (COMPACT && (t & 1) == 0) *reinterpret_cast<uint32_t *>(pair + 768 + 4 * (lane >> 1)) = bytes4(hw[0], hw[1]);
    } else {
        uint8_t *one = grp + (size_t)tiles * kTile + (left == 3 ? 2 * kCell : 0);
        uint32_t w[3], hw;
        half_step(0, 0, w, hw);
#pragma unroll
        for (int q = 0; q < 3; q++) *reinterpret_cast<uint32_t *>(one + 128 * q + 4 * lane) = w[q];
        if ((t & 1) == 0) {
            if (COMPACT) *reinterpret_cast<uint16_t *>(one + 384 + 2 * (lane >> 1)) = (uint16_t)((hw & 0xffu) | ((hw >> 8) & 0xff00u));
            else *reinterpret_cast<uint32_t *>(one + 384 + 4 * (lane >> 1)) = hw;
        }
    }
    if (bad) {
        atomicAdd(ctx_bad, (uint32_t)bad);               // the context's own count: llvq_status reports it
        if (bad_count) atomicAdd(bad_count, (uint32_t)bad);
    }
}

__global__ void __launch_bounds__(256) expand_onehot_kernel(DeviceTables T, const uint64_t *__restrict__ codes, int64_t rows, int64_t nb,
                                                            uint8_t *__restrict__ out, uint32_t *bad_count, uint32_t *ctx_bad) {
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = (int)(gid & 31);
    const int64_t cell_id = gid >> 5;
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (cell_id >= groups * nb) return;
    const int64_t rg = cell_id / nb, b = cell_id % nb;
    const int64_t row = rg * kRowsPerGroup + lane;
    Decoded d;
    bool ok = true;
    if (row < rows) ok = decode_code(codes[row * nb + b], T, d);
    else { d.cls = kEmptyClass; d.gain = 0; d.smask = 0; d.mag[0] = d.mag[1] = d.mag[2] = 0; }
    uint32_t mask[4] = {0, 0, 0, 0};
    if (d.cls != kEmptyClass) {
        const uint8_t *dist = T.cls_dist + d.cls * 8;
        const int d1 = dist[1], d2 = dist[2], d3 = dist[3], d4 = dist[4];
        const int nd = T.desc[d.cls].ndist;
#pragma unroll
        for (int i = 0; i < 24; i++) {
            const int a = (int)((d.mag[i >> 3] >> (4 * (i & 7))) & 15u);
            if (nd > 1 && a == d1) mask[0] |= 1u << i;
            if (nd > 2 && a == d2) mask[1] |= 1u << i;
            if (nd > 3 && a == d3) mask[2] |= 1u << i;
            if (nd > 4 && a == d4) mask[3] |= 1u << i;
        }
    }
    uint32_t *cell = reinterpret_cast<uint32_t *>(out + (size_t)cell_id * kOneHotCellBytes);
    cell[0 * 32 + lane] = d.smask | ((uint32_t)(d.cls & 255) << 24);
    cell[1 * 32 + lane] = mask[0] | ((uint32_t)(d.cls >> 8) << 24) | ((uint32_t)d.gain << 25);
    cell[2 * 32 + lane] = mask[1];
    cell[3 * 32 + lane] = mask[2];
    cell[4 * 32 + lane] = mask[3];
    if (!ok) {
        atomicAdd(ctx_bad, 1u);
        if (bad_count) atomicAdd(bad_count, 1u);
    }
}


// ---- the exception table of the 10-byte layout is filled in a fixed order, so its entries' places are known before
// they are written.  One warp a tile counts the tile's exceptions (lane = row).  INDEX: the count goes to the index
// entry after the tile's (the running sum over the index then gives every tile's first entry); else the counts are
// added up in *total.
template <bool INDEX>
__global__ void __launch_bounds__(256) overlay_count_kernel(DeviceTables T, const uint64_t *__restrict__ codes, int64_t rows, int64_t nb,
                                                            uint32_t *index, unsigned long long *total) {
    const int64_t tiles = nb / kTileCells;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = (int)(gid & 31);
    const int64_t tile_id = gid >> 5;
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (tile_id >= groups * tiles) return;
    const int64_t rg = tile_id / tiles, u = tile_id % tiles, row = rg * kRowsPerGroup + lane;
    uint32_t count = 0;
#pragma unroll 1
    for (int q = 0; q < kTileCells; q++) {
        Decoded d;
        bool exception = false;
        if (row < rows && decode_code(codes[row * nb + u * kTileCells + q], T, d)) {
            const uint32_t cw[3] = {code_word(d, 0), code_word(d, 1), code_word(d, 2)};
            exception = window_base(cw) == 0u;
        }
        count += __popc(__ballot_sync(0xffffffffu, exception));
    }
    if (lane == 0) {
        if (INDEX) index[tile_id + 1] = count;
        else if (count) atomicAdd(total, (unsigned long long)count);
    }
}

// One CTA: index[i + 1] = counts of the tiles up to i (index[0] = 0), in place.
__global__ void __launch_bounds__(1024) overlay_index_kernel(uint32_t *index, int64_t n) {
    __shared__ uint32_t warp_sum[32];
    __shared__ uint32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { carry_s = 0; index[0] = 0; }
    __syncthreads();
    for (int64_t base = 0; base < n; base += 1024) {
        const int64_t g = base + tid;
        const uint32_t c = g < n ? index[g + 1] : 0u;
        uint32_t incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += v;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        uint32_t before = carry_s;
        for (int w = 0; w < warp; w++) before += warp_sum[w];
        if (g < n) index[g + 1] = before + incl;
        __syncthreads();
        if (tid == 1023) carry_s = before + incl;
        __syncthreads();
    }
}

// After the table is filled (one CTA): the index stops at the capacity (so that no reader looks past the table), the
// entries that found no room are counted, and the bytes between the parts of the buffer are zeroed.
__global__ void __launch_bounds__(1024) overlay_finish_kernel(uint8_t *out, size_t records_end, size_t index_offset, size_t table_offset,
                                                              int64_t n, uint32_t capacity, uint32_t *overflow) {
    uint32_t *index = reinterpret_cast<uint32_t *>(out + index_offset);
    const int tid = threadIdx.x;
    if (tid == 0 && index[n] > capacity) atomicAdd(overflow, index[n] - capacity);
    __syncthreads();                                       // the total is read before it is clamped
    for (int64_t i = tid; i <= n; i += blockDim.x) index[i] = min(index[i], capacity);
    for (size_t i = records_end + tid; i < index_offset; i += blockDim.x) out[i] = 0;
    for (size_t i = index_offset + (size_t)(n + 1) * 4 + tid; i < table_offset; i += blockDim.x) out[i] = 0;
}

}  // namespace

cudaError_t launch_overlay_count(const llvq_ctx *ctx, const uint64_t *codes, int64_t rows, int64_t nb, unsigned long long *counter,
                                 cudaStream_t s) {
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup, tiles = nb / kTileCells;
    if (tiles == 0) return cudaSuccess;
    const int64_t blocks = (groups * tiles * 32 + 255) / 256;
    overlay_count_kernel<false><<<(unsigned)blocks, 256, 0, s>>>(ctx->dev, codes, rows, nb, nullptr, counter);
    return cudaGetLastError();
}

cudaError_t launch_expand(const llvq_ctx *ctx, int layout, const uint64_t *codes, int64_t rows, int64_t nb,
                          void *out, size_t out_bytes, uint32_t *bad_count, cudaStream_t s) {
    const int64_t groups = (rows + kRowsPerGroup - 1) / kRowsPerGroup;
    if (layout == LLVQ_PLANES || layout == LLVQ_PLANES13 || layout == LLVQ_PLANES10X) {
        const int64_t left = nb % kTileCells, tiles = nb / kTileCells;
        const int64_t pieces = tiles + (left >= 2 ? 1 : 0) + (left & 1);
        const int64_t threads = groups * pieces * 32;
        const int64_t blocks = (threads + 255) / 256;
        if (layout == LLVQ_PLANES10X) {
            uint8_t *o8 = (uint8_t *)out;
            const size_t index_offset = overlay_index_offset(rows, nb), table_offset = overlay_table_offset(rows, nb);
            uint32_t *index = reinterpret_cast<uint32_t *>(o8 + index_offset);
            uint4 *table = reinterpret_cast<uint4 *>(o8 + table_offset);
            const size_t room = (out_bytes - table_offset) / 16;
            const uint32_t capacity = room > 0xffffffffull ? 0xffffffffu : (uint32_t)room;
            // count the tiles' exceptions into the index, turn the counts into first entries, expand, close the index
            if (tiles > 0)
                overlay_count_kernel<true><<<(unsigned)((groups * tiles * 32 + 255) / 256), 256, 0, s>>>(ctx->dev, codes, rows, nb, index, nullptr);
            overlay_index_kernel<<<1, 1024, 0, s>>>(index, groups * tiles);
            expand_planes_kernel<LLVQ_PLANES10X><<<(unsigned)blocks, 256, 0, s>>>(ctx->dev, codes, rows, nb, o8, bad_count, ctx->bad_codes, index, table, capacity);
            overlay_finish_kernel<<<1, 1024, 0, s>>>(o8, (size_t)groups * overlay_group_bytes(nb), index_offset, table_offset, groups * tiles, capacity,
                                                     ctx->overflow);
        } else if (layout == LLVQ_PLANES13) {
            expand_planes_kernel<LLVQ_PLANES13><<<(unsigned)blocks, 256, 0, s>>>(ctx->dev, codes, rows, nb, (uint8_t *)out, bad_count, ctx->bad_codes, nullptr, nullptr, 0);
        } else {
            expand_planes_kernel<LLVQ_PLANES><<<(unsigned)blocks, 256, 0, s>>>(ctx->dev, codes, rows, nb, (uint8_t *)out, bad_count, ctx->bad_codes, nullptr, nullptr, 0);
        }
    } else {
        const int64_t threads = groups * nb * 32;
        const int64_t blocks = (threads + 255) / 256;
        expand_onehot_kernel<<<(unsigned)blocks, 256, 0, s>>>(ctx->dev, codes, rows, nb, (uint8_t *)out, bad_count, ctx->bad_codes);
    }
    return cudaGetLastError();
}

}  // namespace llvq
