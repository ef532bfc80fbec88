// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/llvq.h"
#include "llvq_tables.h"

namespace llvq {

// Geometry of the 14-byte layout (see include/llvq.h).
constexpr int kRowsPerGroup = 32;
constexpr int kCellBytes = 448;        // 32 rows x 14 bytes
constexpr int kTileCells = 4;
constexpr int kTileBytes = 1792;
constexpr int kOneHotCellBytes = 640;  // 32 rows x 20 bytes
constexpr int kCell13Bytes = 416;      // 13-byte layout: 32 rows x 13 bytes
constexpr int kTile13Bytes = 1664;
constexpr int kTile10Bytes = 1280;     // 10-byte layout: 9 words a lane and 128 header bytes a tile; its leftover blocks are 13-byte cells
constexpr int kMaxGridCtas = 256;      // the GEMV launches one CTA a multiprocessor; more multiprocessors than this share the work of 256

// The 10-byte layout's buffer: row groups, then (128-byte aligned) the index, then (128-byte aligned) the exception table.
__host__ __device__ inline size_t overlay_group_bytes(int64_t nb) { return (size_t)(nb / kTileCells) * kTile10Bytes + (size_t)(nb % kTileCells) * kCell13Bytes; }
__host__ __device__ inline size_t overlay_index_offset(int64_t rows, int64_t nb) {
    return ((size_t)((rows + kRowsPerGroup - 1) / kRowsPerGroup) * overlay_group_bytes(nb) + 127) / 128 * 128;
}
__host__ __device__ inline size_t overlay_table_offset(int64_t rows, int64_t nb) {
    // the index: one entry a tile, and one more
    return overlay_index_offset(rows, nb) + ((size_t)((rows + kRowsPerGroup - 1) / kRowsPerGroup * (nb / kTileCells) + 1) * 4 + 127) / 128 * 128;
}

struct DeviceTables {
    const uint64_t *base;            // num_classes + 1
    const ClassDesc *desc;           // num_classes
    const uint32_t *golay_by_weight; // 4096
    const uint32_t *golay_by_message;// 4096
    const float *cls_scale;          // 512
    const uint32_t *cls_parity;      // 512
    const float *cls_value;          // 512 x 8
    const uint8_t *cls_dist;         // 512 x 8
    const float2 *cls_block;         // 512 x {1 / (4 sqrt m), parity - 16}
    const uint4 *lane_table;         // 32 x {b0, b1, b2, xs}: a lane's operand offsets in two consecutive x records
    int weight_offset[25];
    int num_classes;
    uint64_t num_points;
};

// n / d by one multiply-high and one shift, for 0 <= n < 2^31 and a divisor fixed per launch
// (mul = floor(2^(31+l) / d) + 1, shift = l - 1, l = ceil(log2 d); mul = 0 stands for d = 1)
struct FastDiv {
    uint32_t mul, shift;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f = {0u, 0u};
    if (d <= 1) return f;
    uint32_t l = 0;
    while ((1ull << l) < d) l++;
    f.mul = (uint32_t)(((1ull << (31 + l)) / d) + 1);
    f.shift = l - 1;
    return f;
}

struct GemvProblemDev {
    const uint8_t *layout;
    const __half *row_scale;
    float *y;
    int rows;
    int group_begin;   // index of this matrix's first row group in the concatenation
    float gain0, gain1;
    int qexp_base;     // log2 of this matrix's fixed-point quantum, before the exponent of max |x| is added
    const uint32_t *exc_index;   // 10-byte layout: entry i = exception-table entries of this matrix's tiles before tile i (row group by row group)
    const uint4 *exc_table;      // 10-byte layout: the exact records the short records leave out
};

// A CTA's share of a launch, planned on the host: its first unit, the panel that unit lies in and the panel's first
// unit, and the blocks of x [blk_lo, blk_hi) its units touch (the whole panels its range of units meets).
struct CtaShare {
    int first;
    int panel_first;
    uint16_t blk_lo, blk_hi;
    uint16_t panel, pad;
};

struct GemvParams {
    GemvProblemDev prob[LLVQ_MAX_GROUP];
    int nprob;
    const __half *x;             // batch vectors of 24 nb halves, one after the other
    int batch;                   // activation vectors of the launch (1; up to LLVQ_MAX_BATCH through llvq_gemv_batch)
    int y_stride;                // floats between the outputs of consecutive vectors
    int nb, tiles, tail_cells;
    int units;             // units a row group: tiles, plus one for the nb mod 4 last columns
    int total_groups;
    int total_units;       // total_groups * units
    int units_base, units_rem;   // total_units divided by the warps of the grid (set by gemv_plan; the one-hot arm's order)
    int panel, npanels;          // unit columns a panel, panels (set by gemv_plan; the 14-byte layout's order of work)
    FastDiv div_panel_units, div_panel, div_last;   // by total_groups * panel, by panel, by the last panel's width
    int xblocks;                 // most blocks of x any CTA needs (set by gemv_plan)
    uint32_t group_bytes;        // bytes of a row group's records (set by gemv_plan)
    CtaShare cta[kMaxGridCtas + 1];    // the share of every CTA of the grid; [grid].first is the total (set by gemv_plan)
    unsigned long long *accum;   // total_groups x 32 fixed-point row accumulators (context scratch, zero between launches)
    const float *cls_scale;
    const uint32_t *cls_parity;
    const float *cls_value;
    const float2 *cls_block;     // 512 x {1 / (4 sqrt m), parity - 16 as an integer's bits}; zeros for an unused class slot
    const uint4 *lane_table;     // 32 x this lane's offsets of its operand words in the x records of a half-step
    // the class constants the 14-byte GEMV needs, in the parameters themselves (no load from global memory
    // stands between a CTA's start and its block-constant table)
    uint32_t cls_shell_nibbles[64];   // nibble c & 7 of word c >> 3: shell of class c, 0 if unused
    uint32_t cls_odd_bits[16];        // bit c & 31 of word c >> 5: odd type
    float shell_inv_norm[16];         // [m] = 1 / (4 sqrt m)
    int *error;               // set when a bounded wait ran out
    // rotation of x inside the GEMV (llvq_gemv_rotated); rot_log2 = 0 means none
    int rot_log2;             // log2 of the rotation's block length (3..)
    int rot_n;                // coordinates rotated: a multiple of the block length, at most 24 nb
    int rot_span;             // most coordinates any CTA rotates (set by gemv_plan)
    const uint32_t *rot_negate;   // sign-flip bits, or null
    double rot_scale;         // 2^-24 / sqrt(block length)
};

}  // namespace llvq

struct llvq_ctx {
    int device;
    llvq::HostTables host;
    llvq::DeviceTables dev;
    void *table_blob;        // one allocation holding every table
    unsigned long long *accum;   // reduction scratch: one 64-bit accumulator a row of the largest launch
    size_t accum_slots;
    int *error;              // device flag: a kernel's bounded wait ran out
    uint32_t *bad_codes;     // device count: codes that named no point, over the expansions since the last llvq_status
    uint32_t *overflow;      // device count: exception-table entries that found no room, since the last llvq_status
    unsigned long long *counter;   // device scratch of llvq_overlay_count
    int use_pdl;             // launch the GEMV with programmatic stream serialization
    int weights_dirty;       // an expansion was enqueued since the last GEMV: that GEMV must not read records ahead of it
    int sm_count;
    int max_smem_optin;
};

namespace llvq {
cudaError_t launch_expand(const llvq_ctx *ctx, int layout, const uint64_t *codes, int64_t rows, int64_t nb,
                          void *out, size_t out_bytes, uint32_t *bad_count, cudaStream_t s);
// adds the number of blocks the 10-byte layout would keep in its exception table to *counter (device)
cudaError_t launch_overlay_count(const llvq_ctx *ctx, const uint64_t *codes, int64_t rows, int64_t nb, unsigned long long *counter,
                                 cudaStream_t s);
struct GemvLaunch {
    int grid;
    size_t smem;
};
// Completes the launch geometry in `p` (order of work, shares of x) and returns grid and dynamic shared memory.
GemvLaunch gemv_plan(int layout, GemvParams &p, int sm_count);
void gemv_lane_table(uint32_t (*out)[4]);      // fills the 32 entries of DeviceTables::lane_table (host)
cudaError_t launch_gemv(int layout, const GemvParams &p, const GemvLaunch &g, bool no_weights, bool pdl, cudaStream_t s);
cudaError_t launch_wait_limit_selftest(const llvq_ctx *ctx, cudaStream_t s);
cudaError_t launch_gemv_fp16(const __half *W, const __half *x, float *y, int64_t rows, int64_t k, cudaStream_t s);
cudaError_t launch_dequant(const llvq_ctx *ctx, int layout, const uint8_t *buf, const __half *row_scale, float g0, float g1,
                           __half *W, int64_t rows, int64_t nb, cudaStream_t s);
cudaError_t launch_decode_i8(const llvq_ctx *ctx, int layout, const uint8_t *buf, int8_t *coords, uint16_t *class_ids,
                             int64_t rows, int64_t nb, cudaStream_t s);
int gemv_configure(const llvq_ctx *ctx);   // sets the kernels' shared-memory attributes once

// activation rotation: blocks of at most 2^14 coordinates (64-bit partial sums in 128 KiB of shared memory)
constexpr int kRotMaxBlockLog2 = 14;
int rotate_block_log2(int64_t n, int64_t block);   // log2 of the block length used, -1 if `block` is not acceptable
int rotate_configure();                            // sets the kernel's shared-memory attribute once a device
cudaError_t launch_rotate(const __half *x, __half *y, const uint32_t *negate, int64_t n, int block_log2, bool pdl,
                          cudaStream_t s);
}  // namespace llvq
