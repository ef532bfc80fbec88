// C ABI of the library: argument checks, context set-up, and the hand-off to the kernels.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "llvq_internal.cuh"

using namespace llvq;

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// The fixed-point quantum is a power of two formed from the exponent of the larger gain: gains whose larger
// magnitude lies outside [2^-60, 2^60) (zero excepted: a matrix of zero gain is all zeros) are refused.
bool gain_in_range(const float *gain) {
    const float gm = std::fmax(std::fabs(gain[0]), std::fabs(gain[1]));
    return gm == 0.f || (gm >= 8.673617379884035e-19f && gm < 1.152921504606847e18f);
}

int layout_cell_bytes(int layout) { return layout == LLVQ_PLANES ? kCellBytes : (layout == LLVQ_PLANES13 ? kCell13Bytes : kOneHotCellBytes); }

}  // namespace

extern "C" {

const char *llvq_strerror(int code) {
    switch (code) {
        case LLVQ_OK: return "ok";
        case LLVQ_EINVAL: return "invalid argument (null pointer, bad shape or unknown layout)";
        case LLVQ_EALIGN: return "device pointer not aligned as documented";
        case LLVQ_ESIZE: return "buffer or context scratch too small (from llvq_status: an exception table had no room for some of its entries)";
        case LLVQ_ECUDA: return "CUDA runtime error";
        case LLVQ_ETIMEOUT: return "a bounded wait inside a kernel ran out; the affected outputs are incomplete";
        case LLVQ_EINDEX: return "a code word named no point of the ball (index out of range or bits above bit 47 set); its record is empty";
        default: return "unknown error";
    }
}

int llvq_create(llvq_ctx **out, int device, size_t scratch_bytes) {
    if (!out) return LLVQ_EINVAL;
    *out = nullptr;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) return LLVQ_ECUDA;
    if (device < 0 || device >= ndev) return LLVQ_EINVAL;
    DeviceGuard guard(device);
    if (!guard.ok) return LLVQ_ECUDA;
    llvq_ctx *ctx = new (std::nothrow) llvq_ctx();
    if (!ctx) return LLVQ_ECUDA;
    ctx->device = device;
    ctx->table_blob = nullptr; ctx->accum = nullptr; ctx->error = nullptr; ctx->bad_codes = nullptr; ctx->use_pdl = 1; ctx->weights_dirty = 0;
    if (!build_tables(ctx->host)) { delete ctx; return LLVQ_EINVAL; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return LLVQ_ECUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_smem_optin = (int)prop.sharedMemPerBlockOptin;

    const HostTables &h = ctx->host;
    uint32_t lanes[32][4];
    gemv_lane_table(lanes);
    struct Part { const void *src; size_t bytes; size_t off; } parts[10] = {
        {h.base.data(), h.base.size() * 8, 0},          {h.desc.data(), h.desc.size() * sizeof(ClassDesc), 0},
        {h.golay_by_weight.data(), 4096 * 4, 0},        {h.golay_by_message.data(), 4096 * 4, 0},
        {h.cls_scale.data(), kClassSlots * 4, 0},       {h.cls_parity.data(), kClassSlots * 4, 0},
        {h.cls_value.data(), kClassSlots * 8 * 4, 0},   {h.cls_dist.data(), kClassSlots * 8, 0},
        {h.cls_block.data(), kClassSlots * 8, 0},       {lanes, sizeof lanes, 0}};
    size_t total = 0;
    for (auto &p : parts) { p.off = total; total += round_up(p.bytes, 256); }
    if (cudaMalloc(&ctx->table_blob, total) != cudaSuccess) { delete ctx; return LLVQ_ECUDA; }
    for (auto &p : parts)
        if (cudaMemcpy((char *)ctx->table_blob + p.off, p.src, p.bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
            llvq_destroy(ctx);
            return LLVQ_ECUDA;
        }
    char *blob = (char *)ctx->table_blob;
    DeviceTables &d = ctx->dev;
    d.base = (const uint64_t *)(blob + parts[0].off);
    d.desc = (const ClassDesc *)(blob + parts[1].off);
    d.golay_by_weight = (const uint32_t *)(blob + parts[2].off);
    d.golay_by_message = (const uint32_t *)(blob + parts[3].off);
    d.cls_scale = (const float *)(blob + parts[4].off);
    d.cls_parity = (const uint32_t *)(blob + parts[5].off);
    d.cls_value = (const float *)(blob + parts[6].off);
    d.cls_dist = (const uint8_t *)(blob + parts[7].off);
    d.cls_block = (const float2 *)(blob + parts[8].off);
    d.lane_table = (const uint4 *)(blob + parts[9].off);
    std::memcpy(d.weight_offset, h.weight_offset, sizeof d.weight_offset);
    d.num_classes = h.num_classes;
    d.num_points = h.num_points;

    if (scratch_bytes == 0) scratch_bytes = (size_t)8 << 20;
    ctx->accum_slots = scratch_bytes / 8;
    if (cudaMalloc(&ctx->accum, ctx->accum_slots * 8) != cudaSuccess ||
        cudaMemset(ctx->accum, 0, ctx->accum_slots * 8) != cudaSuccess ||
        cudaMalloc(&ctx->error, 32) != cudaSuccess || cudaMemset(ctx->error, 0, 32) != cudaSuccess) {
        llvq_destroy(ctx);
        return LLVQ_ECUDA;
    }
    // one small block: the error flag, the two counts llvq_status reports, and the scratch of llvq_overlay_count
    ctx->bad_codes = reinterpret_cast<uint32_t *>(ctx->error + 1);
    ctx->overflow = reinterpret_cast<uint32_t *>(ctx->error + 2);
    ctx->counter = reinterpret_cast<unsigned long long *>(ctx->error + 4);
    if (gemv_configure(ctx) != 0 || rotate_configure() != 0 || cudaDeviceSynchronize() != cudaSuccess) { llvq_destroy(ctx); return LLVQ_ECUDA; }
    *out = ctx;
    return LLVQ_OK;
}

void llvq_destroy(llvq_ctx *ctx) {
    if (!ctx) return;
    DeviceGuard guard(ctx->device);
    cudaFree(ctx->table_blob);
    cudaFree(ctx->accum);
    cudaFree(ctx->error);
    delete ctx;
}

int llvq_status(llvq_ctx *ctx, void *stream) {
    if (!ctx) return LLVQ_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    int flags[3] = {0, 0, 0};                          // {a wait ran out, codes that named no point, table entries without room}
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemcpy(flags, ctx->error, 12, cudaMemcpyDeviceToHost) != cudaSuccess) return LLVQ_ECUDA;
    if (flags[0]) {
        cudaMemset(ctx->error, 0, 4);
        cudaMemset(ctx->accum, 0, ctx->accum_slots * 8);   // an abandoned reduction leaves sums behind
        return LLVQ_ETIMEOUT;
    }
    if (flags[2]) {
        cudaMemset(ctx->overflow, 0, 4);
        return LLVQ_ESIZE;
    }
    if (flags[1]) {
        cudaMemset(ctx->bad_codes, 0, 4);
        return LLVQ_EINDEX;
    }
    return LLVQ_OK;
}

int llvq_selftest_wait_limit(llvq_ctx *ctx, void *stream) {
    if (!ctx) return LLVQ_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return launch_wait_limit_selftest(ctx, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_set_pdl(llvq_ctx *ctx, int enabled) {
    if (!ctx) return LLVQ_EINVAL;
    ctx->use_pdl = enabled ? 1 : 0;
    return LLVQ_OK;
}

int llvq_num_classes(const llvq_ctx *ctx) { return ctx ? ctx->host.num_classes : LLVQ_EINVAL; }

uint64_t llvq_class_base(const llvq_ctx *ctx, int c) {
    if (!ctx || c < 0 || c > ctx->host.num_classes) return ~0ull;
    return ctx->host.base[(size_t)c];
}

int llvq_overlay_bytes(int64_t rows, int64_t k_padded, uint64_t exceptions, size_t *bytes) {
    if (!bytes || rows <= 0 || k_padded <= 0 || k_padded % 24 != 0 || k_padded / 24 >= ((int64_t)1 << 19)) return LLVQ_EINVAL;
    *bytes = overlay_table_offset(rows, k_padded / 24) + (size_t)exceptions * 16;
    return LLVQ_OK;
}

int llvq_overlay_count(llvq_ctx *ctx, const uint64_t *codes, int64_t rows, int64_t nb, uint64_t *count, void *stream) {
    if (!ctx || !codes || !count || rows <= 0 || nb <= 0 || nb >= ((int64_t)1 << 19)) return LLVQ_EINVAL;
    if (!aligned(codes, 8)) return LLVQ_EALIGN;
    if (rows * nb > ((int64_t)1 << 36)) return LLVQ_ESIZE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t s = (cudaStream_t)stream;
    unsigned long long n = 0;
    if (cudaMemsetAsync(ctx->counter, 0, 8, s) != cudaSuccess || launch_overlay_count(ctx, codes, rows, nb, ctx->counter, s) != cudaSuccess ||
        cudaMemcpyAsync(&n, ctx->counter, 8, cudaMemcpyDeviceToHost, s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess)
        return LLVQ_ECUDA;
    *count = n;
    return LLVQ_OK;
}

int llvq_layout_bytes(int layout, int64_t rows, int64_t k_padded, size_t *bytes) {
    if (!bytes || rows <= 0 || k_padded <= 0 || k_padded % 24 != 0) return LLVQ_EINVAL;
    if (layout == LLVQ_PLANES10X)       // room for one exception in 32 blocks
        return llvq_overlay_bytes(rows, k_padded, (uint64_t)((rows * (k_padded / 24) + 31) / 32), bytes);
    if (layout != LLVQ_PLANES && layout != LLVQ_ONEHOT && layout != LLVQ_PLANES13) return LLVQ_EINVAL;
    const size_t groups = (size_t)((rows + kRowsPerGroup - 1) / kRowsPerGroup);
    *bytes = groups * (size_t)(k_padded / 24) * (size_t)layout_cell_bytes(layout);
    return LLVQ_OK;
}

int llvq_expand(llvq_ctx *ctx, int layout, const uint64_t *codes, int64_t rows, int64_t nb, void *layout_out,
                size_t out_bytes, uint32_t *bad_count, void *stream) {
    if (!ctx || !codes || !layout_out || rows <= 0 || nb <= 0) return LLVQ_EINVAL;
    size_t need = 0;
    // the 10-byte layout takes whatever room the buffer has past its fixed part for the exception table
    if ((layout == LLVQ_PLANES10X ? llvq_overlay_bytes(rows, nb * 24, 0, &need) : llvq_layout_bytes(layout, rows, nb * 24, &need)) != LLVQ_OK) return LLVQ_EINVAL;
    if (out_bytes < need) return LLVQ_ESIZE;
    if (!aligned(layout_out, 128) || !aligned(codes, 8) || (bad_count && !aligned(bad_count, 4))) return LLVQ_EALIGN;
    if (rows * nb > ((int64_t)1 << 36)) return LLVQ_ESIZE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    // the GEMV reads records ahead of its wait for the previous kernel of the stream: the next one on this context
    // is launched as an ordinary kernel, so that it cannot overtake this expansion
    ctx->weights_dirty = 1;
    return launch_expand(ctx, layout, codes, rows, nb, layout_out, out_bytes, bad_count, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

constexpr int kVectorsPerPass = 4;      // activation vectors one launch of the GEMV kernel carries

int llvq_gemv_plan(int sm_count, const int64_t *rows, int n, int64_t k_padded, int batch, int32_t *out, int out_len) {
    if (!rows || !out || n < 1 || n > LLVQ_MAX_GROUP || sm_count < 1 || batch < 1 || batch > kVectorsPerPass) return LLVQ_EINVAL;
    if (k_padded <= 0 || k_padded % 24 != 0) return LLVQ_EINVAL;
    if (k_padded > LLVQ_MAX_K) return LLVQ_ESIZE;
    GemvParams p;
    std::memset(&p, 0, sizeof p);
    p.nprob = n;
    p.batch = batch;
    p.nb = (int)(k_padded / 24);
    p.tiles = p.nb / kTileCells;
    p.tail_cells = p.nb % kTileCells;
    p.units = p.tiles + (p.tail_cells ? 1 : 0);
    int64_t groups = 0;
    for (int i = 0; i < n; i++) {
        if (rows[i] <= 0 || rows[i] > ((int64_t)1 << 30)) return LLVQ_EINVAL;
        p.prob[i].group_begin = (int)groups;
        p.prob[i].rows = (int)rows[i];
        groups += (rows[i] + kRowsPerGroup - 1) / kRowsPerGroup;
    }
    if (groups > ((int64_t)1 << 26) || p.units > 2047 || groups * p.units > 0x7fffffffll) return LLVQ_ESIZE;
    p.total_groups = (int)groups;
    p.total_units = (int)(groups * p.units);
    const GemvLaunch g = gemv_plan(LLVQ_PLANES, p, sm_count);
    if (out_len < 8 + g.grid + 1) return LLVQ_ESIZE;
    out[0] = g.grid; out[1] = (int32_t)g.smem; out[2] = p.units; out[3] = p.total_units;
    out[4] = p.panel; out[5] = p.npanels; out[6] = p.xblocks; out[7] = p.total_groups;
    for (int c = 0; c <= g.grid; c++) out[8 + c] = p.cta[c].first;
    return LLVQ_OK;
}

static int run_gemv(llvq_ctx *ctx, int layout, const llvq_problem *problems, int n, const void *x, int64_t k_padded,
                    bool no_weights, void *stream, int batch = 1, const llvq_rotation *rot = nullptr) {
    if (!ctx || !problems || !x || n < 1 || n > LLVQ_MAX_GROUP) return LLVQ_EINVAL;
    if (batch < 1 || batch > kVectorsPerPass || (batch > 1 && (n != 1 || layout != LLVQ_PLANES || no_weights))) return LLVQ_EINVAL;
    if (layout != LLVQ_PLANES && layout != LLVQ_ONEHOT && layout != LLVQ_PLANES13 && layout != LLVQ_PLANES10X) return LLVQ_EINVAL;
    if ((layout == LLVQ_PLANES13 || layout == LLVQ_PLANES10X) && (no_weights || batch != 1 || rot)) return LLVQ_EINVAL;
    if (layout == LLVQ_PLANES10X && k_padded / 24 >= ((int64_t)1 << 19)) return LLVQ_EINVAL;
    if (k_padded <= 0 || k_padded % 24 != 0) return LLVQ_EINVAL;
    if (k_padded > LLVQ_MAX_K) return LLVQ_ESIZE;
    if (!aligned(x, 16)) return LLVQ_EALIGN;
    GemvParams p;
    std::memset(&p, 0, sizeof p);
    p.nprob = n;
    p.x = (const __half *)x;
    p.batch = batch;
    p.y_stride = (int)problems[0].rows;
    p.nb = (int)(k_padded / 24);
    p.tiles = p.nb / kTileCells;
    p.tail_cells = p.nb % kTileCells;
    p.units = p.tiles + (p.tail_cells ? 1 : 0);
    int64_t groups = 0;
    float gain_max = 0.f;
    for (int i = 0; i < n; i++) {
        const llvq_problem &q = problems[i];
        if ((!q.layout && !no_weights) || !q.row_scale || !q.y || q.rows <= 0) return LLVQ_EINVAL;
        if (!aligned(q.layout, 128) || !aligned(q.row_scale, 2) || !aligned(q.y, 4)) return LLVQ_EALIGN;
        p.prob[i].layout = (const uint8_t *)q.layout;
        p.prob[i].row_scale = (const __half *)q.row_scale;
        p.prob[i].y = q.y;
        p.prob[i].rows = (int)q.rows;
        p.prob[i].group_begin = (int)groups;
        p.prob[i].gain0 = q.gain[0];
        p.prob[i].gain1 = q.gain[1];
        if (layout == LLVQ_PLANES10X) {
            p.prob[i].exc_index = reinterpret_cast<const uint32_t *>(p.prob[i].layout + overlay_index_offset(q.rows, p.nb));
            p.prob[i].exc_table = reinterpret_cast<const uint4 *>(p.prob[i].layout + overlay_table_offset(q.rows, p.nb));
        }
        gain_max = std::fmax(gain_max, std::fmax(std::fabs(q.gain[0]), std::fabs(q.gain[1])));
        if (q.rows > ((int64_t)1 << 30)) return LLVQ_ESIZE;
        groups += (q.rows + kRowsPerGroup - 1) / kRowsPerGroup;
    }
    if (groups > ((int64_t)1 << 26) || p.units > 2047 || groups * p.units > 0x7fffffffll) return LLVQ_ESIZE;
    if ((size_t)groups * 32 * (size_t)batch > ctx->accum_slots) return LLVQ_ESIZE;
    if (!(gain_max < 3.0e38f)) return LLVQ_EINVAL;
    for (int i = 0; i < n; i++)
        if (!gain_in_range(problems[i].gain)) return LLVQ_EINVAL;
    // quantum of the fixed-point row accumulators, per matrix so that grouping does not change it:
    // a unit sums at most four blocks, each bounded by max|gain| * sqrt(24) * max|x| < 2^ge * 5 * 2^xe;
    // 4 * 5 < 2^5, and the unit value is kept under 2^39 quanta (see deliver() in llvq_gemv.cu), which
    // puts the quantum some 2^-32 below a typical unit sum: far finer than the f32 sums it collects
    for (int i = 0; i < n; i++) {
        const float gm = std::fmax(std::fabs(problems[i].gain[0]), std::fabs(problems[i].gain[1]));
        int ge = 0;
        std::frexp(gm > 0.f ? gm : 1.f, &ge);                              // gm < 2^ge
        p.prob[i].qexp_base = ge + 5 - 39;
    }
    p.total_groups = (int)groups;
    p.total_units = (int)(groups * p.units);
    p.accum = ctx->accum;
    p.cls_scale = ctx->dev.cls_scale;
    p.cls_parity = ctx->dev.cls_parity;
    p.cls_value = ctx->dev.cls_value;
    p.cls_block = ctx->dev.cls_block;
    p.lane_table = ctx->dev.lane_table;
    std::memcpy(p.cls_shell_nibbles, ctx->host.cls_shell_nibbles, sizeof p.cls_shell_nibbles);
    std::memcpy(p.cls_odd_bits, ctx->host.cls_odd_bits, sizeof p.cls_odd_bits);
    std::memcpy(p.shell_inv_norm, ctx->host.shell_inv_norm, sizeof p.shell_inv_norm);
    p.error = ctx->error;
    if (rot) {
        // the rotation acts on the first rot->n entries of x; what follows (the padding) passes through
        if (layout != LLVQ_PLANES || no_weights || batch != 1 || rot->n <= 0 || rot->n > k_padded || rot->n % 8 != 0) return LLVQ_EINVAL;
        const int l = rotate_block_log2(rot->n, rot->block);
        if (l < 3) return LLVQ_EINVAL;                 // blocks shorter than eight: rotate with llvq_rotate instead
        if (!aligned(rot->negate_bits, 4)) return LLVQ_EALIGN;
        p.rot_log2 = l;
        p.rot_n = (int)rot->n;
        p.rot_negate = rot->negate_bits;
        p.rot_scale = std::ldexp(1.0 / std::sqrt((double)((int64_t)1 << l)), -24);
    }
    const GemvLaunch g = gemv_plan(layout, p, ctx->sm_count);
    if (g.smem + 1024 > (size_t)ctx->max_smem_optin) return LLVQ_ESIZE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const bool pdl = ctx->use_pdl != 0 && !ctx->weights_dirty;
    ctx->weights_dirty = 0;
    return launch_gemv(layout, p, g, no_weights, pdl, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_gemv(llvq_ctx *ctx, int layout, const void *layout_buf, const void *row_scale, const float *gain, const void *x,
              float *y, int64_t rows, int64_t k_padded, void *stream) {
    if (!gain) return LLVQ_EINVAL;
    llvq_problem q;
    q.layout = layout_buf; q.row_scale = row_scale; q.y = y; q.rows = rows; q.gain[0] = gain[0]; q.gain[1] = gain[1];
    return run_gemv(ctx, layout, &q, 1, x, k_padded, false, stream);
}

int llvq_gemv_batch(llvq_ctx *ctx, const void *layout_buf, const void *row_scale, const float *gain, const void *x, float *y,
                    int64_t rows, int64_t k_padded, int batch, void *stream) {
    if (!gain || !y || !x || batch < 1 || batch > LLVQ_MAX_BATCH || rows <= 0 || k_padded <= 0) return LLVQ_EINVAL;
    // the kernel carries up to four vectors a pass; a larger batch is that many passes over the records, one
    // after the other on the stream (they share the context's scratch)
    for (int first = 0; first < batch; first += kVectorsPerPass) {
        const int n = batch - first < kVectorsPerPass ? batch - first : kVectorsPerPass;
        llvq_problem q;
        q.layout = layout_buf; q.row_scale = row_scale; q.y = y + (size_t)first * (size_t)rows; q.rows = rows;
        q.gain[0] = gain[0]; q.gain[1] = gain[1];
        const int rc = run_gemv(ctx, LLVQ_PLANES, &q, 1, (const __half *)x + (size_t)first * (size_t)k_padded, k_padded, false, stream, n);
        if (rc != LLVQ_OK) return rc;
    }
    return LLVQ_OK;
}

int llvq_gemv_grouped(llvq_ctx *ctx, int layout, const llvq_problem *problems, int n, const void *x, int64_t k_padded,
                      void *stream) {
    return run_gemv(ctx, layout, problems, n, x, k_padded, false, stream);
}

int llvq_gemv_rotated(llvq_ctx *ctx, const llvq_problem *problems, int n, const void *x, int64_t k_padded,
                      const llvq_rotation *rotation, void *stream) {
    if (!rotation) return LLVQ_EINVAL;
    return run_gemv(ctx, LLVQ_PLANES, problems, n, x, k_padded, false, stream, 1, rotation);
}

int llvq_gemv_noweights(llvq_ctx *ctx, const void *row_scale, const void *x, float *y, int64_t rows, int64_t k_padded,
                        void *stream) {
    llvq_problem q;
    q.layout = nullptr; q.row_scale = row_scale; q.y = y; q.rows = rows; q.gain[0] = 1.f; q.gain[1] = 1.f;
    return run_gemv(ctx, LLVQ_PLANES, &q, 1, x, k_padded, true, stream);
}

int llvq_gemv_fp16(const void *W, const void *x, float *y, int64_t rows, int64_t k, void *stream) {
    if (!W || !x || !y || rows <= 0 || k <= 0 || k % 8 != 0) return LLVQ_EINVAL;
    if (!aligned(W, 16) || !aligned(x, 16) || !aligned(y, 4)) return LLVQ_EALIGN;
    if ((rows + 7) / 8 > 0x7fffffffll) return LLVQ_ESIZE;
    return launch_gemv_fp16((const __half *)W, (const __half *)x, y, rows, k, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int64_t llvq_rotate_block(int64_t n, int64_t block) {
    const int l = rotate_block_log2(n, block);
    return l < 0 ? 0 : (int64_t)1 << l;
}

int llvq_rotate(llvq_ctx *ctx, const void *x, void *y, const uint32_t *negate_bits, int64_t n, int64_t block, void *stream) {
    if (!ctx || !x || !y || n <= 0 || n % 8 != 0) return LLVQ_EINVAL;
    const int l = rotate_block_log2(n, block);
    if (l < 0) return LLVQ_EINVAL;
    if (!aligned(x, 16) || !aligned(y, 16) || !aligned(negate_bits, 4)) return LLVQ_EALIGN;
    if (n > ((int64_t)1 << 40)) return LLVQ_ESIZE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return launch_rotate((const __half *)x, (__half *)y, negate_bits, n, l, ctx->use_pdl != 0, (cudaStream_t)stream) == cudaSuccess
               ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_dequant_fp16(llvq_ctx *ctx, int layout, const void *layout_buf, const void *row_scale, const float *gain, void *W,
                      int64_t rows, int64_t k_padded, void *stream) {
    if (!ctx || !layout_buf || !row_scale || !gain || !W || rows <= 0 || k_padded <= 0 || k_padded % 24 != 0) return LLVQ_EINVAL;
    if (layout != LLVQ_PLANES && layout != LLVQ_ONEHOT) return LLVQ_EINVAL;
    if (!aligned(layout_buf, 128) || !aligned(W, 16) || !aligned(row_scale, 2)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return launch_dequant(ctx, layout, (const uint8_t *)layout_buf, (const __half *)row_scale, gain[0], gain[1], (__half *)W, rows,
                          k_padded / 24, (cudaStream_t)stream) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

int llvq_decode_i8(llvq_ctx *ctx, int layout, const void *layout_buf, int8_t *coords, uint16_t *class_ids, int64_t rows,
                   int64_t nb, void *stream) {
    if (!ctx || !layout_buf || !coords || !class_ids || rows <= 0 || nb <= 0) return LLVQ_EINVAL;
    if (layout != LLVQ_PLANES && layout != LLVQ_ONEHOT && layout != LLVQ_PLANES13 && layout != LLVQ_PLANES10X) return LLVQ_EINVAL;
    if (!aligned(layout_buf, 128) || !aligned(class_ids, 2)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return launch_decode_i8(ctx, layout, (const uint8_t *)layout_buf, coords, class_ids, rows, nb, (cudaStream_t)stream) == cudaSuccess
               ? LLVQ_OK : LLVQ_ECUDA;
}

}  // extern "C"
