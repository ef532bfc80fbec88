// The fused dequantize-plus-matvec (paper Sec. 2.3, "The kernel"), re-designed for sm_100a.
//
// Geometry.  A lane owns a row: the 32 lanes of a warp work on the 32 rows of one row group and
// walk the same block columns together, so every read of x is a shared-memory broadcast and no
// shuffle reduction is needed.  A work item is (row group, chunk of kChunkTiles tiles); items
// are dealt round-robin to the warps of a grid sized to the machine.  Each item leaves a
// 32-float partial in the context's scratch; the warp that delivers the last partial of a row
// group adds them in chunk order, applies the row scale and writes y.  The order of additions
// for a row therefore depends on nb alone.
//
// Decode.  One rotate and one three-input logic op turn a payload word into a pair of fp16 bit
// patterns whose value is (+-)|x_i| * 2^-21 (a subnormal built in place: level bits at [6:4],
// the class parity or-ed in at bit 3, the sign at bit 15).  A mixed-precision fused multiply-add
// (fp16 x fp16 + f32) accumulates the exact product with the fp16 activation.  Per block one
// multiply applies gain[g] * 2^21 / (4 sqrt m), looked up by the 10-bit header.  Every lane runs
// the same instructions whatever its class.
#include "llvq_internal.cuh"

namespace llvq {
namespace {

constexpr int kWarps = 16;                 // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kPairMask = 0x80708070u;

struct BlockConst { float scale; uint32_t parity; };   // indexed by class | gain << 9

__device__ __forceinline__ void fma_pair(float &lo, float &hi, uint32_t w, uint32_t x) {
    asm("{\n\t.reg .f16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %2;\n\t"
        "mov.b32 {xl, xh}, %3;\n\t"
        "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
        "fma.rn.f32.f16 %1, wh, xh, %1;\n\t}"
        : "+f"(lo), "+f"(hi)
        : "r"(w), "r"(x));
}

// sum over the 24 coordinates of one block of (+-|x_i| * 2^-21) * x[i]
__device__ __forceinline__ float block_dot(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t parity, const uint4 *xs) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    const uint32_t w[3] = {w0, w1, w2};
#pragma unroll
    for (int j = 0; j < 3; j++) {
        const uint4 xv = xs[j];                      // x[8j .. 8j+7] as four fp16 pairs (broadcast read)
        const uint32_t xp[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const uint32_t r = k ? __funnelshift_r(w[j], w[j], 4 * k) : w[j];
            const uint32_t v = (r & kPairMask) | parity;
            if (k & 1) fma_pair(a2, a3, v, xp[k]); else fma_pair(a0, a1, v, xp[k]);
        }
    }
    return (a0 + a1) + (a2 + a3);
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

// Delivers one item's partial; the last arrival of a row group finishes the rows.
__device__ __forceinline__ void deliver(const GemvParams &p, const GemvProblemDev &pr, int group, int chunk, int lane, float acc) {
    const int row = (group - pr.group_begin) * kRowsPerGroup + lane;
    if (p.nchunk == 1) {
        if (row < pr.rows) pr.y[row] = acc * __half2float(pr.row_scale[row]);
        return;
    }
    float *slot = p.partial + ((size_t)group * p.nchunk) * 32;
    __stcg(slot + chunk * 32 + lane, acc);
    __threadfence();
    unsigned old = 0;
    if (lane == 0) old = atomicAdd(p.counter + group, 1u);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old == (unsigned)p.nchunk - 1) {
        __threadfence();
        float sum = 0.f;
        for (int c = 0; c < p.nchunk; c++) sum += __ldcg(slot + c * 32 + lane);
        if (row < pr.rows) pr.y[row] = sum * __half2float(pr.row_scale[row]);
        if (lane == 0) p.counter[group] = 0;      // leave the scratch ready for the next launch
    }
}

template <bool NO_WEIGHTS>
__global__ void __launch_bounds__(kThreads, 1) gemv_planes_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    BlockConst *bc = reinterpret_cast<BlockConst *>(smem);                 // 1024 entries a matrix of the group
    uint4 *xs = reinterpret_cast<uint4 *>(smem + (size_t)p.nprob * 1024 * sizeof(BlockConst));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // block constants per problem: gain[g] * 2^21 / (4 sqrt m) and the parity pattern
    for (int e = tid; e < p.nprob * 1024; e += kThreads) {
        const int q = e >> 10, c = e & 511, g = (e >> 9) & 1;
        BlockConst v;
        v.scale = p.cls_scale[c] * (g ? p.prob[q].gain1 : p.prob[q].gain0);
        v.parity = p.cls_parity[c];
        bc[e] = v;
    }
    // x, once per CTA: 3 nb 16-byte words
    const uint4 *xg = reinterpret_cast<const uint4 *>(p.x);
    for (int e = tid; e < 3 * p.nb; e += kThreads) xs[e] = __ldg(xg + e);
    __syncthreads();

    const int warps_total = gridDim.x * kWarps;
    for (int item = warp * gridDim.x + blockIdx.x; item < p.total_items; item += warps_total) {
        const int group = item / p.nchunk, chunk = item - group * p.nchunk;
        const int q = find_problem(p, group);
        const GemvProblemDev &pr = p.prob[q];
        const uint8_t *grp = pr.layout + (size_t)(group - pr.group_begin) * (size_t)p.nb * kCellBytes;
        const BlockConst *bcq = bc + q * 1024;
        const int t0 = chunk * kChunkTiles, t1 = min(t0 + kChunkTiles, p.tiles);
        float acc = 0.f;
        if (!NO_WEIGHTS) {
            for (int t = t0; t < t1; t++) {
                const uint8_t *tile = grp + (size_t)t * kTileBytes;
                const uint4 a0 = __ldcs(reinterpret_cast<const uint4 *>(tile + 16 * lane));
                const uint4 a1 = __ldcs(reinterpret_cast<const uint4 *>(tile + 512 + 16 * lane));
                const uint4 a2 = __ldcs(reinterpret_cast<const uint4 *>(tile + 1024 + 16 * lane));
                const uint2 hh = __ldcs(reinterpret_cast<const uint2 *>(tile + 1536 + 8 * lane));
                const uint32_t w0[4] = {a0.x, a0.y, a0.z, a0.w}, w1[4] = {a1.x, a1.y, a1.z, a1.w}, w2[4] = {a2.x, a2.y, a2.z, a2.w};
                const uint32_t hd[4] = {hh.x & 0xffffu, hh.x >> 16, hh.y & 0xffffu, hh.y >> 16};
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    const BlockConst k = bcq[hd[c] & 1023u];
                    const float dot = block_dot(w0[c], w1[c], w2[c], k.parity, xs + 3 * (4 * t + c));
                    acc = fmaf(k.scale, dot, acc);
                }
            }
            if (chunk == p.nchunk - 1) {
                for (int c = 0; c < p.tail_cells; c++) {
                    const uint8_t *cell = grp + (size_t)p.tiles * kTileBytes + (size_t)c * kCellBytes;
                    const uint32_t w0 = __ldcs(reinterpret_cast<const uint32_t *>(cell + 4 * lane));
                    const uint32_t w1 = __ldcs(reinterpret_cast<const uint32_t *>(cell + 128 + 4 * lane));
                    const uint32_t w2 = __ldcs(reinterpret_cast<const uint32_t *>(cell + 256 + 4 * lane));
                    const uint32_t hd = *reinterpret_cast<const uint16_t *>(cell + 384 + 2 * lane);
                    const BlockConst k = bcq[hd & 1023u];
                    const float dot = block_dot(w0, w1, w2, k.parity, xs + 3 * (4 * p.tiles + c));
                    acc = fmaf(k.scale, dot, acc);
                }
            }
        }
        deliver(p, pr, group, chunk, lane, acc);
    }
}

__global__ void __launch_bounds__(kThreads, 1) gemv_onehot_kernel(const __grid_constant__ GemvParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4 *xs4 = reinterpret_cast<uint4 *>(smem);
    const __half *xs = reinterpret_cast<const __half *>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4 *xg = reinterpret_cast<const uint4 *>(p.x);
    for (int e = tid; e < 3 * p.nb; e += kThreads) xs4[e] = __ldg(xg + e);
    __syncthreads();
    const int warps_total = gridDim.x * kWarps;
    for (int item = warp * gridDim.x + blockIdx.x; item < p.total_items; item += warps_total) {
        const int group = item / p.nchunk, chunk = item - group * p.nchunk;
        const int q = find_problem(p, group);
        const GemvProblemDev &pr = p.prob[q];
        const uint8_t *grp = pr.layout + (size_t)(group - pr.group_begin) * (size_t)p.nb * kOneHotCellBytes;
        // same chunking as the bit-plane kernel: tiles of four cells, the tail cells in the last chunk
        const int c0 = chunk * kChunkTiles * kTileCells;
        const int c1 = (chunk == p.nchunk - 1) ? p.nb : min(c0 + kChunkTiles * kTileCells, p.tiles * kTileCells);
        float acc = 0.f;
        for (int c = c0; c < c1; c++) {
            const uint32_t *cell = reinterpret_cast<const uint32_t *>(grp + (size_t)c * kOneHotCellBytes);
            uint32_t v[5];
#pragma unroll
            for (int t = 0; t < 5; t++) v[t] = __ldcs(cell + 32 * t + lane);
            const int cls = (int)(v[0] >> 24) | (int)(((v[1] >> 24) & 1u) << 8);
            const float g = ((v[1] >> 25) & 1u) ? pr.gain1 : pr.gain0;
            const float4 lv = __ldg(reinterpret_cast<const float4 *>(p.cls_value + cls * 8));
            const float l4 = __ldg(p.cls_value + cls * 8 + 4);
            const float val[5] = {lv.x, lv.y, lv.z, lv.w, l4};
            acc = fmaf(g, onehot_dot(v, val, xs + 24 * c), acc);
        }
        deliver(p, pr, group, chunk, lane, acc);
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
    const size_t xbytes = (size_t)nb * 48;
    return layout == LLVQ_PLANES ? (size_t)nprob * 1024 * sizeof(BlockConst) + xbytes : xbytes;
}

int gemv_configure(const llvq_ctx *ctx) {
    const int bytes = ctx->max_smem_optin;
    if (cudaFuncSetAttribute(gemv_planes_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return -1;
    if (cudaFuncSetAttribute(gemv_planes_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return -1;
    if (cudaFuncSetAttribute(gemv_onehot_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return -1;
    return 0;
}

cudaError_t launch_gemv(const llvq_ctx *ctx, int layout, const GemvParams &p, bool no_weights, cudaStream_t s) {
    const size_t smem = gemv_smem_bytes(layout, p.nb, p.nprob);
    int grid = ctx->sm_count;
    const int needed = (p.total_items + kWarps - 1) / kWarps;
    if (grid > needed) grid = needed;
    if (grid < 1) grid = 1;
    if (layout == LLVQ_PLANES) {
        if (no_weights) gemv_planes_kernel<true><<<grid, kThreads, smem, s>>>(p);
        else gemv_planes_kernel<false><<<grid, kThreads, smem, s>>>(p);
    } else {
        gemv_onehot_kernel<<<grid, kThreads, smem, s>>>(p);
    }
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
