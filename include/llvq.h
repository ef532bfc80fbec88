/*
 * llvq.h - C ABI of the B200 (sm_100a) library for the batch-1 fused dequantize-plus-matvec over
 * weights quantised to the multi-shell Leech-lattice codebook Lambda24(12).
 *
 * The path (paper sections in brackets):
 *   llvq_expand      [Sec. 2.2 "Unfolding at load time"]  48-bit block codes -> in-memory records
 *   llvq_gemv        [Sec. 2.3 "The kernel"]               records, row scales, x -> y
 *   llvq_overlay_count, llvq_overlay_bytes [Sec. 3.3, the sparse overlay] size the exception table of LLVQ_PLANES10X
 *   llvq_gemv_grouped[Sec. 3.4 "Attribution": row-concatenated q/k/v and gate/up launches]
 *   llvq_gemv_batch  [Sec. 5 "Batching"]                  the same for 2..8 activation vectors a pass
 *   llvq_gemv_static                                      llvq_gemv without a context or any allocation
 *   llvq_rotate      [Sec. 2.3, Sec. 5 "The rotated basis"] Walsh-Hadamard rotation of x ahead of a projection
 *   llvq_gemv_rotated                                     the same rotation inside the GEMV's own launch
 *   llvq_gemv_fp16, llvq_gemv_noweights [Sec. 3.2, Table "layout scale": the FP16 control and the
 *                    no-weights control that prices the launch geometry]
 *   llvq_dequant_fp16, llvq_decode_i8: helpers that feed the FP16 arm and the bit-exact decode check.
 *
 * Conventions.
 *   - A block is 24 consecutive weights of one row.  A matrix has `rows` rows and `nb` blocks a
 *     row; k_padded = 24 * nb.  x has k_padded entries; the caller zero-fills the padding.
 *   - A code word is a uint64: bits 0..46 the index into the ball (valid below
 *     111 043 117 458 000), bit 47 the gain bit, bits 48..63 zero  [Sec. 2.1].
 *   - Every pointer is a DEVICE pointer owned by the caller unless it says "host".  The library
 *     allocates only what a context owns (its tables and its reduction scratch) at llvq_create.
 *   - Every call takes the caller's CUDA stream (a cudaStream_t passed as void*), enqueues its
 *     work there and returns without synchronising, unless stated otherwise.
 *   - A context holds reduction scratch that its GEMV launches share: launches on one context
 *     must be ordered on one stream (or otherwise serialised).  Use one context per stream.
 *   - Return value: 0 on success, a negative LLVQ_E* code otherwise.  No call aborts, throws or
 *     traps; a failed call enqueues nothing.
 *
 * Layouts (all written by llvq_expand, read by the GEMV; rows are taken 32 at a time, a "row
 * group", rows past the end are filled with the empty record, class id 511):
 *   LLVQ_PLANES  14 bytes a block [Sec. 3.2 "Planes14": class id 9 b, gain 1 b, sign mask 24 b,
 *                three binary planes of the per-coordinate level 3 x 24 b = 106 bits in 112].
 *                The class fixes the parity of every coordinate, so sign and level (|x_i| >> 1) of a
 *                coordinate are stored as one four-bit code u_i = 8 + floor(x_i / 2): x_i = 2 (u_i - 8)
 *                + parity.  Per block a 16-bit header = class | gain << 9 and 24 codes; the empty
 *                record has u_i = 8.  The codes are laid out as the operand fragments of the integer
 *                tensor-core instruction the GEMV uses (16 rows x 32 or 16 positions, a byte each once
 *                the nibbles are split):
 *                  row of a group r = 16 m + 8 e + g (m, e in {0,1}, g in 0..7); lane L = 4 g + t.
 *                  A half-step is 16 rows (one m) of two block slots, 48 positions k: k < 24 is
 *                  coordinate k of slot 0, else coordinate k - 24 of slot 1.  Lane L owns three words;
 *                  nibble n = 2 i + c (i = 0..3, c = 0..1) of a word is bits 4n..4n+3:
 *                    Wa: code of row (m, e=0, g) at position 16 c + 4 t + i
 *                    Wb: code of row (m, e=1, g) at position 16 c + 4 t + i
 *                    Wc: code of row (m, e=c, g) at position 32 + 4 t + i
 *                  and lane pair P = 2 g + (t >> 1) owns one header word:
 *                    header(row (m,0,g), slot t >> 1) | header(row (m,1,g), slot t >> 1) << 16.
 *                  Tile = blocks 4T..4T+3 of a row group, 1792 bytes: half-step h = 2 s + m has slots
 *                  4T+2s, 4T+2s+1; word w = 3 h + (0 Wa, 1 Wb, 2 Wc) of lane L at byte
 *                  512 (w >> 2) + 16 L + 4 (w & 3); header word h of pair P at 1536 + 16 P + 4 h.
 *                  The nb mod 4 blocks left over follow the tiles: if two or three, first a pair
 *                  (896 bytes; half-steps m = 0,1 with the next two blocks as slots; word
 *                  w = 3 m + (0,1,2) of lane L at 128 w + 4 L; header word m of pair P at
 *                  768 + 8 P + 4 m); if one or three, last a single (448 bytes; one half-step whose
 *                  slot s is rows 16 s..16 s+15 of the last block, i.e. "row (m,e,g), slot s" above
 *                  reads row (s,e,g); word w of lane L at 128 w + 4 L; header word of pair P at
 *                  384 + 4 P).  A row group takes 448*nb bytes.
 *   LLVQ_ONEHOT  20 bytes a block [Sec. 3.2 "Slot32": class id, gain, sign mask, one 24-bit
 *                one-hot mask per non-zero level].  Level = rank of |x_i| among the class's
 *                distinct magnitudes.  Per cell five arrays of 32 words (word t of row l at
 *                128t+4l): V0 = smask | class[7:0]<<24, V1 = mask1 | class[8]<<24 | gain<<25,
 *                V2..V4 = mask2..mask4.  A row group takes 640*nb bytes.
 *   LLVQ_PLANES13 13 bytes a block, exact for every block.  Not the paper's next rate point (its sparse overlay, for
 *                which see LLVQ_PLANES10X below): no short record, no exception table.
 *                Here the rate comes from the header instead of the levels: the matvec needs of the
 *                class only what fixes the block's scale and the parity of its coordinates, so the
 *                16-bit header becomes one byte = shell (4 bits, 0 for the empty record) | parity << 4
 *                | gain << 5, and the 24 four-bit codes stay as they are - no level cap, no exception
 *                table, no second stream.  The code words sit where LLVQ_PLANES has them; the header
 *                bytes follow them: tile 1664 bytes, byte of pair P, half-step h, row half e at
 *                1536 + 8 P + 2 h + e; pair 832 bytes, byte at 768 + 4 P + 2 m + e; single 416 bytes,
 *                byte at 384 + 2 P + e.  A row group takes 416*nb bytes.
 *                Accepted by llvq_layout_bytes, llvq_expand, llvq_gemv, llvq_gemv_grouped and
 *                llvq_decode_i8 (which returns the header byte in place of a class id); the other
 *                calls return LLVQ_EINVAL for it.  y is bit for bit what LLVQ_PLANES gives.
 *   LLVQ_PLANES10X 10 bytes a block plus a sparse table of exact records: this library's form of the paper's
 *                "Planes12x" overlay [Sec. 3.3: a short record for most blocks, the exact record of the others in
 *                a per-matrix exception table, the correction applied in the same launch, reconstruction
 *                bit-exact].  The paper's short record keeps a two-bit level and a sign a coordinate, which a
 *                class table turns into a value; the tensor-core contraction used here wants a code the value
 *                is affine in, so the short record keeps a three-bit WINDOW code instead, and the header
 *                byte of LLVQ_PLANES13 in place of the class:
 *                  v_i = u_i - o, u_i the four-bit code of LLVQ_PLANES, o the block's window base: the
 *                  smallest o in {3, 4, 5, 6} with o <= min u_i and max u_i <= o + 7;
 *                  header byte = (f ^ shell) | shell << 4 with f = (o - 3) | parity << 2 | gain << 3;
 *                  x_i = 2 (v_i + o - 8) + parity.  (The byte indexes a table in shared memory whose bank is
 *                  chosen by the low four bits: with the shell mixed into them, the headers that occur
 *                  together in a tile - a few shells, either parity, either gain - fall into different banks.)
 *                A block with no such o (its codes span more than eight consecutive values, or reach below 3)
 *                is an EXCEPTION: its short record is all zero - the empty record, which adds nothing - and
 *                its exact record goes to the table.  Rows past the end and codes that name no point also
 *                get the all-zero record (and no table entry).
 *                  Tile = blocks 4T..4T+3 of a row group, 1280 bytes; rows, lanes, half-steps and positions
 *                  as in LLVQ_PLANES.  Group(h, e, c) of lane L = 4g + t is the four codes of row (m, e, g)
 *                  of half-step h = 2s + m at positions 16c + 4t + i (c = 0, 1) or 32 + 4t + i (c = 2),
 *                  i = 0..3.  The lane owns nine words V0..V8; byte i of a word carries code i of two
 *                  groups, in bits 0..2 and 3..5:
 *                    V(2h + e), h = 0..3, e = 0, 1:  Group(h, e, 0), Group(h, e, 1)
 *                    V8:                             Group(0, 0, 2), Group(1, 0, 2)
 *                  and bits 6, 7 of the bytes carry the six groups left, X0..X5 = Group(0, 1, 2),
 *                  Group(1, 1, 2), Group(2, 0, 2), Group(2, 1, 2), Group(3, 0, 2), Group(3, 1, 2): bits
 *                  0, 1 of code i of Xk are bits 6, 7 of byte i of Vk; bit 2 of code i of Xk is bit
 *                  6 + (k & 1) of byte i of V(6 + (k >> 1)).
 *                  Vk of lane L at byte 16 L + 4 k (k < 4), 512 + 16 L + 4 (k - 4) (k < 8), 1024 + 4 L
 *                  (k = 8); header byte of pair P, half-step h, row half e at 1152 + 8 P + 2 h + e.
 *                  The nb mod 4 blocks left over follow the tiles exactly as in LLVQ_PLANES13 (four-bit
 *                  codes, that layout's header byte: a pair of 832 bytes, a single of 416): they
 *                  hold every block exactly and never make an exception.  A row group takes
 *                  1280 (nb / 4) + 416 (nb mod 4) bytes.
 *                  After the last row group, at the next multiple of 128 bytes: the index, one uint32 a
 *                  tile (row group by row group, nb / 4 tiles each) and one more - entry i = table entries
 *                  of the tiles before tile i.  After the index, at the next multiple of 128 bytes: the
 *                  table, 16 bytes an entry, ordered by row group, tile, block, row:  word 0 = shell | parity << 4 | gain << 5 | (row of the
 *                  group) << 8 | (block column) << 13;  words 1..3 = the 24 four-bit codes, coordinate
 *                  8 j + n in nibble n of word 1 + j.  Bytes between the parts are zero.
 *                The table's size depends on the data: llvq_overlay_count counts the exceptions of a matrix,
 *                llvq_overlay_bytes sizes the buffer for a given number, llvq_layout_bytes sizes it for one
 *                exception in 32 blocks.  llvq_expand takes the room for entries from out_bytes; entries that
 *                do not fit are dropped, the index stops at the capacity, and the next llvq_status returns
 *                LLVQ_ESIZE.  k_padded / 24 must be below 2^19.
 *                Accepted by the calls that accept LLVQ_PLANES13.  y is reproducible (the same bits for the
 *                same buffer whatever the launch) and agrees with LLVQ_PLANES to within a few accumulator
 *                quanta a tile, not bit for bit: a block's integer sum is the same, but its two halves (low
 *                and high limbs of x) split differently for a shifted code before each is rounded to f32, and
 *                an exception's product is rounded to the quantum by itself instead of with its tile's.
 */
#ifndef LLVQ_H
#define LLVQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LLVQ_PLANES 0
#define LLVQ_ONEHOT 1
#define LLVQ_PLANES13 2   /* no counterpart record in the paper: see above */
#define LLVQ_PLANES10X 3  /* the paper's sparse overlay ("Planes12x") with a window code: see above */

#define LLVQ_OK 0
#define LLVQ_EINVAL (-1) /* null pointer, bad shape, unknown layout                         */
#define LLVQ_EALIGN (-2) /* a device pointer is not aligned as documented                   */
#define LLVQ_ESIZE (-3)  /* a buffer or the context's scratch is too small for the request; from llvq_status:
                            an LLVQ_PLANES10X expansion had more exceptions than its buffer had room for */
#define LLVQ_ECUDA (-4)  /* a CUDA runtime call failed                                      */
#define LLVQ_ETIMEOUT (-5) /* a bounded wait inside a kernel ran out (llvq_status, llvq_static_status) */
#define LLVQ_EINDEX (-6) /* an expanded code word named no point of the ball (llvq_status only) */

#define LLVQ_MAX_GROUP 8       /* matrices in one grouped launch                             */
#define LLVQ_MAX_K 98304       /* largest k_padded the GEMV accepts                          */
#define LLVQ_MAX_BATCH 8       /* activation vectors in one llvq_gemv_batch call             */

typedef struct llvq_ctx llvq_ctx;

/* One matrix of a grouped launch: its records, fp16 row scales, two gain centroids, output. */
typedef struct {
    const void *layout;     /* device, 128-byte aligned                                      */
    const void *row_scale;  /* device, fp16[rows]                                            */
    float *y;               /* device, f32[rows]                                             */
    int64_t rows;
    float gain[2];          /* centroid chosen by each block's gain bit [Sec. 2.1]           */
} llvq_problem;

/* The rotation of x that llvq_gemv_rotated applies (the arguments of llvq_rotate). */
typedef struct llvq_rotation {
    const uint32_t *negate_bits; /* device, may be null: bit i & 31 of word i >> 5 set = x_i negated first */
    int64_t n;                   /* entries of x that are rotated: a multiple of the block length, <= k_padded;
                                    the entries after them (the zero padding) pass through */
    int64_t block;               /* block length, a power of two in 8..16384 that divides n; 0 = the largest */
} llvq_rotation;

/* Builds the class, index-base and Golay tables on the host, uploads them to `device`, and
 * allocates the context's reduction scratch (scratch_bytes; 0 = default 8 MiB, eight bytes a row
 * of the largest launch, rows rounded up to 32 per matrix).  Synchronous.  (The third argument is
 * this library's addition to the call the paper's statement of the problem implies: the scratch is
 * the one thing whose size depends on the caller's largest launch.) */
int llvq_create(llvq_ctx **out, int device, size_t scratch_bytes);
void llvq_destroy(llvq_ctx *ctx);
const char *llvq_strerror(int code);

/* Synchronises `stream` and reports whether any GEMV launched on this context since the last
 * call gave up on one of its bounded waits (LLVQ_ETIMEOUT; the flag and the scratch are then
 * reset), else whether an LLVQ_PLANES10X expansion ran out of room for its exception table (LLVQ_ESIZE;
 * expand again into a larger buffer), else whether any llvq_expand on this context since the last call met a code word that
 * names no point (LLVQ_EINDEX; the count is then reset - the 512-slot class table exists so that
 * such a code can never index out of bounds [Sec. 2.3], and this is how a caller that passed no
 * bad_count learns of it).  Every wait inside the kernels on an asynchronous copy has a time limit
 * of about a second; none can spin forever, and none traps. */
int llvq_status(llvq_ctx *ctx, void *stream);

/* Enqueues a one-warp kernel that waits, with a limit of about a millisecond, on a barrier nothing
 * completes, and then raises the context's error flag exactly as a GEMV whose copy never arrived
 * would: the next llvq_status returns LLVQ_ETIMEOUT, the one after LLVQ_OK.  Lets a caller (and the
 * tests) check the failure path without any fault on the GPU. */
int llvq_selftest_wait_limit(llvq_ctx *ctx, void *stream);

/* The GEMV is launched with programmatic dependent launch (on by default): its record prefetch
 * starts while the previous kernel of the stream drains, and it waits for that kernel before it
 * touches x, y or the scratch.  What it reads AHEAD of that wait are the caller's weights: the layout
 * buffer, the row scales and a rotation's negate_bits.  They must therefore be complete before the
 * kernel that precedes the GEMV on the stream starts (weights loaded once satisfy this trivially);
 * llvq_expand takes care of it by itself (the next GEMV on the context is launched as an ordinary
 * kernel); a caller whose own kernel writes scales or records right before a GEMV disables the
 * feature.  enabled = 0 launches every GEMV as an ordinary kernel. */
int llvq_set_pdl(llvq_ctx *ctx, int enabled);

/* Host queries.  Number of classes (301), points in the ball, and first index of class c
 * (c = 301 gives the number of points)  [Sec. 2.1]. */
int llvq_num_classes(const llvq_ctx *ctx);
uint64_t llvq_class_base(const llvq_ctx *ctx, int c);

/* Bytes of a layout buffer for a rows x (k_padded/24) matrix. Host query. */
int llvq_layout_bytes(int layout, int64_t rows, int64_t k_padded, size_t *bytes);

/* [Sec. 3.3, the exception table of the sparse overlay] Host queries and a counting pass for LLVQ_PLANES10X.
 * llvq_overlay_count decodes the rows*nb code words and writes to *count (HOST) how many blocks the layout keeps
 * in its exception table; it synchronises `stream`.  llvq_overlay_bytes gives the bytes of a layout buffer with
 * room for `exceptions` table entries. */
int llvq_overlay_count(llvq_ctx *ctx, const uint64_t *codes, int64_t rows, int64_t nb, uint64_t *count, void *stream);
int llvq_overlay_bytes(int64_t rows, int64_t k_padded, uint64_t exceptions, size_t *bytes);

/* [Sec. 2.2] Unfolds rows*nb code words (row-major, codes[row*nb + b]) into `layout_out`
 * (128-byte aligned, at least llvq_layout_bytes).  A code that names no point (index not below
 * the number of points, or bits above bit 47 set) becomes the empty record (class 511, all
 * fields zero) and, if bad_count is not null, adds one to *bad_count (device uint32, which the
 * caller zeroes).  The context counts such codes as well, whether or not bad_count is given: the next
 * llvq_status returns LLVQ_EINDEX if any expansion since the last one met one.  Bit-exact by construction:
 * integer arithmetic only.  The GEMV enqueued next on this context is launched without programmatic dependent
 * launch, so that it cannot read records ahead of this expansion (see llvq_set_pdl). */
int llvq_expand(llvq_ctx *ctx, int layout, const uint64_t *codes, int64_t rows, int64_t nb,
                void *layout_out, size_t out_bytes, uint32_t *bad_count, void *stream);

/* [Sec. 2.3] y[row] = row_scale[row] * sum_b gain[g_b] / (4 sqrt(m_b)) * sum_i x_b,i * x[24b+i],
 * m_b the shell of block b's class.  gain is a HOST pointer to two floats; the larger of their magnitudes
 * must be zero or lie in [2^-60, 2^60) (LLVQ_EINVAL otherwise: the fixed-point quantum is a power of two
 * formed from its exponent).  x is fp16, 16-byte
 * aligned; y is f32; x must be finite.  LLVQ_PLANES: x is taken as fixed point on a scale set by
 * the largest |x| (X_i = rint(x_i 2^F), |X_i| < 2^29; exact for every x_i within 2^-18 of the
 * largest, rounded to within 2^-29 of the largest below that), the inner sums over a block are integer and
 * exact, the per-block scale is applied in f32.  LLVQ_ONEHOT: f32 products and sums.  Either way a
 * row is summed in pieces of at most four blocks whose bounds depend on nb alone; the pieces meet
 * in a fixed-point accumulator (integer addition, exact and order-free, finer than f32), so the
 * result never depends on the launch geometry and a grouped launch returns bit-identical rows. */
int llvq_gemv(llvq_ctx *ctx, int layout, const void *layout_buf, const void *row_scale,
              const float *gain, const void *x, float *y, int64_t rows, int64_t k_padded, void *stream);

/* [Sec. 5 "Batching", the paper's stated boundary: one record decode reused across activations]
 * llvq_gemv on the LLVQ_PLANES layout for batch (1..LLVQ_MAX_BATCH) activation vectors in one pass
 * over the records: x is fp16 [batch][k_padded], y is f32 [batch][rows].  Up to four vectors share
 * one pass (the records are read and decoded once for them); five to eight take two passes.  Each
 * vector has its own fixed-point scale and its own accumulators, and y[j] is bit-identical to what
 * llvq_gemv returns for x[j].  Needs min(batch, 4) times the scratch of llvq_gemv (LLVQ_ESIZE
 * otherwise). */
int llvq_gemv_batch(llvq_ctx *ctx, const void *layout_buf, const void *row_scale, const float *gain,
                    const void *x, float *y, int64_t rows, int64_t k_padded, int batch, void *stream);

/* Host query and test hook (no GPU needed): the launch plan llvq_gemv / llvq_gemv_grouped / llvq_gemv_batch
 * (batch <= 4: one pass) would use on a device with sm_count multiprocessors for n matrices of rows[i] rows.
 * out (host, out_len >= 8 + grid + 1 int32): grid, dynamic shared memory bytes, units a row group (tiles of
 * four blocks, plus one for leftover blocks), total units, unit columns a panel, panels, most blocks of x a
 * CTA prepares, row groups; then the first unit of every CTA and the total. */
int llvq_gemv_plan(int sm_count, const int64_t *rows, int n, int64_t k_padded, int batch, int32_t *out, int out_len);

/* [Sec. 3.4] One launch over n <= LLVQ_MAX_GROUP row-concatenated matrices that share x and
 * k_padded (q/k/v, gate/up).  `problems` is a HOST array, copied before the call returns. */
int llvq_gemv_grouped(llvq_ctx *ctx, int layout, const llvq_problem *problems, int n,
                      const void *x, int64_t k_padded, void *stream);

/* [Sec. 2.3 and Sec. 5, the rotated basis] llvq_gemv_grouped(LLVQ_PLANES) on the rotated activation, in one
 * launch: y = W * rotate(x).  The paper runs the rotation as a kernel of its own ahead of every projection,
 * one thread block holding the whole activation; here every CTA of the GEMV rotates, in its prologue, the
 * rotation blocks that meet its part of x, with llvq_rotate's arithmetic: the values that enter the matvec are
 * bit for bit the FP16 values llvq_rotate(x, rotation->n, rotation->block, rotation->negate_bits) would store,
 * so y agrees with llvq_rotate followed by llvq_gemv_grouped to within the GEMV's fixed-point quantum (the
 * scale of that quantum comes from ||x||_2, which bounds every rotated entry, instead of from the largest
 * entry).  x itself is not modified.  The blocks a CTA rotates must fit its shared memory beside the GEMV's
 * own: block lengths up to 4096 always do; a longer block may return LLVQ_ESIZE (rotate with llvq_rotate then).
 * Errors: those of llvq_gemv_grouped; LLVQ_EINVAL also for a null rotation, n not a positive multiple of 8
 * or above k_padded, a block that is not acceptable or shorter than 8. */
int llvq_gemv_rotated(llvq_ctx *ctx, const llvq_problem *problems, int n, const void *x, int64_t k_padded,
                      const llvq_rotation *rotation, void *stream);

/* No counterpart in the paper: the LLVQ_PLANES llvq_gemv for callers that cannot allocate device
 * memory - a process whose memory pool already owns the whole GPU, a plug-in that receives buffers
 * but no allocator, code that runs while a stream is being captured, a loop that cannot afford the
 * device synchronisation an allocation implies.  Such callers cannot use a context either
 * (llvq_create allocates), so this call takes none: the reduction scratch and the error flag are
 * file-scope device arrays inside the library (about 512 KiB on every GPU that loads it, held
 * until the process exits).  Same arguments, layout (LLVQ_PLANES only), alignment rules and
 * results as llvq_gemv; it runs on the CURRENT device.  Limits and rules:
 *   - rows, rounded up to a multiple of 32, must not exceed 65536 (the built-in scratch holds one
 *     64-bit accumulator a row); more returns LLVQ_ESIZE and launches nothing.
 *   - The first call on a device sets the arrays up (resolves their device addresses, zeroes the
 *     scratch - synchronous, no allocation).  Make that first call
 *     before any stream capture begins.
 *   - Every call shares the one scratch array.  A launch that completes leaves it zeroed for the
 *     next; launches that overlap on the GPU (two streams) race on it - serialise them.
 * It calls no cudaMalloc, cudaFree or other allocating routine. */
int llvq_gemv_static(const void *layout_buf, const void *row_scale, const float *gain, const void *x, float *y,
                     int64_t rows, int64_t k_padded, void *stream);

/* llvq_status for llvq_gemv_static (which has no context to ask): synchronises `stream` and reports whether a
 * llvq_gemv_static launch on the CURRENT device gave up on one of its bounded waits since the last call
 * (LLVQ_ETIMEOUT).  The flag and the built-in scratch are then cleared (two memsets, no allocation), so the
 * calls that follow start clean; without this call such a time-out would go unseen and leave partial sums in
 * the shared scratch.  llvq_static_selftest_wait_limit enqueues the one-warp kernel of
 * llvq_selftest_wait_limit against that flag: the next llvq_static_status returns LLVQ_ETIMEOUT, the one after
 * LLVQ_OK. */
int llvq_static_status(void *stream);
int llvq_static_selftest_wait_limit(void *stream);

/* [Table "layout scale", FP16 control] y = W x, W fp16 row-major rows x k (k a multiple of 8,
 * W and x 16-byte aligned), f32 accumulation, f32 y. */
int llvq_gemv_fp16(const void *W, const void *x, float *y, int64_t rows, int64_t k, void *stream);

/* [Table "layout scale", no-weights control] The launch llvq_gemv(LLVQ_PLANES) would make - same
 * grid, shared memory, x staging, reduction and epilogue - with no record read; y = 0. */
int llvq_gemv_noweights(llvq_ctx *ctx, const void *row_scale, const void *x, float *y,
                        int64_t rows, int64_t k_padded, void *stream);

/* [Sec. 2.3: the activation is rotated by a kernel of its own ahead of the matvec; Sec. 5, the
 * paragraph on the rotated basis: a Walsh-Hadamard transform, which every consumer of the stored
 * weights applies.]  y = rotation of x, both fp16 vectors of n entries (n a multiple of 8, both
 * 16-byte aligned; y may be x):
 *     y[B c + k] = (1 / sqrt(B)) * sum_{i < B} (-1)^popcount(i & k) * s_i * x[B c + i],
 * the natural-order (Sylvester) Hadamard matrix on each block of B consecutive coordinates.
 *   - block: B, a power of two <= 16384 that divides n; 0 = the largest such power of two
 *     (512 for n = 2560 or 9728, 4096 for n = 4096 or 12288, 1024 for n = 17408 or 25600).
 *     The paper names the transform only: the block-diagonal form for lengths that are not powers
 *     of two, the order and the scale are this library's reading.
 *   - negate_bits: optional (may be null).  Bit i & 31 of word i >> 5 set = s_i = -1, the sign
 *     flip of a randomised rotation; ceil(n / 32) words, 4-byte aligned.  Null = no flips.
 *   - Arithmetic: the sums are exact (64-bit integers in units of 2^-24); the result is scaled in
 *     f64 and rounded once to fp16, to nearest even.  While a block's sum of |x| is below 2^29 the
 *     output is the correctly rounded value of the formula, bit for bit whatever the launch.
 *     x must be finite.  A value beyond the fp16 range rounds to infinity.
 *   - The launch is a link of the same programmatic-dependent-launch chain as the GEMV
 *     (llvq_set_pdl): the GEMV enqueued after it on the stream sets up while it runs.
 * Errors: LLVQ_EINVAL (null pointer, n <= 0 or not a multiple of 8, block not acceptable),
 * LLVQ_EALIGN, LLVQ_ESIZE (n > 2^40), LLVQ_ECUDA. */
int llvq_rotate(llvq_ctx *ctx, const void *x, void *y, const uint32_t *negate_bits, int64_t n,
                int64_t block, void *stream);

/* Host query: the block length llvq_rotate uses for (n, block); 0 if it would refuse them. */
int64_t llvq_rotate_block(int64_t n, int64_t block);

/* Decoded weights as fp16, W[row*k_padded + 24b + i] = fp16(row_scale * gain[g] * x_i / (4 sqrt m))
 * (product formed in f32, rounded once).  Feeds llvq_gemv_fp16. */
int llvq_dequant_fp16(llvq_ctx *ctx, int layout, const void *layout_buf, const void *row_scale,
                      const float *gain, void *W, int64_t rows, int64_t k_padded, void *stream);

/* Test hook: the integer coordinates (coords[(row*nb + b)*24 + i]) and class id
 * (class_ids[row*nb + b]) a layout buffer decodes to, for the bit-exact check of Sec. 2.4.
 * LLVQ_PLANES13 keeps no class id: class_ids receives the header byte (shell | parity << 4 | gain << 5). */
int llvq_decode_i8(llvq_ctx *ctx, int layout, const void *layout_buf, int8_t *coords,
                   uint16_t *class_ids, int64_t rows, int64_t nb, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LLVQ_H */
