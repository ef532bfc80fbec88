/*
 * CPU oracle for the multi-shell Leech-lattice (Lambda24(12)) index decode, the unfolded
 * records and the f64 dequantize-plus-matvec.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA library is
 * checked against.  It shares no code, table or header with the CUDA path, and nothing in
 * the product may call it: only the tests, the smoke check and the benchmark's CPU-baseline
 * leg do.
 *
 * What it follows (paper sections):
 *   Sec. 2.1  "What a Lambda24 index is": the ball Lambda24(12) in sqrt(8)*Lambda24 < Z^24,
 *             its three membership conditions, the 301 classes, the 47-bit index that lists
 *             classes first and arrangements and signs inside a class, the gain bit.
 *   Sec. 2.2  "Unfolding at load time": the decoded-field record (class id, gain bit,
 *             sign mask, per-coordinate magnitude level as bit planes or one-hot masks).
 *   Sec. 2.3  "The kernel": y[row] = r_row * sum over blocks of the decoded unit
 *             direction times the gain centroid, dotted with x (here in f64).
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   - Golay code: extended cyclic code, generator polynomial 0xC75 on coordinates 0..22,
 *     coordinate 23 is the overall parity bit; bit i of a word is coordinate i.
 *   - Class order: shell ascending; even type before odd type; Golay weight ascending;
 *     then the sorted magnitude tuples compared lexicographically (support part first).
 *   - Order inside a class: mixed radix, codeword rank most significant, then the
 *     arrangement rank on the support, the arrangement rank off the support, signs least
 *     significant (even type); arrangement rank times 4096 plus the 12 message bits of the
 *     codeword (odd type).
 *   - Bit-plane level of a coordinate = |x_i| >> 1 (the class fixes the parity of every
 *     magnitude, so |x_i| = 2*level + parity).  One-hot level = rank of |x_i| among the
 *     distinct magnitudes of the class, ascending; masks exist for ranks 1..4.
 *
 * Parity pins (tests/test_oracle_pins.py): Golay weight enumerator and self-duality, 301
 * classes, the total N = 111 043 117 458 000, the count through shell 13, per-shell counts
 * against the Leech theta series, membership of every decoded point by a test written
 * separately in Python, exhaustive injectivity on shell 2, encode/decode round trips, worked
 * index -> point examples, unit norm of every block direction, and textbook special cases
 * of the matvec.  Literal equality with the paper's own on-disk numbering: parity unpinned
 * (the paper prints neither its order nor its fingerprint).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define NCOORD 24
#define MAX_CLASSES 1024
#define MAX_SHELL_LIMIT 13

/* ------------------------------------------------------------------------------------ */
/* Extended binary Golay code (Sec. 2.1 cites it through the lattice's definition).       */
/* ------------------------------------------------------------------------------------ */

static uint32_t g_row[12];        /* generator rows                                      */
static uint32_t g_word[4096];     /* word for message k = XOR of rows selected by k's bits */
static uint32_t g_sorted[4096];   /* all words, ascending as integers                      */
static int g_nw[25];              /* number of words of each weight                        */
static uint32_t *g_byw[25];       /* words of one weight, ascending as integers            */

static int popcount32(uint32_t v) { int n = 0; while (v) { v &= v - 1; n++; } return n; }

static int cmp_u32(const void *a, const void *b) {
    uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return (x > y) - (x < y);
}

static void golay_build(void) {
    const uint32_t poly = 0xC75u; /* x^11+x^10+x^6+x^5+x^4+x^2+1 */
    for (int i = 0; i < 12; i++) {
        uint32_t w = poly << i;                       /* cyclic shift stays inside 23 bits */
        if (popcount32(w) & 1) w |= 1u << 23;         /* overall parity on coordinate 23   */
        g_row[i] = w;
    }
    memset(g_nw, 0, sizeof g_nw);
    for (int k = 0; k < 4096; k++) {
        uint32_t w = 0;
        for (int i = 0; i < 12; i++) if ((k >> i) & 1) w ^= g_row[i];
        g_word[k] = w;
        g_sorted[k] = w;
        g_nw[popcount32(w)]++;
    }
    qsort(g_sorted, 4096, sizeof(uint32_t), cmp_u32);
    for (int w = 0; w <= 24; w++) {
        free(g_byw[w]);
        g_byw[w] = NULL;
        if (!g_nw[w]) continue;
        g_byw[w] = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)g_nw[w]);
        int n = 0;
        for (int k = 0; k < 4096; k++) if (popcount32(g_sorted[k]) == w) g_byw[w][n++] = g_sorted[k];
    }
}

static int golay_contains(uint32_t w) {
    return bsearch(&w, g_sorted, 4096, sizeof(uint32_t), cmp_u32) != NULL;
}

/* ------------------------------------------------------------------------------------ */
/* Classes (Sec. 2.1: orbits fixed by a codeword weight, a magnitude multiset, a coset).  */
/* ------------------------------------------------------------------------------------ */

typedef struct {
    int shell;            /* m: sum of squares = 16 m                                     */
    int odd;              /* 0: all coordinates even, 1: all odd                          */
    int w;                /* Golay weight of the support (even type); 0 for odd type      */
    int mags[NCOORD];     /* even: sorted support magnitudes (w of them) then sorted
                             off-support magnitudes; odd: the 24 sorted magnitudes        */
    uint64_t permA, permB;/* distinct arrangements of each part (odd: permA, permB = 1)   */
    int nzB;              /* non-zero off-support entries (even type)                     */
    uint64_t size, base;  /* points in the class, index of its first point               */
    int ndist;            /* number of distinct magnitudes                                */
    int dist[8];          /* the distinct magnitudes, ascending                           */
} cls_t;

static cls_t g_cls[MAX_CLASSES];
static int g_ncls = 0;
static uint64_t g_total = 0;
static int g_maxshell = 0;
static uint64_t g_shell_count[MAX_SHELL_LIMIT + 1];

/* number of distinct orderings of a sorted multiset a[0..n) */
static uint64_t multiset_perms(const int *a, int n) {
    /* product of binomials: choose the places of each run among what is left */
    uint64_t r = 1;
    int left = n, i = 0;
    while (i < n) {
        int j = i;
        while (j < n && a[j] == a[i]) j++;
        int k = j - i;
        /* r *= C(left, k), exact at every step */
        uint64_t c = 1;
        for (int t = 1; t <= k; t++) c = c * (uint64_t)(left - k + t) / (uint64_t)t;
        r *= c;
        left -= k;
        i = j;
    }
    return r;
}

static int cls_cmp(const void *pa, const void *pb) {
    const cls_t *a = (const cls_t *)pa, *b = (const cls_t *)pb;
    if (a->shell != b->shell) return a->shell - b->shell;
    if (a->odd != b->odd) return a->odd - b->odd;
    if (a->w != b->w) return a->w - b->w;
    for (int i = 0; i < NCOORD; i++) if (a->mags[i] != b->mags[i]) return a->mags[i] - b->mags[i];
    return 0;
}

static void cls_finish(cls_t *c) {
    if (c->odd) {
        c->permA = multiset_perms(c->mags, NCOORD);
        c->permB = 1;
        c->nzB = 0;
        c->size = c->permA * 4096u;
    } else {
        c->permA = multiset_perms(c->mags, c->w);
        c->permB = multiset_perms(c->mags + c->w, NCOORD - c->w);
        c->nzB = 0;
        for (int i = c->w; i < NCOORD; i++) if (c->mags[i]) c->nzB++;
        uint64_t signs = (uint64_t)1 << c->nzB;
        if (c->w > 0) signs <<= (c->w - 1);
        c->size = (uint64_t)g_nw[c->w] * c->permA * c->permB * signs;
    }
    int tmp[NCOORD];
    memcpy(tmp, c->mags, sizeof tmp);
    for (int i = 1; i < NCOORD; i++) { /* insertion sort of the whole multiset */
        int v = tmp[i], j = i - 1;
        while (j >= 0 && tmp[j] > v) { tmp[j + 1] = tmp[j]; j--; }
        tmp[j + 1] = v;
    }
    c->ndist = 0;
    for (int i = 0; i < NCOORD; i++)
        if (i == 0 || tmp[i] != tmp[i - 1]) c->dist[c->ndist++] = tmp[i];
}

/* recursive listing of sorted multisets: n entries from vals[vi..nv) with given sum of squares */
typedef void (*emit_fn)(const int *a, int n, void *ctx);

static void multisets_rec(const int *vals, int nv, int vi, int n, int pos, int sq, int *a, emit_fn emit, void *ctx) {
    if (pos == n) { if (sq == 0) emit(a, n, ctx); return; }
    for (int i = vi; i < nv; i++) {
        int v = vals[i], rem = n - pos;
        if (v * v * rem > sq) break;              /* values ascend: all later are too large */
        a[pos] = v;
        multisets_rec(vals, nv, i, n, pos + 1, sq - v * v, a, emit, ctx);
    }
}

typedef struct { int shell, w, sqA; const int *valsB; int nvB; int a[NCOORD]; } even_ctx;

static void emit_even_B(const int *b, int n, void *vctx) {
    even_ctx *e = (even_ctx *)vctx;
    if (e->w == 0) { /* no support: the sum condition falls on the multiset itself */
        int s = 0;
        for (int i = 0; i < n; i++) s += b[i];
        if (s % 8) return;
    }
    cls_t *c = &g_cls[g_ncls++];
    memset(c, 0, sizeof *c);
    c->shell = e->shell; c->odd = 0; c->w = e->w;
    memcpy(c->mags, e->a, sizeof(int) * (size_t)e->w);
    memcpy(c->mags + e->w, b, sizeof(int) * (size_t)n);
}

static void emit_even_A(const int *a, int n, void *vctx) {
    even_ctx *e = (even_ctx *)vctx;
    memcpy(e->a, a, sizeof(int) * (size_t)n);
    int sqA = 0;
    for (int i = 0; i < n; i++) sqA += a[i] * a[i];
    int b[NCOORD] = {0};
    multisets_rec(e->valsB, e->nvB, 0, NCOORD - e->w, 0, 16 * e->shell - sqA, b, emit_even_B, e);
}

typedef struct { int shell; } odd_ctx;

static void emit_odd(const int *a, int n, void *vctx) {
    odd_ctx *o = (odd_ctx *)vctx;
    /* with the zero codeword every coordinate is congruent to 1 mod 4: +a if a = 1 mod 4, else -a */
    int s = 0;
    for (int i = 0; i < n; i++) s += (a[i] % 4 == 1) ? a[i] : -a[i];
    if (((s % 8) + 8) % 8 != 4) return;
    cls_t *c = &g_cls[g_ncls++];
    memset(c, 0, sizeof *c);
    c->shell = o->shell; c->odd = 1; c->w = 0;
    memcpy(c->mags, a, sizeof(int) * (size_t)n);
}

/* Build the class list for shells 2..max_shell. Returns the number of classes. */
int llvqo_init_shells(int max_shell) {
    if (max_shell < 2 || max_shell > MAX_SHELL_LIMIT) return -1;
    golay_build();
    g_ncls = 0;
    static const int valsA[] = {2, 6, 10, 14};       /* support: congruent to 2 mod 4 */
    static const int valsB[] = {0, 4, 8, 12};        /* off support: multiples of 4    */
    static const int valsM[] = {1, 3, 5, 7, 9, 11, 13};
    static const int weights[] = {0, 8, 12, 16, 24};
    for (int m = 2; m <= max_shell; m++) {
        for (int wi = 0; wi < 5; wi++) {
            even_ctx e;
            e.shell = m; e.w = weights[wi]; e.valsB = valsB; e.nvB = 4;
            int a[NCOORD];
            /* every split of 16 m between the support and the rest */
            for (int sqA = 0; sqA <= 16 * m; sqA += 4) {
                if (e.w == 0 && sqA) break;
                multisets_rec(valsA, 4, 0, e.w, 0, sqA, a, emit_even_A, &e);
            }
        }
        odd_ctx o; o.shell = m;
        int a[NCOORD];
        multisets_rec(valsM, 7, 0, NCOORD, 0, 16 * m, a, emit_odd, &o);
    }
    qsort(g_cls, (size_t)g_ncls, sizeof(cls_t), cls_cmp);
    g_total = 0;
    memset(g_shell_count, 0, sizeof g_shell_count);
    for (int c = 0; c < g_ncls; c++) {
        cls_finish(&g_cls[c]);
        g_cls[c].base = g_total;
        g_total += g_cls[c].size;
        g_shell_count[g_cls[c].shell] += g_cls[c].size;
    }
    g_maxshell = max_shell;
    return g_ncls;
}

int llvqo_init(void) { return llvqo_init_shells(12); }

int llvqo_num_classes(void) { return g_ncls; }
uint64_t llvqo_total_points(void) { return g_total; }
uint64_t llvqo_shell_count(int m) { return (m >= 0 && m <= MAX_SHELL_LIMIT) ? g_shell_count[m] : 0; }

/* out[0..5] = shell, odd, w, ndist, nzB, (unused); mags[24]; size, base */
int llvqo_class_info(int c, int *out, int *mags, uint64_t *size, uint64_t *base) {
    if (c < 0 || c >= g_ncls) return -1;
    const cls_t *k = &g_cls[c];
    out[0] = k->shell; out[1] = k->odd; out[2] = k->w; out[3] = k->ndist; out[4] = k->nzB; out[5] = 0;
    for (int i = 0; i < NCOORD; i++) mags[i] = k->mags[i];
    *size = k->size; *base = k->base;
    return 0;
}

uint32_t llvqo_golay_word(int k) { return g_word[k & 4095]; }
uint32_t llvqo_golay_sorted(int k) { return g_sorted[k & 4095]; }

/* ------------------------------------------------------------------------------------ */
/* Arrangement ranks: lexicographic over the distinct orderings, smaller magnitude first. */
/* ------------------------------------------------------------------------------------ */

/* rank -> sequence. cnt[v] = copies of magnitude v still to place. */
static void unrank_arrangement(uint64_t rank, const int *sorted, int n, int *seq) {
    int cnt[16] = {0};
    for (int i = 0; i < n; i++) cnt[sorted[i]]++;
    uint64_t total = multiset_perms(sorted, n);
    int left = n;
    for (int pos = 0; pos < n; pos++) {
        for (int v = 0; v < 16; v++) {
            if (!cnt[v]) continue;
            /* orderings that put v here: total * cnt[v] / left */
            uint64_t sub = total * (uint64_t)cnt[v] / (uint64_t)left;
            if (rank < sub) { seq[pos] = v; cnt[v]--; total = sub; left--; break; }
            rank -= sub;
        }
    }
}

static uint64_t rank_arrangement(const int *seq, int n) {
    int cnt[16] = {0}, sorted[NCOORD];
    for (int i = 0; i < n; i++) cnt[seq[i]]++;
    int k = 0;
    for (int v = 0; v < 16; v++) for (int j = 0; j < cnt[v]; j++) sorted[k++] = v;
    uint64_t total = multiset_perms(sorted, n), rank = 0;
    int left = n;
    for (int pos = 0; pos < n; pos++) {
        for (int v = 0; v < seq[pos]; v++) {
            if (!cnt[v]) continue;
            rank += total * (uint64_t)cnt[v] / (uint64_t)left;
        }
        int v = seq[pos];
        total = total * (uint64_t)cnt[v] / (uint64_t)left;
        cnt[v]--; left--;
    }
    return rank;
}

/* ------------------------------------------------------------------------------------ */
/* Index -> point (Sec. 2.1: classes first, then arrangements and signs in a fixed order). */
/* ------------------------------------------------------------------------------------ */

static int find_class(uint64_t idx) {
    for (int c = 0; c < g_ncls; c++) if (idx < g_cls[c].base + g_cls[c].size) return c;
    return -1;
}

/* Returns the class id, or -1 when idx is not below the number of points. */
int llvqo_decode(uint64_t idx, int8_t *x) {
    int c = (idx < g_total) ? find_class(idx) : -1;
    if (c < 0) { memset(x, 0, NCOORD); return -1; }
    const cls_t *k = &g_cls[c];
    uint64_t r = idx - k->base;
    if (k->odd) {
        uint64_t msg = r % 4096u, rho = r / 4096u;
        uint32_t cw = g_word[msg];
        int seq[NCOORD];
        unrank_arrangement(rho, k->mags, NCOORD, seq);
        for (int i = 0; i < NCOORD; i++) {
            int a = seq[i];
            int want = 1 + 2 * (int)((cw >> i) & 1);           /* x_i mod 4 */
            x[i] = (int8_t)((a % 4 == want) ? a : -a);
        }
        return c;
    }
    int w = k->w;
    uint64_t nsign = (uint64_t)1 << (k->nzB + (w > 0 ? w - 1 : 0));
    uint64_t sigma = r % nsign; r /= nsign;
    uint64_t rhoB = r % k->permB; r /= k->permB;
    uint64_t rhoA = r % k->permA; r /= k->permA;
    uint32_t cw = g_byw[w][r];                                 /* r-th word of that weight */
    int seqA[NCOORD], seqB[NCOORD];
    unrank_arrangement(rhoA, k->mags, w, seqA);
    unrank_arrangement(rhoB, k->mags + w, NCOORD - w, seqB);
    int ia = 0, ib = 0, v[NCOORD];
    for (int i = 0; i < NCOORD; i++) v[i] = ((cw >> i) & 1) ? seqA[ia++] : seqB[ib++];
    /* signs: first the non-zero off-support coordinates, ascending, one bit each */
    int bit = 0;
    for (int i = 0; i < NCOORD; i++)
        if (!((cw >> i) & 1) && v[i]) { if ((sigma >> bit) & 1) v[i] = -v[i]; bit++; }
    /* then the support coordinates except the last one */
    int last = -1, seen = 0;
    for (int i = 0; i < NCOORD; i++)
        if ((cw >> i) & 1) {
            seen++;
            if (seen == w) { last = i; break; }
            if ((sigma >> bit) & 1) v[i] = -v[i];
            bit++;
        }
    /* the last support sign repairs the sum condition: sum = 0 mod 8 */
    if (last >= 0) {
        int s = 0;
        for (int i = 0; i < NCOORD; i++) s += v[i];
        if (((s % 8) + 8) % 8 != 0) v[last] = -v[last];
    }
    for (int i = 0; i < NCOORD; i++) x[i] = (int8_t)v[i];
    return c;
}

/* Point -> index; -1 when the point is not in the ball or not in the lattice. */
int64_t llvqo_encode(const int8_t *x) {
    int par = ((x[0] % 2) + 2) % 2, sq = 0, sum = 0;
    for (int i = 0; i < NCOORD; i++) {
        if ((((x[i] % 2) + 2) % 2) != par) return -1;
        sq += x[i] * x[i]; sum += x[i];
    }
    if (sq % 16 || sq / 16 < 2 || sq / 16 > g_maxshell) return -1;
    if ((((sum - 4 * par) % 8) + 8) % 8) return -1;
    uint32_t cw = 0;
    for (int i = 0; i < NCOORD; i++) {
        int res = ((x[i] % 4) + 4) % 4;                        /* even: 0 or 2; odd: 1 or 3 */
        if (res >= 2) cw |= 1u << i;
    }
    if (!golay_contains(cw)) return -1;
    cls_t key;
    memset(&key, 0, sizeof key);
    key.shell = sq / 16; key.odd = par;
    int seqA[NCOORD], seqB[NCOORD], na = 0, nb = 0;
    if (par) {
        for (int i = 0; i < NCOORD; i++) seqA[na++] = abs(x[i]);
    } else {
        key.w = popcount32(cw);
        for (int i = 0; i < NCOORD; i++) { if ((cw >> i) & 1) seqA[na++] = abs(x[i]); else seqB[nb++] = abs(x[i]); }
    }
    /* sorted copies make the class key */
    int sa[NCOORD], sb[NCOORD];
    memcpy(sa, seqA, sizeof(int) * (size_t)na); memcpy(sb, seqB, sizeof(int) * (size_t)nb);
    for (int i = 1; i < na; i++) { int v = sa[i], j = i - 1; while (j >= 0 && sa[j] > v) { sa[j + 1] = sa[j]; j--; } sa[j + 1] = v; }
    for (int i = 1; i < nb; i++) { int v = sb[i], j = i - 1; while (j >= 0 && sb[j] > v) { sb[j + 1] = sb[j]; j--; } sb[j + 1] = v; }
    memcpy(key.mags, sa, sizeof(int) * (size_t)na); memcpy(key.mags + na, sb, sizeof(int) * (size_t)nb);
    int c = -1;
    for (int i = 0; i < g_ncls; i++) if (cls_cmp(&key, &g_cls[i]) == 0) { c = i; break; }
    if (c < 0) return -1;
    const cls_t *k = &g_cls[c];
    if (par) {
        /* message bits: solve cw = XOR of rows; the code is small enough to search */
        int msg = -1;
        for (int m = 0; m < 4096; m++) if (g_word[m] == cw) { msg = m; break; }
        return (int64_t)(k->base + rank_arrangement(seqA, NCOORD) * 4096u + (uint64_t)msg);
    }
    uint64_t kw = 0;
    for (int i = 0; i < g_nw[key.w]; i++) if (g_byw[key.w][i] == cw) { kw = (uint64_t)i; break; }
    uint64_t sigma = 0; int bit = 0;
    for (int i = 0; i < NCOORD; i++)
        if (!((cw >> i) & 1) && x[i]) { if (x[i] < 0) sigma |= (uint64_t)1 << bit; bit++; }
    int seen = 0;
    for (int i = 0; i < NCOORD; i++)
        if ((cw >> i) & 1) { seen++; if (seen == key.w) break; if (x[i] < 0) sigma |= (uint64_t)1 << bit; bit++; }
    uint64_t nsign = (uint64_t)1 << (k->nzB + (key.w > 0 ? key.w - 1 : 0));
    uint64_t r = kw;
    r = r * k->permA + rank_arrangement(seqA, na);
    r = r * k->permB + rank_arrangement(seqB, nb);
    r = r * nsign + sigma;
    return (int64_t)(k->base + r);
}

/* ------------------------------------------------------------------------------------ */
/* Records (Sec. 2.2) and the two in-memory layouts.                                       */
/* ------------------------------------------------------------------------------------ */

#define SENTINEL_CLASS 511   /* class id of a code that names no point: all fields zero */

typedef struct {
    int cls, gain;
    uint32_t smask;            /* bit i: x_i < 0                                          */
    uint32_t plane[3];         /* bit i of plane t: bit t of (|x_i| >> 1)                 */
    uint32_t onehot[4];        /* bit i of mask l-1: rank level of x_i equals l, l = 1..4 */
    int8_t x[NCOORD];
} record_t;

/* code word = index | gain << 47 */
static void make_record(uint64_t code, record_t *rec) {
    memset(rec, 0, sizeof *rec);
    rec->gain = (int)((code >> 47) & 1);
    uint64_t idx = code & (((uint64_t)1 << 47) - 1);
    int c = (code >> 48) ? -1 : llvqo_decode(idx, rec->x);
    if (c < 0) { rec->cls = SENTINEL_CLASS; rec->gain = 0; memset(rec->x, 0, NCOORD); return; }
    rec->cls = c;
    const cls_t *k = &g_cls[c];
    for (int i = 0; i < NCOORD; i++) {
        int a = abs(rec->x[i]);
        if (rec->x[i] < 0) rec->smask |= 1u << i;
        for (int t = 0; t < 3; t++) if (((a >> 1) >> t) & 1) rec->plane[t] |= 1u << i;
        int lvl = 0;
        while (k->dist[lvl] != a) lvl++;
        if (lvl > 0) rec->onehot[lvl - 1] |= 1u << i;
    }
}

/* fields[0]=class, [1]=gain, [2]=smask, [3..5]=planes, [6..9]=one-hot masks */
int llvqo_record(uint64_t code, uint32_t *fields, int8_t *x) {
    record_t r;
    make_record(code, &r);
    fields[0] = (uint32_t)r.cls; fields[1] = (uint32_t)r.gain; fields[2] = r.smask;
    for (int t = 0; t < 3; t++) fields[3 + t] = r.plane[t];
    for (int t = 0; t < 4; t++) fields[6 + t] = r.onehot[t];
    memcpy(x, r.x, NCOORD);
    return r.cls;
}

size_t llvqo_planes_bytes(int64_t rows, int64_t nb) { return (size_t)((rows + 31) / 32) * (size_t)nb * 448u; }
size_t llvqo_planes13_bytes(int64_t rows, int64_t nb) { return (size_t)((rows + 31) / 32) * (size_t)nb * 416u; }
size_t llvqo_onehot_bytes(int64_t rows, int64_t nb) { return (size_t)((rows + 31) / 32) * (size_t)nb * 640u; }

/*
 * 14-byte layout ("planes"): per block a 16-bit header = class | gain << 9 and 24 four-bit codes
 * u_i = 8 + floor(x_i / 2), so x_i = 2 (u_i - 8) + parity of the class; the same 106 bits as the
 * record's sign mask and three level planes (u_i = 8 + level for a positive coordinate,
 * 8 - level - parity for a negative one).  The sentinel record has u_i = 8.
 *
 * Rows are taken 32 at a time (a row group; rows past the end hold the sentinel); row
 * r = 16 m + 8 e + g with m, e in {0,1}, g in 0..7.  A lane is L = 4 g + t, t in 0..3.
 *
 * A half-step covers 16 rows (one m) of two block slots, 48 positions kappa: kappa < 24 is
 * coordinate kappa of slot 0, otherwise coordinate kappa - 24 of slot 1.  Lane L owns three words;
 * nibble n = 2 i + c (i = 0..3, c = 0..1) of a word sits at bits 4n .. 4n+3:
 *   Wa: code of row (m, e=0, g) at position 16 c + 4 t + i
 *   Wb: code of row (m, e=1, g) at position 16 c + 4 t + i
 *   Wc: code of row (m, e=c, g) at position 32 + 4 t + i
 * and lane pair P = 2 g + (t >> 1) owns one header word:
 *   header(row (m,0,g), slot t >> 1) | header(row (m,1,g), slot t >> 1) << 16.
 *
 * Tile = blocks 4T .. 4T+3 of a row group, 1792 bytes: half-step h = 2 s + m has slots 4T+2s and
 * 4T+2s+1; word w = 3 h + (0 Wa, 1 Wb, 2 Wc) of lane L at 512 (w >> 2) + 16 L + 4 (w & 3); header
 * word h of pair P at 1536 + 16 P + 4 h.
 * The c = nb mod 4 blocks left over follow the tiles, 448 c bytes:
 *   c >= 2: a pair (896 bytes) for the next two blocks: half-steps m = 0,1 with those two blocks
 *           as slots; word w = 3 m + (0,1,2) of lane L at 128 w + 4 L; header word m of pair P at
 *           768 + 8 P + 4 m.
 *   c odd:  a single (448 bytes) for the last block: one half-step whose slot s is rows
 *           16 s .. 16 s + 15 of that block (read "row (m,e,g), slot s" above as row (s,e,g));
 *           word w of lane L at 128 w + 4 L; header word of pair P at 384 + 4 P.
 * A row group occupies 448 nb bytes.
 *
 * 13-byte layout: the matvec needs of the header only what fixes the block's scale and the
 * parity of its coordinates, so the 16-bit header shrinks to one byte
 *     shell (4 bits, 0 for the sentinel) | parity << 4 | gain << 5
 * and everything else stays: the same code words at the same places, then the header bytes.
 *   tile, 1664 bytes: header byte of pair P, half-step h, row half e at 1536 + 8 P + 2 h + e;
 *   pair, 832 bytes: header byte of pair P, half-step m, row half e at 768 + 4 P + 2 m + e;
 *   single, 416 bytes: header byte of pair P (slot = t >> 1 = the 16-row half), row half e at 384 + 2 P + e.
 * A row group occupies 416 nb bytes.  Every lattice point of the ball has such a record: the
 * layout is exact for all blocks at 4.33 bits a weight (the rate the paper reaches with a
 * 12-byte record plus an exception table for five-level blocks, Sec. 3.3).
 */
typedef struct { const uint8_t *code; const uint16_t *hdr; int64_t nb; } group_t;   /* code[(r*nb+b)*24+i], hdr[r*nb+b] */

/* code at position kappa of a half-step: rows 16 m + 8 e + g of blocks b0 (slot 0) and b1 (slot 1);
 * in a single (b1 < 0) the slot picks the row half instead */
static uint32_t hs_code(const group_t *G, int64_t b0, int64_t b1, int m, int e, int g, int kappa) {
    int slot = kappa / 24, i = kappa % 24;
    int row = (b1 < 0) ? 16 * slot + 8 * e + g : 16 * m + 8 * e + g;
    int64_t b = (b1 < 0) ? b0 : (slot ? b1 : b0);
    return G->code[((size_t)row * G->nb + b) * 24 + i];
}
static uint32_t hs_header(const group_t *G, int64_t b0, int64_t b1, int m, int e, int g, int slot) {
    int row = (b1 < 0) ? 16 * slot + 8 * e + g : 16 * m + 8 * e + g;
    int64_t b = (b1 < 0) ? b0 : (slot ? b1 : b0);
    return G->hdr[(size_t)row * G->nb + b];
}
/* the three words of lane (g, t) and the header word of its pair */
static void hs_words(const group_t *G, int64_t b0, int64_t b1, int m, int g, int t, uint32_t w[3], uint32_t *hw) {
    w[0] = w[1] = w[2] = 0;
    for (int i = 0; i < 4; i++)
        for (int c = 0; c < 2; c++) {
            int n = 2 * i + c;
            w[0] |= hs_code(G, b0, b1, m, 0, g, 16 * c + 4 * t + i) << (4 * n);
            w[1] |= hs_code(G, b0, b1, m, 1, g, 16 * c + 4 * t + i) << (4 * n);
            w[2] |= hs_code(G, b0, b1, m, c, g, 32 + 4 * t + i) << (4 * n);
        }
    *hw = hs_header(G, b0, b1, m, 0, g, t >> 1) | hs_header(G, b0, b1, m, 1, g, t >> 1) << 16;
}

static void pack_planes_any(const uint64_t *codes, int64_t rows, int64_t nb, uint8_t *out, int compact) {
    const size_t cell = compact ? 416u : 448u, words4 = 1536u, words2 = 768u, words1 = 384u;
    int64_t ngroups = (rows + 31) / 32, ntiles = nb / 4, left = nb % 4;
    uint8_t *code = malloc((size_t)32 * nb * 24);
    uint16_t *hdr = malloc((size_t)32 * nb * 2);
    for (int64_t rg = 0; rg < ngroups; rg++) {
        for (int r = 0; r < 32; r++)
            for (int64_t b = 0; b < nb; b++) {
                record_t rec;
                int64_t row = rg * 32 + r;
                if (row < rows) make_record(codes[row * nb + b], &rec);
                else { memset(&rec, 0, sizeof rec); rec.cls = SENTINEL_CLASS; }
                int parity = rec.cls == SENTINEL_CLASS ? 0 : (rec.x[0] & 1);
                for (int i = 0; i < NCOORD; i++) code[((size_t)r * nb + b) * 24 + i] = (uint8_t)(8 + (rec.x[i] - parity) / 2);
                hdr[(size_t)r * nb + b] = compact ? (uint16_t)((rec.cls == SENTINEL_CLASS ? 0 : g_cls[rec.cls].shell) | (parity << 4) | (rec.gain << 5))
                                                  : (uint16_t)(rec.cls | (rec.gain << 9));
            }
        group_t G = {code, hdr, nb};
        uint8_t *grp = out + (size_t)rg * (size_t)nb * cell;
        uint32_t w[3], hw;
        for (int g = 0; g < 8; g++)
            for (int t = 0; t < 4; t++) {
                int L = 4 * g + t, P = 2 * g + (t >> 1);
                for (int64_t T = 0; T < ntiles; T++)
                    for (int h = 0; h < 4; h++) {
                        hs_words(&G, 4 * T + 2 * (h >> 1), 4 * T + 2 * (h >> 1) + 1, h & 1, g, t, w, &hw);
                        uint8_t *tile = grp + (size_t)T * 4u * cell;
                        for (int q = 0; q < 3; q++) { int k = 3 * h + q; memcpy(tile + 512 * (k >> 2) + 16 * L + 4 * (k & 3), &w[q], 4); }
                        if (compact) { tile[words4 + 8 * P + 2 * h] = (uint8_t)hw; tile[words4 + 8 * P + 2 * h + 1] = (uint8_t)(hw >> 16); }
                        else memcpy(tile + words4 + 16 * P + 4 * h, &hw, 4);
                    }
                uint8_t *rest = grp + (size_t)ntiles * 4u * cell;
                if (left >= 2) {
                    for (int m = 0; m < 2; m++) {
                        hs_words(&G, 4 * ntiles, 4 * ntiles + 1, m, g, t, w, &hw);
                        for (int q = 0; q < 3; q++) memcpy(rest + 128 * (3 * m + q) + 4 * L, &w[q], 4);
                        if (compact) { rest[words2 + 4 * P + 2 * m] = (uint8_t)hw; rest[words2 + 4 * P + 2 * m + 1] = (uint8_t)(hw >> 16); }
                        else memcpy(rest + words2 + 8 * P + 4 * m, &hw, 4);
                    }
                    rest += 2u * cell;
                }
                if (left & 1) {
                    hs_words(&G, nb - 1, -1, 0, g, t, w, &hw);
                    for (int q = 0; q < 3; q++) memcpy(rest + 128 * q + 4 * L, &w[q], 4);
                    if (compact) { rest[words1 + 2 * P] = (uint8_t)hw; rest[words1 + 2 * P + 1] = (uint8_t)(hw >> 16); }
                    else memcpy(rest + words1 + 4 * P, &hw, 4);
                }
            }
    }
    free(code); free(hdr);
}
void llvqo_pack_planes(const uint64_t *codes, int64_t rows, int64_t nb, uint8_t *out) { pack_planes_any(codes, rows, nb, out, 0); }
void llvqo_pack_planes13(const uint64_t *codes, int64_t rows, int64_t nb, uint8_t *out) { pack_planes_any(codes, rows, nb, out, 1); }

/*
 * 10-byte layout with an exception table (the sparse overlay of Sec. 3.3, with a window code in place of the
 * paper's level code).  For a block with four-bit codes u_0..u_23 (u_i = 8 + floor(x_i / 2)) the window base o
 * is the smallest of 3, 4, 5, 6 with o <= min u and max u <= o + 7; the short record keeps v_i = u_i - o in three
 * bits and the header byte (f ^ shell) | shell << 4, f = (o - 3) | parity << 2 | gain << 3.  A block with no such o is an
 * exception: all-zero short record, exact record in the table.  Rows past the end and codes that name no point:
 * all-zero short record, no table entry.
 *
 * Tile (blocks 4T..4T+3 of a row group), 1280 bytes.  Rows, lanes, half-steps, positions as in the 14-byte layout.
 * Group(h, e, c) of lane (g, t): the codes of row (m, e, g), m = h & 1, at positions 16 c + 4 t + i (c < 2) or
 * 32 + 4 t + i (c = 2), i = 0..3, of half-step h.  Nine words V0..V8 a lane; byte i of a word holds code i of two
 * groups (bits 0..2 and 3..5): V(2h+e) = Group(h,e,0), Group(h,e,1); V8 = Group(0,0,2), Group(1,0,2).  The other six
 * groups X0..X5 = Group(0,1,2), Group(1,1,2), Group(2,0,2), Group(2,1,2), Group(3,0,2), Group(3,1,2) live in bits 6, 7:
 * bits 0, 1 of code i of Xk are bits 6, 7 of byte i of Vk; bit 2 of it is bit 6 + (k & 1) of byte i of V(6 + (k >> 1)).
 * Vk of lane L at 16 L + 4 k (k < 4), 512 + 16 L + 4 (k - 4) (k < 8), 1024 + 4 L (k = 8); header byte of pair P,
 * half-step h, row half e at 1152 + 8 P + 2 h + e.
 * The nb mod 4 last blocks follow in the 13-byte layout's pair and single (four-bit codes, that layout's header byte, exact).
 * After the row groups, at the next multiple of 128: the index (one uint32 a tile, row group by row group, and one
 * more; entry i = exceptions of the tiles before tile i, never above the capacity); after it, at the next multiple
 * of 128: the table, 16 bytes an
 * entry, in the order row group, tile, block, row: word 0 = shell | parity << 4 | gain << 5 | row of the group << 8 |
 * block column << 13, words 1..3 the four-bit codes (coordinate 8 j + n in nibble n of word 1 + j).
 */
static size_t up128(size_t v) { return (v + 127u) & ~(size_t)127u; }
static size_t p10_group_bytes(int64_t nb) { return (size_t)(nb / 4) * 1280u + (size_t)(nb % 4) * 416u; }
static size_t p10_index_offset(int64_t rows, int64_t nb) { return up128((size_t)((rows + 31) / 32) * p10_group_bytes(nb)); }
static size_t p10_table_offset(int64_t rows, int64_t nb) { return p10_index_offset(rows, nb) + up128((size_t)((rows + 31) / 32 * (nb / 4) + 1) * 4u); }
size_t llvqo_planes10x_bytes(int64_t rows, int64_t nb, uint64_t exceptions) { return p10_table_offset(rows, nb) + (size_t)exceptions * 16u; }

/* window base of a block's codes, 0 if none fits */
static int window_base(const uint8_t *u) {
    int lo = 15, hi = 0;
    for (int i = 0; i < NCOORD; i++) { if (u[i] < lo) lo = u[i]; if (u[i] > hi) hi = u[i]; }
    for (int o = 3; o <= 6; o++) if (o <= lo && hi <= o + 7) return o;
    return 0;
}

/* returns the number of exceptions met (all of them, also those past `capacity`, which are not stored) */
int64_t llvqo_pack_planes10x(const uint64_t *codes, int64_t rows, int64_t nb, uint8_t *out, uint64_t capacity) {
    const int64_t ngroups = (rows + 31) / 32, ntiles = nb / 4, left = nb % 4;
    const size_t gbytes = p10_group_bytes(nb);
    memset(out, 0, llvqo_planes10x_bytes(rows, nb, capacity));
    uint32_t *index = (uint32_t *)(out + p10_index_offset(rows, nb));
    uint8_t *table = out + p10_table_offset(rows, nb);
    uint8_t *u = malloc((size_t)32 * nb * 24);        /* four-bit codes */
    uint8_t *v = malloc((size_t)32 * nb * 24);        /* what the short record stores */
    uint8_t *hb = malloc((size_t)32 * nb);            /* header byte of the exact record (no window bits) */
    uint8_t *hs = malloc((size_t)32 * nb);            /* header byte of the short record */
    uint8_t *exc = malloc((size_t)32 * nb);
    uint64_t count = 0;
    for (int64_t rg = 0; rg < ngroups; rg++) {
        for (int r = 0; r < 32; r++)
            for (int64_t b = 0; b < nb; b++) {
                record_t rec;
                int64_t row = rg * 32 + r;
                size_t at = (size_t)r * nb + b;
                if (row < rows) make_record(codes[row * nb + b], &rec);
                else { memset(&rec, 0, sizeof rec); rec.cls = SENTINEL_CLASS; }
                int empty = rec.cls == SENTINEL_CLASS;
                int parity = empty ? 0 : (rec.x[0] & 1);
                for (int i = 0; i < NCOORD; i++) u[at * 24 + i] = (uint8_t)(8 + (rec.x[i] - parity) / 2);
                hb[at] = empty ? 0 : (uint8_t)(g_cls[rec.cls].shell | (parity << 4) | (rec.gain << 5));
                int o = empty ? 0 : window_base(u + at * 24);
                exc[at] = !empty && o == 0;
                hs[at] = o ? (uint8_t)((((o - 3) | (parity << 2) | (rec.gain << 3)) ^ g_cls[rec.cls].shell) | (g_cls[rec.cls].shell << 4)) : 0;
                for (int i = 0; i < NCOORD; i++) v[at * 24 + i] = o ? (uint8_t)(u[at * 24 + i] - o) : 0;
            }
        uint8_t *grp = out + (size_t)rg * gbytes;
        /* the tiles: three-bit codes */
        for (int64_t T = 0; T < ntiles; T++) {
            index[rg * ntiles + T] = (uint32_t)(count < capacity ? count : capacity);
            uint8_t *tile = grp + (size_t)T * 1280u;
            for (int g = 0; g < 8; g++)
                for (int t = 0; t < 4; t++) {
                    int L = 4 * g + t, P = 2 * g + (t >> 1);
                    uint32_t grpw[4][2][3];              /* [h][e][c]: byte i = code i of Group(h, e, c) */
                    for (int h = 0; h < 4; h++)
                        for (int e = 0; e < 2; e++)
                            for (int c = 0; c < 3; c++) {
                                uint32_t w = 0;
                                for (int i = 0; i < 4; i++) {
                                    int kappa = (c < 2 ? 16 * c : 32) + 4 * t + i;
                                    int64_t b = 4 * T + 2 * (h >> 1) + kappa / 24;
                                    int row = 16 * (h & 1) + 8 * e + g;
                                    w |= (uint32_t)v[((size_t)row * nb + b) * 24 + kappa % 24] << (8 * i);
                                }
                                grpw[h][e][c] = w;
                            }
                    uint32_t V[9];
                    for (int k = 0; k < 8; k++) V[k] = grpw[k >> 1][k & 1][0] | grpw[k >> 1][k & 1][1] << 3;
                    V[8] = grpw[0][0][2] | grpw[1][0][2] << 3;
                    const uint32_t X[6] = {grpw[0][1][2], grpw[1][1][2], grpw[2][0][2], grpw[2][1][2], grpw[3][0][2], grpw[3][1][2]};
                    for (int k = 0; k < 6; k++) {
                        V[k] |= (X[k] & 0x03030303u) << 6;
                        V[6 + (k >> 1)] |= ((X[k] >> 2) & 0x01010101u) << (6 + (k & 1));
                    }
                    for (int k = 0; k < 9; k++) {
                        size_t at = k < 4 ? 16u * L + 4u * k : (k < 8 ? 512u + 16u * L + 4u * (k - 4) : 1024u + 4u * L);
                        memcpy(tile + at, &V[k], 4);
                    }
                    for (int h = 0; h < 4; h++)
                        for (int e = 0; e < 2; e++) {
                            int row = 16 * (h & 1) + 8 * e + g;
                            int64_t b = 4 * T + 2 * (h >> 1) + (t >> 1);
                            tile[1152 + 8 * P + 2 * h + e] = hs[(size_t)row * nb + b];
                        }
                }
            /* the tile's exceptions: block by block, row by row */
            for (int q = 0; q < 4; q++)
                for (int r = 0; r < 32; r++) {
                    size_t at = (size_t)r * nb + 4 * T + q;
                    if (!exc[at]) continue;
                    if (count < capacity) {
                        uint32_t e4[4] = {(uint32_t)hb[at] | (uint32_t)r << 8 | (uint32_t)(4 * T + q) << 13, 0, 0, 0};
                        for (int i = 0; i < NCOORD; i++) e4[1 + i / 8] |= (uint32_t)u[at * 24 + i] << (4 * (i % 8));
                        memcpy(table + (size_t)count * 16u, e4, 16);
                    }
                    count++;
                }
        }
        /* the blocks left over: the 13-byte layout's pair and single */
        uint16_t *hdr16 = malloc((size_t)32 * nb * 2);
        for (size_t at = 0; at < (size_t)32 * nb; at++) hdr16[at] = hb[at];
        group_t G = {u, hdr16, nb};
        uint8_t *rest0 = grp + (size_t)ntiles * 1280u;
        uint32_t w[3], hw;
        for (int g = 0; g < 8; g++)
            for (int t = 0; t < 4; t++) {
                int L = 4 * g + t, P = 2 * g + (t >> 1);
                uint8_t *rest = rest0;
                if (left >= 2) {
                    for (int m = 0; m < 2; m++) {
                        hs_words(&G, 4 * ntiles, 4 * ntiles + 1, m, g, t, w, &hw);
                        for (int q = 0; q < 3; q++) memcpy(rest + 128 * (3 * m + q) + 4 * L, &w[q], 4);
                        rest[768 + 4 * P + 2 * m] = (uint8_t)hw; rest[768 + 4 * P + 2 * m + 1] = (uint8_t)(hw >> 16);
                    }
                    rest += 832;
                }
                if (left & 1) {
                    hs_words(&G, nb - 1, -1, 0, g, t, w, &hw);
                    for (int q = 0; q < 3; q++) memcpy(rest + 128 * q + 4 * L, &w[q], 4);
                    rest[384 + 2 * P] = (uint8_t)hw; rest[384 + 2 * P + 1] = (uint8_t)(hw >> 16);
                }
            }
        free(hdr16);
    }
    index[ngroups * ntiles] = (uint32_t)(count < capacity ? count : capacity);
    free(u); free(v); free(hb); free(hs); free(exc);
    return (int64_t)count;
}

/*
 * One-hot layout, 20 bytes a block: the cell of (row group, block column) is five arrays of 32
 * words, one entry a row: V0 = smask | class[7:0] << 24, V1 = mask1 | class[8] << 24 | gain << 25,
 * V2 = mask2, V3 = mask3, V4 = mask4.  Word t of row l sits at 128 t + 4 l; a row group occupies
 * 640 nb bytes.
 */
void llvqo_pack_onehot(const uint64_t *codes, int64_t rows, int64_t nb, uint8_t *out) {
    int64_t ngroups = (rows + 31) / 32;
    for (int64_t rg = 0; rg < ngroups; rg++)
        for (int l = 0; l < 32; l++) {
            int64_t row = rg * 32 + l;
            for (int64_t b = 0; b < nb; b++) {
                record_t r;
                if (row < rows) make_record(codes[row * nb + b], &r);
                else { memset(&r, 0, sizeof r); r.cls = SENTINEL_CLASS; }
                uint32_t v[5];
                v[0] = r.smask | ((uint32_t)(r.cls & 255) << 24);
                v[1] = r.onehot[0] | ((uint32_t)(r.cls >> 8) << 24) | ((uint32_t)r.gain << 25);
                v[2] = r.onehot[1]; v[3] = r.onehot[2]; v[4] = r.onehot[3];
                uint8_t *cell = out + ((size_t)rg * (size_t)nb + (size_t)b) * 640u;
                for (int t = 0; t < 5; t++) memcpy(cell + 128 * t + 4 * l, &v[t], 4);
            }
        }
}

/* ------------------------------------------------------------------------------------ */
/* Dequantised weights and the f64 matvec (Sec. 2.3).                                      */
/* ------------------------------------------------------------------------------------ */

static double half_to_double(uint16_t h) {
    int s = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)f, -24);
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp((double)(f + 1024), e - 25);
    return s ? -v : v;
}

/* W[row, 24 b + i] = r_row * gain[g] * x_i / (4 sqrt(m)); one block written to w[24] */
static void block_weights(uint64_t code, double rscale, const double *gain, double *w) {
    record_t r;
    make_record(code, &r);
    if (r.cls == SENTINEL_CLASS) { for (int i = 0; i < NCOORD; i++) w[i] = 0.0; return; }
    double unit = 1.0 / (4.0 * sqrt((double)g_cls[r.cls].shell));
    for (int i = 0; i < NCOORD; i++) w[i] = rscale * gain[r.gain] * (double)r.x[i] * unit;
}

void llvqo_dequant(const uint64_t *codes, int64_t rows, int64_t nb, const uint16_t *row_scale,
                   const double *gain, double *W) {
    for (int64_t row = 0; row < rows; row++)
        for (int64_t b = 0; b < nb; b++)
            block_weights(codes[row * nb + b], half_to_double(row_scale[row]), gain, W + (row * nb + b) * NCOORD);
}

typedef struct {
    const uint64_t *codes; int64_t rows, nb, row0, row1;
    const uint16_t *row_scale, *x; const double *gain;
    double *y, *wnorm, *abssum;
} mv_job;

static void *mv_worker(void *arg) {
    mv_job *j = (mv_job *)arg;
    for (int64_t row = j->row0; row < j->row1; row++) {
        double acc = 0.0, n2 = 0.0, as = 0.0, w[NCOORD];
        double rs = half_to_double(j->row_scale[row]);
        for (int64_t b = 0; b < j->nb; b++) {
            block_weights(j->codes[row * j->nb + b], rs, j->gain, w);
            for (int i = 0; i < NCOORD; i++) {
                double xv = half_to_double(j->x[b * NCOORD + i]);
                acc += w[i] * xv; n2 += w[i] * w[i]; as += fabs(w[i] * xv);
            }
        }
        j->y[row] = acc;
        if (j->wnorm) j->wnorm[row] = sqrt(n2);
        if (j->abssum) j->abssum[row] = as;
    }
    return NULL;
}

/* y = W x in f64; wnorm[row] = ||W[row,:]||_2, abssum[row] = sum |w x| (either may be NULL).
 * Rows are split over nthreads threads; every row is summed in the same order whatever the split. */
void llvqo_matvec(const uint64_t *codes, int64_t rows, int64_t nb, const uint16_t *row_scale,
                  const double *gain, const uint16_t *x, double *y, double *wnorm, double *abssum, int nthreads) {
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    pthread_t th[256]; mv_job job[256];
    int64_t per = (rows + nthreads - 1) / nthreads;
    int started = 0;
    for (int t = 0; t < nthreads; t++) {
        int64_t r0 = t * per, r1 = r0 + per > rows ? rows : r0 + per;
        if (r0 >= r1) break;
        job[t] = (mv_job){codes, rows, nb, r0, r1, row_scale, x, gain, y, wnorm, abssum};
        if (nthreads == 1) mv_worker(&job[t]); else pthread_create(&th[t], NULL, mv_worker, &job[t]);
        started++;
    }
    if (nthreads > 1) for (int t = 0; t < started; t++) pthread_join(th[t], NULL);
}

/* decode a batch: x[n][24], cls[n] (sentinel -1 for codes that name no point) */
void llvqo_decode_batch(const uint64_t *codes, int64_t n, int8_t *x, int32_t *cls) {
    for (int64_t i = 0; i < n; i++) {
        uint64_t idx = codes[i] & (((uint64_t)1 << 47) - 1);
        cls[i] = (codes[i] >> 48) ? -1 : llvqo_decode(idx, x + i * NCOORD);
        if (cls[i] < 0) memset(x + i * NCOORD, 0, NCOORD);
    }
}

/* ------------------------------------------------------------------------------------ */
/* Activation rotation: the Walsh-Hadamard transform applied to the activation ahead of   */
/* every projection (Sec. 2.3, the kernel; Sec. 5, the paragraph on the rotated basis).     */
/* ------------------------------------------------------------------------------------ */
/*
 * The definition written out, block by block:
 *     y[B c + k] = (1 / sqrt(B)) * sum_{i < B} (-1)^popcount(i & k) * s_i * x[B c + i],
 * the Sylvester (natural-order) Hadamard matrix H_B[k][i] = (-1)^popcount(k & i), normalised
 * so that the rotation is orthogonal.  B^2 operations a block: no fast transform here.
 *
 * Readings (the paper names the transform and nothing else about it):
 *   - Lengths that are not powers of two (2560, 9728, 17408 ...): the rotation is block
 *     diagonal, B the largest power of two that divides n (at most 16384) unless the caller
 *     names a smaller power of two.
 *   - Order: natural (Sylvester) order; scale 1 / sqrt(B).
 *   - An optional sign flip s_i = -1 per input coordinate ahead of the transform (the usual
 *     randomised form of an incoherence rotation); none when `negate` is NULL.
 *   - Input and output are FP16, as the GEMV reads them.  The sum is taken exactly (every
 *     FP16 value is a multiple of 2^-24, so the sum is an integer in that unit), scaled in
 *     f64 and rounded once to FP16, to nearest even: the output is the correctly rounded
 *     value of the definition whenever the block's sum of |x| stays below 2^29.
 */
static uint16_t double_to_half(double v) {
    uint16_t sign = (uint16_t)(signbit(v) ? 0x8000 : 0);
    double a = fabs(v);
    if (isnan(a)) return (uint16_t)(sign | 0x7E00);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7C00);
    int e;
    (void)frexp(a, &e);                       /* a = m 2^e, 1/2 <= m < 1: leading bit at 2^(e-1) */
    int q = (e - 1 < -14 ? -14 : e - 1) - 10; /* weight of the last kept bit */
    double r = rint(ldexp(a, -q));            /* exact scaling; ties to even in the default mode */
    if (r >= 2048.0) { r = 1024.0; q += 1; }
    if (r < 1024.0) return (uint16_t)(sign | (uint16_t)r);            /* subnormal, q = -24 */
    int biased = q + 10 + 15;
    if (biased >= 31) return (uint16_t)(sign | 0x7C00);
    return (uint16_t)(sign | (biased << 10) | ((int)r - 1024));
}
uint16_t llvqo_double_to_half(double v) { return double_to_half(v); }

int64_t llvqo_rotate_block(int64_t n, int64_t block) {
    if (n <= 0) return 0;
    if (block == 0) {
        block = 1;
        while (block < 16384 && n % (2 * block) == 0) block *= 2;
        return block;
    }
    if (block < 1 || block > 16384 || (block & (block - 1)) || n % block) return 0;
    return block;
}

/* x[n], out[n] FP16 bit patterns; negate[n] bytes (non-zero = flip the sign of x_i) or NULL.
 * Returns the block length used, 0 if `block` is not a power of two that divides n. */
int64_t llvqo_rotate(const uint16_t *x, int64_t n, int64_t block, const uint8_t *negate, uint16_t *out) {
    int64_t B = llvqo_rotate_block(n, block);
    if (B == 0) return 0;
    double scale = ldexp(1.0 / sqrt((double)B), -24);
    int64_t *t = (int64_t *)malloc((size_t)B * sizeof(int64_t));
    for (int64_t c = 0; c < n / B; c++) {
        for (int64_t i = 0; i < B; i++) {
            uint16_t h = x[B * c + i];
            int e = (h >> 10) & 31, f = h & 1023;
            int64_t v = e == 0 ? (int64_t)f : (int64_t)(f + 1024) << (e - 1);   /* |x_i| in units of 2^-24 */
            if (h >> 15) v = -v;
            if (negate && negate[B * c + i]) v = -v;
            t[i] = v;
        }
        for (int64_t k = 0; k < B; k++) {
            __int128 s = 0;
            for (int64_t i = 0; i < B; i++) s += (__builtin_popcountll((unsigned long long)(i & k)) & 1) ? -t[i] : t[i];
            out[B * c + k] = double_to_half((double)s * scale);
        }
    }
    free(t);
    return B;
}
