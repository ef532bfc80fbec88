#include "llvq_tables.h"

#include <algorithm>
#include <array>
#include <cmath>
#include <cstring>

namespace llvq {
namespace {

struct Pascal {
    uint64_t c[25][25];
    Pascal() {
        std::memset(c, 0, sizeof c);
        for (int n = 0; n <= 24; n++) {
            c[n][0] = 1;
            for (int k = 1; k <= n; k++) c[n][k] = c[n - 1][k - 1] + (k <= n - 1 ? c[n - 1][k] : 0);
        }
    }
};

// orderings of a multiset given by its multiplicities
uint64_t orderings(const uint8_t *cnt, int n_values, const Pascal &p) {
    int total = 0;
    for (int i = 0; i < n_values; i++) total += cnt[i];
    uint64_t r = 1;
    for (int i = 0; i < n_values; i++) {
        r *= p.c[total][cnt[i]];
        total -= cnt[i];
    }
    return r;
}

struct Draft {
    int shell, odd, w;
    std::array<int, 24> sorted;   // sort key: support magnitudes ascending, then the rest ascending
    ClassDesc d;
};

void expand_sorted(Draft &k, const int *va, int na, const int *vb, int nbv) {
    int pos = 0;
    for (int i = 0; i < na; i++) for (int j = 0; j < k.d.cnt[i]; j++) k.sorted[pos++] = va[i];
    for (int i = 0; i < nbv; i++) for (int j = 0; j < k.d.cnt[4 + i]; j++) k.sorted[pos++] = vb[i];
}

}  // namespace

bool build_tables(HostTables &t) {
    static const Pascal pascal;

    // ---- extended Golay code: cyclic generator 0xC75 on coordinates 0..22, parity on 23
    t.golay_by_message.assign(4096, 0);
    uint32_t rows[12];
    for (int i = 0; i < 12; i++) {
        uint32_t w = 0xC75u << i;
        w |= (uint32_t)(__builtin_popcount(w) & 1) << 23;
        rows[i] = w;
    }
    for (int k = 1; k < 4096; k++) {
        int low = __builtin_ctz(k);
        t.golay_by_message[k] = t.golay_by_message[k & (k - 1)] ^ rows[low];
    }
    t.golay_by_weight = t.golay_by_message;
    std::sort(t.golay_by_weight.begin(), t.golay_by_weight.end(), [](uint32_t a, uint32_t b) {
        int wa = __builtin_popcount(a), wb = __builtin_popcount(b);
        return wa != wb ? wa < wb : a < b;
    });
    int n_of_weight[25] = {0};
    for (uint32_t w : t.golay_by_weight) n_of_weight[__builtin_popcount(w)]++;
    int off = 0;
    for (int w = 0; w <= 24; w++) { t.weight_offset[w] = off; off += n_of_weight[w]; }
    if (n_of_weight[0] != 1 || n_of_weight[8] != 759 || n_of_weight[12] != 2576 || n_of_weight[16] != 759 || n_of_weight[24] != 1)
        return false;

    // ---- classes: loops over multiplicity vectors
    static const int va[4] = {2, 6, 10, 14}, vb[4] = {0, 4, 8, 12}, vm[7] = {1, 3, 5, 7, 9, 11, 13};
    static const int weights[5] = {0, 8, 12, 16, 24};
    std::vector<Draft> all;
    for (int shell = 2; shell <= kMaxShell; shell++) {
        const int target = 16 * shell;
        for (int w : weights) {
            for (int a2 = 0; a2 <= w; a2++)
                for (int a1 = 0; a1 + a2 <= w; a1++) {
                    int a0 = w - a1 - a2;
                    int sq_a = 4 * a0 + 36 * a1 + 100 * a2;
                    if (sq_a > target) continue;
                    int rest = 24 - w;
                    for (int b3 = 0; b3 <= rest; b3++)
                        for (int b2 = 0; b2 + b3 <= rest; b2++)
                            for (int b1 = 0; b1 + b2 + b3 <= rest; b1++) {
                                if (sq_a + 16 * b1 + 64 * b2 + 144 * b3 != target) continue;
                                if (w == 0 && (4 * b1 + 8 * b2 + 12 * b3) % 8 != 0) continue;   // sum condition
                                Draft k{};
                                k.shell = shell; k.odd = 0; k.w = w;
                                k.d.cnt[0] = (uint8_t)a0; k.d.cnt[1] = (uint8_t)a1; k.d.cnt[2] = (uint8_t)a2; k.d.cnt[3] = 0;
                                k.d.cnt[4] = (uint8_t)(rest - b1 - b2 - b3); k.d.cnt[5] = (uint8_t)b1; k.d.cnt[6] = (uint8_t)b2; k.d.cnt[7] = (uint8_t)b3;
                                expand_sorted(k, va, 4, vb, 4);
                                all.push_back(k);
                            }
                }
        }
        // odd type: multiplicities of 1,3,..,13
        int c[7];
        for (c[6] = 0; c[6] * 169 <= target; c[6]++)
        for (c[5] = 0; c[5] * 121 + c[6] * 169 <= target; c[5]++)
        for (c[4] = 0; c[4] * 81 + c[5] * 121 + c[6] * 169 <= target; c[4]++)
        for (c[3] = 0; c[3] * 49 + c[4] * 81 + c[5] * 121 + c[6] * 169 <= target; c[3]++)
        for (c[2] = 0; c[2] * 25 + c[3] * 49 + c[4] * 81 + c[5] * 121 + c[6] * 169 <= target; c[2]++)
        for (c[1] = 0; c[1] * 9 + c[2] * 25 + c[3] * 49 + c[4] * 81 + c[5] * 121 + c[6] * 169 <= target; c[1]++) {
            int used = c[1] + c[2] + c[3] + c[4] + c[5] + c[6];
            if (used > 24) continue;
            c[0] = 24 - used;
            int sq = 0, signed_sum = 0;
            for (int i = 0; i < 7; i++) {
                sq += c[i] * vm[i] * vm[i];
                signed_sum += c[i] * (vm[i] % 4 == 1 ? vm[i] : -vm[i]);   // representative congruent to 1 mod 4
            }
            if (sq != target) continue;
            if (((signed_sum % 8) + 8) % 8 != 4) continue;                 // sum condition for odd vectors
            Draft k{};
            k.shell = shell; k.odd = 1; k.w = 0;
            int pos = 0;
            for (int i = 0; i < 7; i++) { k.d.cnt[i] = (uint8_t)c[i]; for (int j = 0; j < c[i]; j++) k.sorted[pos++] = vm[i]; }
            all.push_back(k);
        }
    }
    std::sort(all.begin(), all.end(), [](const Draft &a, const Draft &b) {
        if (a.shell != b.shell) return a.shell < b.shell;
        if (a.odd != b.odd) return a.odd < b.odd;
        if (a.w != b.w) return a.w < b.w;
        return a.sorted < b.sorted;
    });

    t.num_classes = (int)all.size();
    t.base.assign(all.size() + 1, 0);
    t.desc.resize(all.size());
    t.cls_scale.assign(kClassSlots, 0.f);
    t.cls_parity.assign(kClassSlots, 0u);
    t.cls_value.assign(kClassSlots * 8, 0.f);
    t.cls_dist.assign(kClassSlots * 8, 0);
    uint64_t running = 0;
    for (size_t c = 0; c < all.size(); c++) {
        Draft &k = all[c];
        ClassDesc &d = k.d;
        d.odd = (uint8_t)k.odd; d.w = (uint8_t)k.w; d.shell = (uint8_t)k.shell;
        uint64_t size;
        if (k.odd) {
            d.perm_a = orderings(d.cnt, 7, pascal);
            d.perm_b = 1;
            d.nz_b = 0; d.sign_bits = 0;
            size = d.perm_a * 4096u;
        } else {
            d.perm_a = orderings(d.cnt, 4, pascal);
            d.perm_b = orderings(d.cnt + 4, 4, pascal);
            d.nz_b = (uint8_t)(d.cnt[5] + d.cnt[6] + d.cnt[7]);
            d.sign_bits = (uint8_t)(d.nz_b + (k.w ? k.w - 1 : 0));
            size = (uint64_t)n_of_weight[k.w] * d.perm_a * d.perm_b << d.sign_bits;
        }
        std::array<int, 24> s = k.sorted;
        std::sort(s.begin(), s.end());
        d.ndist = 0;
        for (int i = 0; i < 24; i++) if (i == 0 || s[i] != s[i - 1]) d.dist[d.ndist++] = (uint8_t)s[i];
        if (d.ndist > 5) return false;
        t.desc[c] = d;
        t.base[c] = running;
        running += size;
        double inv_norm = 1.0 / (4.0 * std::sqrt((double)k.shell));
        t.cls_scale[c] = (float)(2097152.0 * inv_norm);
        t.cls_parity[c] = k.odd ? 0x00080008u : 0u;
        for (int l = 0; l < d.ndist; l++) {
            t.cls_value[c * 8 + l] = (float)(d.dist[l] * inv_norm);
            t.cls_dist[c * 8 + l] = d.dist[l];
        }
    }
    std::memset(t.cls_shell_nibbles, 0, sizeof t.cls_shell_nibbles);
    std::memset(t.cls_odd_bits, 0, sizeof t.cls_odd_bits);
    for (int m = 0; m < 16; m++) t.shell_inv_norm[m] = (m >= 2 && m <= 12) ? (float)(1.0 / (4.0 * std::sqrt((double)m))) : 0.f;
    t.cls_block.assign(kClassSlots, HostTables::BlockConst{0.f, 0});
    for (size_t c = 0; c < all.size(); c++) {
        t.cls_shell_nibbles[c >> 3] |= (uint32_t)all[c].shell << (4 * (c & 7));
        if (all[c].odd) t.cls_odd_bits[c >> 5] |= 1u << (c & 31);
        t.cls_block[c] = HostTables::BlockConst{t.shell_inv_norm[all[c].shell], (all[c].odd ? 1 : 0) - 16};
    }
    t.base[all.size()] = running;
    t.num_points = running;
    return t.num_classes == 301 && t.num_points == 111043117458000ull;
}

}  // namespace llvq
