// Host-side construction of the tables the CUDA kernels read: the class list of the ball
// Lambda24(12) with its index bases (paper Sec. 2.1), the extended Golay code in the two orders
// the index uses, and the per-class constants of the GEMV (paper Sec. 2.3: the unit-direction
// normalisation is a per-class constant).
#pragma once
#include <cstdint>
#include <vector>

namespace llvq {

constexpr int kMaxShell = 12;
constexpr int kClassSlots = 512;       // a 9-bit id can never index out of bounds (Sec. 2.3)
constexpr int kEmptyClass = 511;       // record of a code that names no point
constexpr uint64_t kIndexBits = 47;

// What the expander needs to un-rank an index inside one class.  40 bytes.
struct ClassDesc {
    uint64_t perm_a;      // even: orderings of the support magnitudes; odd: orderings of all 24
    uint64_t perm_b;      // even: orderings of the off-support magnitudes; odd: 1
    uint8_t cnt[8];       // even: [0..3] copies of 2,6,10,14 on the support, [4..7] copies of
                          // 0,4,8,12 off it; odd: [0..6] copies of 1,3,..,13
    uint8_t odd, w, shell, sign_bits;   // sign_bits = free sign bits of the even type
    uint8_t nz_b, ndist, pad0, pad1;    // non-zero off-support entries; distinct magnitudes
    uint8_t dist[8];      // the distinct magnitudes, ascending (rank levels of the one-hot layout)
};
static_assert(sizeof(ClassDesc) == 40, "ClassDesc layout");

struct HostTables {
    int num_classes = 0;
    uint64_t num_points = 0;
    std::vector<uint64_t> base;            // num_classes + 1 entries
    std::vector<ClassDesc> desc;           // num_classes entries
    std::vector<uint32_t> golay_by_weight; // 4096 words sorted by (weight, value)
    int weight_offset[25];                 // first entry of each weight in golay_by_weight
    std::vector<uint32_t> golay_by_message;// word of message k = XOR of generator rows in k
    std::vector<float> cls_scale;          // kClassSlots: 2^21 / (4 sqrt(shell)), 0 if unused
    std::vector<uint32_t> cls_parity;      // kClassSlots: parity * 0x00080008
    // the class constants of the 14-byte GEMV, small enough to travel in kernel parameters
    // (x_i = 2 u_i + parity - 16, scale 1 / (4 sqrt(shell))):
    uint32_t cls_shell_nibbles[64];        // nibble c & 7 of word c >> 3: shell of class c (2..12), 0 if unused
    uint32_t cls_odd_bits[16];             // bit c & 31 of word c >> 5: class c is of the odd type
    float shell_inv_norm[16];              // [m] = 1 / (4 sqrt(m)) for m = 2..12, else 0
    struct BlockConst { float inv_norm; int32_t offset; };
    std::vector<BlockConst> cls_block;     // kClassSlots: {1 / (4 sqrt(shell)), parity - 16}; zeros if unused
    std::vector<float> cls_value;          // kClassSlots * 8: dist[l] / (4 sqrt(shell)), l < 5
    std::vector<uint8_t> cls_dist;         // kClassSlots * 8: dist[l]
};

// Returns false if an internal consistency check fails (class count, total, Golay weights).
bool build_tables(HostTables &t);

}  // namespace llvq
