// Host-side table generator of the LLVQ library: Golay codewords, class list
// with cardinalities and offsets, per-class unranking descriptors.
// Written independently of the test oracle; the two are compared in the tests.
#pragma once
#include <cstdint>
#include <vector>

namespace llvq {

typedef unsigned __int128 u128;

constexpr int kDim = 24;
constexpr int kMaxLevels = 8;

// One "choose k of the slots still free" step of the arrangement unranking
// (App. A step 4).  magic = floor((2^64 - 1) / radix) for division by multiply-high.
struct LevelDesc {
    uint32_t radix;   // C(n, k)
    uint8_t k;        // slots taken by this value
    uint8_t val;      // absolute value placed
    uint8_t n;        // slots free before this step
    uint8_t pad;
    uint64_t magic;
};
static_assert(sizeof(LevelDesc) == 16, "LevelDesc layout");

// Everything the kernels need to rebuild a point of one class from its
// class-local index (App. A steps 3-4).  Group 1 = positions F1(c) (values
// = 2 mod 4 of an even class); group 0 = positions F0(c) of an even class, or
// all 24 positions of an odd class.
struct ClassDesc {
    uint8_t parity;    // 0 even, 1 odd
    uint8_t w;         // even: Golay weight required (= #coordinates 2 mod 4)
    uint8_t B;         // free sign bits
    uint8_t signpar;   // even: (#values 4 mod 8 + #values 6 mod 8) & 1
    uint8_t nlev1;     // unranking steps in group 1
    uint8_t nlev0;     // unranking steps in group 0
    uint8_t fill1;     // value filling the rest of group 1 (unused if w == 0)
    uint8_t fill0;     // value filling the rest of group 0
    uint16_t goff;     // first admissible codeword in the sorted Golay table
    uint16_t A;        // number of admissible codewords
    uint32_t m;        // shell
    uint64_t magicA;   // floor((2^64 - 1) / A)
    uint64_t reserved;
    LevelDesc lev[kMaxLevels];   // group-1 steps first, then group-0 steps
};
static_assert(sizeof(ClassDesc) == 32 + 16 * kMaxLevels, "ClassDesc layout");

struct ClassInfo {           // host-only description, for queries and tests
    int m, parity, w, B;
    uint64_t A;
    u128 card, offset;
    std::vector<int> values, mults;   // distinct absolute values descending
};

struct HostTables {
    int m_lo = 0, m_hi = 0, W = 0;
    u128 N = 0;
    std::vector<uint32_t> golay;          // 4096 words sorted by (weight, value)
    int woff[25] = {0}, wcnt[25] = {0};
    std::vector<ClassInfo> info;
    std::vector<ClassDesc> desc;
    std::vector<u128> offset;             // nclasses + 1 entries, offset[nclasses] = N
    uint32_t pascal[25 * 25] = {0};       // C(n, k) at [n * 25 + k]
    int max_levels = 0;
};

// Returns false if the code is outside what the kernels support.
bool build_tables(int m_lo, int m_hi, HostTables& out);

}  // namespace llvq
