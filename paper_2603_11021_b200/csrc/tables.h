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

// Compact form of ClassDesc for the codes whose class tables stay in global memory (32 bytes, two 16-byte loads): the
// radix of a step is C(free slots, k) from the Pascal triangle in shared memory and its reciprocals come from two tables
// beside it, so only the multiplicities and the values are stored per class.  Value ids: 0 = filler of group 0,
// 1 = filler of group 1, 2 + l = level l.
struct BigDesc {
    uint8_t w, B;
    uint8_t flags;         // bit0 parity, bit1 signpar, bit2 fill0 is nonzero, bit3 fill1 has value bit 1, bit4 fill0 has value bit 1
    uint8_t nlev;          // nlev1 | (nlev1 + nlev0) << 4
    uint16_t goff, A;
    uint8_t val[8];        // absolute value of ids 0..7
    uint8_t k[8];          // slots taken by level 0..7 (bytes 7 unused: at most 7 levels)
    uint8_t val8;          // absolute value of id 8 (classes with 9 distinct values)
    uint8_t lvl_bit1;      // bit l: the value of level l has value bit 1 (= 2 or 3 mod 4)
    uint8_t lvl_nz;        // bit l: the value of level l is nonzero
    uint8_t small_k;       // bit l: level l takes at most kSmallSubsetMaxK slots (part of the sorted layouts' key)
    uint32_t pad;
};
static_assert(sizeof(BigDesc) == 32, "BigDesc layout");

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

// ---------------------------------------------------------------------------
// Shared-memory table image for codes with few classes ("fast path"): one
// contiguous blob, copied into every CTA's shared memory by bulk copies.
// ---------------------------------------------------------------------------
namespace llvq {

constexpr int kFastMaxLevels = 4;      // unranking steps per class on the fast path
constexpr int kFastDescWords = 20;     // words of a class descriptor that carry data
constexpr int kFastDescValsOdd = 18;   // words 18, 19: absolute value of id 0..7 in the numbering of the odd-only decoder form
constexpr int kFastDescRnorm = 16;     // word holding 1 / sqrt(16 m) as binary32
constexpr int kFastDescMagic0 = 17;    // word holding floor(2^32 / radix) of level 0 (used when the arrangement rank fits 32 bits)
constexpr uint32_t kFastFlagRank32 = 32u;   // descriptor flag: the class has fewer than 2^32 arrangements
constexpr int kSmallSubsetMaxK = 3;    // the table of all k-subsets of 24 slots covers k = 0..3
constexpr int kSmallSubsetWords = 4 + 1 + 24 + 276 + 2024;   // [first entry of k = 0..3][the subsets, by k, each group in numeric order]
constexpr int kFastDescStride = 20;    // words between descriptors: 80 bytes spread consecutive classes over all bank groups
constexpr int kLowBits = 14;           // slots resolved by one table lookup in the subset unranking


// Byte offsets of the parts of the image (all 16-byte aligned) and scalars the kernels need.
struct FastLayout {
    uint32_t golay;       // u32[4096]
    uint32_t lut;         // u16[4096]  class of the first index of bucket (I >> lut_shift)
    uint32_t pascal;      // u32[25*25]
    uint32_t base14;      // u32[16]: [k] = first entry of the k-subsets of 14 slots in r14
    uint32_t r14;         // u16[16384]: the k-subsets of 14 slots as bit masks, k = 0..14, each in numeric order
    uint32_t pd6;         // u8[4096]: [f << 6 | s] = low bits of s deposited into the set bits of f
    uint32_t off;         // u64[ncls + 1]
    uint32_t desc;        // u32[ncls][kFastDescStride]
    uint32_t total;       // bytes of the image proper, multiple of 16
    uint32_t recip64;     // u64[25*25] floor((2^64 - 1) / C(n, k)) and
    uint32_t recip32;     // u32[25*25] floor(2^32 / C(n, k)) (0xffffffff for C = 1): images without class tables only, else 0
    uint32_t sub3;        // u32[kSmallSubsetWords], behind the image proper: kernels with room for it load total_ext bytes
    uint32_t total_ext;   // bytes including sub3, multiple of 16
    uint32_t lut_shift;
    uint32_t ncls;
    uint32_t W;
};

// Word layout of a fast descriptor:
//  0: w | B << 8 | flags << 16 | nlev1 << 24 | nlev << 28
//       flags: bit0 parity, bit1 signpar, bit2 fill0 is nonzero, bit3 fill1 has value bit 1, bit4 fill0 has value bit 1,
//              bit5 the arrangement rank of the class fits 32 bits, bits 6-7 decoder form (0 even with weight 8 / 12 / 16, 1 odd, 2 other)
//  1: goff | A << 16
//  2,3: magicA = floor((2^64-1)/A)
//  4,5: absolute value of id 0..7 (one byte each): id 0 = fill0, id 1 = fill1, ids 2.. = levels in order
//  6,7: magic of level 0 = floor((2^64-1)/radix0)
//  8..11: level l: radix | k << 22 | id << 27 | (value bit 1) << 30 | (value nonzero) << 31; steps the class does not have:
//         radix 1, k 0, reciprocals 0xffffffff (dividing by them leaves the rank unchanged and gives remainder 0)
//  12..14: floor(2^32 / radix) of levels 1..3
//  15: n (free slots before the step) of levels 0..3, one byte each
//  16: binary32 bits of 1 / |x| = 1 / sqrt(16 m) (formed in binary64, rounded once), for the shape-gain form
//  17: floor(2^32 / radix) of level 0
//  18,19: odd classes: absolute value of id 0..7 with id 0 = fill0 and ids 1.. = levels in order (the form that decodes odd
//         classes alone numbers the levels from 1: there is no group 1 whose filler would take id 1)
// with_classes = false builds only the class-independent tables (Golay, Pascal, subsets, deposit): codes whose class
// tables do not fit shared memory keep those in global memory.
bool build_fast_image(const HostTables& t, FastLayout& layout, std::vector<uint8_t>& image, bool with_classes = true);
void build_big_descs(const HostTables& t, std::vector<BigDesc>& out);
void build_bucket_table(const HostTables& t, std::vector<uint32_t>& lut);   // u32[65537], see tables.cpp

// Encoder side (point -> class).  Signature of a class: sum over its 24 absolute values of a fixed pseudo-random
// 64-bit number per value (the multiset fixes shell and parity).  build_class_hash() fills an open-addressing
// table (linear probing from (signature >> 20) & (size - 1), key 0 = empty) and returns false if two classes of the
// code share a signature.
uint64_t sig_of_value(int a);
bool build_class_hash(const HostTables& t, std::vector<uint64_t>& keys, std::vector<uint32_t>& cls);

}  // namespace llvq
