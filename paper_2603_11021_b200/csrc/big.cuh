// Dequantizer for codes whose class tables do not fit shared memory (the 72-bit code: 114 976 classes, up to
// seven unranking steps and nine distinct values per class).  The class-independent tables (Golay, Pascal and the
// reciprocals of its entries, 14-slot subsets, small subsets, deposit) are served from shared memory as on the fast
// path; class offsets and the 32-byte class records are read from global memory (they stay in L2).  Produces the point
// as bit planes of value ids, like the fast path.
#pragma once
#include "decode.cuh"
#include "fast.cuh"

namespace llvq {

// S2: class of index (hi:lo) < N: bucket table on the top 16 bits, then bisection between the classes of this
// bucket's and the next bucket's first index.
__device__ __forceinline__ int big_find_class(const DevCode& dc, uint64_t lo, uint64_t hi, uint64_t& local)
{
    const int sh = dc.W > 16 ? dc.W - 16 : 0;
    const uint32_t bucket = (uint32_t)(sh >= 64 ? hi >> (sh - 64) : (sh ? (lo >> sh) | (hi << (64 - sh)) : lo)) & 0xffffu;
    int a = (int)__ldg(dc.lut16 + bucket), b = (int)__ldg(dc.lut16 + bucket + 1);
    while (a < b) {
        const int mid = (a + b + 1) >> 1;
        const uint64_t ol = __ldg(dc.off_lo + mid);
        const uint64_t oh = __ldg(dc.off_hi + mid);
        if (oh < hi || (oh == hi && ol <= lo)) a = mid; else b = mid - 1;
    }
    local = lo - __ldg(dc.off_lo + a);                   // class sizes fit 63 bits: the difference is exact mod 2^64
    return a;
}

// Result of the table-driven decoder below: the planes of the fast path plus a fourth one, set where the value id is 8
// (classes with nine distinct values or odd classes with eight; rare), and that value.
struct DecodedBig {
    Decoded d;
    uint32_t p3;
    uint32_t val8;
};

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ uint64_t lds_u64(uint32_t addr)
{
    uint64_t v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}

// S3-S6 for any class of a code whose class tables live in global memory, in the manner of fast_decode_local: the class
// record is 32 bytes (BigDesc), the radix of a step is C(free slots, k) from the Pascal triangle in shared memory, its
// reciprocal comes from the tables beside it (64-bit while the arrangement rank needs it, 32-bit afterwards), steps that
// take at most three slots are one lookup in the table of small subsets, and the point comes out as bit planes of value
// ids.  All lanes of `mask` call this together; writes `out` only where `valid` (the caller presets it).
// The class record arrives in registers (h0, h1 = its two 16-byte halves; zeros where !valid), so that a caller can
// request it well before the block's turn.
__device__ __forceinline__ void big_decode_record(const FastSmem& T, const uint4 h0, const uint4 h1, uint64_t local, bool valid, uint32_t mask,
                                                  DecodedBig& out)
{
    const uint32_t w = h0.x & 0xff, B = (h0.x >> 8) & 0xff, flags = (h0.x >> 16) & 0xff;
    const uint32_t nlev1 = (h0.x >> 24) & 0xf, nlev = h0.x >> 28;
    const uint32_t goff = h0.y & 0xffff, A = h0.y >> 16;
    const uint32_t lvl_bit1 = (h1.z >> 8) & 0xff, lvl_nz = (h1.z >> 16) & 0xff;
    const bool odd = (flags & 1u) != 0u;

    // S3: r fastest, then the sign word s, then the arrangement rank p
    uint64_t q = local;
    uint32_t r = 0;
    if (A == 4096u) { r = (uint32_t)local & 4095u; q = local >> 12; }
    else if (A > 1u) {                                   // 759 or 2576 codewords of weight 8 / 16 or 12
        const uint64_t magic = A == 759u ? 0xffffffffffffffffull / 759u : 0xffffffffffffffffull / 2576u;
        q = __umul64hi(local, magic);
        uint64_t rem = local - q * A;
        if (rem >= A) { rem -= A; ++q; }
        r = (uint32_t)rem;
    }
    const uint32_t s = (uint32_t)q & ((1u << B) - 1u);
    uint64_t p = q >> B;

    // S4: Golay codeword
    const uint32_t c = T.golay[goff + r];

    // S5: arrangement.  Group 1 on F1(c), then group 0 on F0(c) (odd classes: one group 0 on all positions).
    const uint32_t F1 = odd ? 0u : c;
    const uint32_t F0 = ~F1 & 0xffffffu;
    uint32_t freem = F1, nfree = odd ? 0u : w;
    bool in_group0 = false;
    uint32_t p0 = 0, p1 = 0, p2 = 0, p3 = 0, bit1 = 0, nz0 = 0;
    const uint32_t pascal_a = smem_addr(T.pascal), r64_a = smem_addr(T.recip64), r32_a = smem_addr(T.recip32);
    const int maxlev = __reduce_max_sync(mask, nlev);
#pragma unroll
    for (int l = 0; l < kMaxLevels - 1; ++l) {
        if (l < maxlev) {
            if (!in_group0 && (uint32_t)l >= nlev1) {               // group 1 done: its filler gets id 1
                p0 |= freem;
                if (flags & 8u) bit1 |= freem;
                freem = F0; nfree = 24u - (odd ? 0u : w); in_group0 = true;
            }
            const bool active = (uint32_t)l < nlev;
            const uint32_t k = active ? ((l < 4 ? h1.x : h1.y) >> (8 * (l & 3))) & 0xffu : 0u;
            const uint32_t cell = nfree * 25u + k;                  // C(nfree, k) and its reciprocals
            const uint32_t radix = lds_u32(pascal_a + cell * 4u);
            uint32_t rho = 0u;
            if (l + 1 == maxlev) {
                // the last step of the warp: what is left of the rank is the step's own digit (a lane without this step holds 0
                // and places the empty subset), no division
                rho = (uint32_t)p;
            } else if (__any_sync(mask, (uint32_t)(p >> 32) != 0u)) {
                const uint64_t qq0 = __umul64hi(p, lds_u64(r64_a + cell * 8u));
                uint64_t qq = qq0, rem = p - qq * radix;
                if (rem >= radix) { rem -= radix; ++qq; }
                if (active) { p = qq; rho = (uint32_t)rem; }
            } else {
                const uint32_t p32 = (uint32_t)p;
                uint32_t qq = __umulhi(p32, lds_u32(r32_a + cell * 4u));
                uint32_t rem = p32 - qq * radix;
                if (rem >= radix) { rem -= radix; ++qq; }
                if (active) { p = qq; rho = rem; }
            }
            uint32_t rel;
            if (T.sub3 != 0u && __all_sync(mask, k <= (uint32_t)kSmallSubsetMaxK)) rel = small_subset(T, k, rho);
            else rel = nth_subset(T, k, rho, (int)__reduce_max_sync(mask, active ? nfree : 0u));
            const uint32_t a = deposit24(T.pd6, rel, freem);
            freem ^= a; nfree -= k;
            if ((l + 2) & 1) p0 |= a;                               // id of level l is l + 2
            if ((l + 2) & 2) p1 |= a;
            if ((l + 2) & 4) p2 |= a;
            if ((l + 2) & 8) p3 |= a;
            if ((lvl_bit1 >> l) & 1u) bit1 |= a;
            if (in_group0 && ((lvl_nz >> l) & 1u)) nz0 |= a;
        }
    }
    if (!in_group0) {
        p0 |= freem;
        if (flags & 8u) bit1 |= freem;
        freem = F0;
    }
    if (flags & 16u) bit1 |= freem;                                 // filler of group 0 keeps id 0
    if (flags & 4u) nz0 |= freem;

    // S6: signs
    uint32_t neg;
    if (__all_sync(mask, odd)) neg = c ^ bit1;                      // 1 mod 4 on F0, 3 mod 4 on F1
    else {
        // the bits of s go to the positions that carry a sign (F1 and the nonzero ones of F0) in ascending order, except the
        // last F1 position: its sign makes the sum 0 mod 8
        const uint32_t last_f1 = F1 ? 0x80000000u >> __clz(F1) : 0u;
        uint32_t neg_even = deposit24(T.pd6, s, (F1 | (odd ? 0u : nz0)) & ~last_f1);
        if ((__popc(neg_even & F1) + (flags >> 1)) & 1u) neg_even |= last_f1;
        neg = odd ? (c ^ bit1) : neg_even;
    }
    if (valid) {
        out.d.p0 = p0; out.d.p1 = p1; out.d.p2 = p2; out.d.neg = neg;
        out.d.vals_lo = h0.z; out.d.vals_hi = h0.w;
        out.p3 = p3; out.val8 = h1.z & 0xffu;
    }
}

// The 32-byte record of class `cls` (zeros where !valid), read from global memory / L2.  The loads are volatile
// statements: they stay where the caller put them relative to its other volatile statements (the table reads of the decoder).
__device__ __forceinline__ void big_load_record(const DevCode& dc, int cls, bool valid, uint4& h0, uint4& h1)
{
    h0 = h1 = make_uint4(0u, 0u, 0u, 0u);
    if (valid) {
        const BigDesc* rec = dc.big + cls;
        asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(h0.x), "=r"(h0.y), "=r"(h0.z), "=r"(h0.w) : "l"(rec));
        asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4+16];" : "=r"(h1.x), "=r"(h1.y), "=r"(h1.z), "=r"(h1.w) : "l"(rec));
    }
}

__device__ __forceinline__ void big_decode_planes(const FastSmem& T, const DevCode& dc, int cls, uint64_t local, bool valid, uint32_t mask,
                                                  DecodedBig& out)
{
    uint4 h0, h1;
    big_load_record(dc, cls, valid, h0, h1);
    big_decode_record(T, h0, h1, local, valid, mask, out);
}

// Where the fourth plane is set the value id is 8: put bf16(gain * val8), signed, over what the three-plane expansion
// left there.  All lanes of the warp call this together.
__device__ __forceinline__ void patch_id8_bf16(const DecodedBig& b, float gain, uint32_t w[12])
{
    if (!__any_sync(kFullMask, b.p3 != 0u)) return;
    const uint32_t v = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(gain * (float)b.val8));
#pragma unroll
    for (int j = 0; j < 12; ++j) {
        const uint32_t lo = (b.p3 >> (2 * j)) & 1u, hi = (b.p3 >> (2 * j + 1)) & 1u;
        const uint32_t m = (lo ? 0xffffu : 0u) | (hi ? 0xffff0000u : 0u);
        const uint32_t sg = (((b.d.neg >> (2 * j)) & 1u) << 15) | (((b.d.neg >> (2 * j + 1)) & 1u) << 31);
        w[j] = (w[j] & ~m) | (((v | v << 16) ^ sg) & m);
    }
}

__device__ __forceinline__ void patch_id8_bytes(const DecodedBig& b, uint32_t out[6])
{
    if (!__any_sync(kFullMask, b.p3 != 0u)) return;
#pragma unroll
    for (int i = 0; i < 24; ++i) {
        if ((b.p3 >> i) & 1u) {
            const uint32_t byte = ((b.d.neg >> i) & 1u) ? (0u - b.val8) & 0xffu : b.val8;
            out[i >> 2] = (out[i >> 2] & ~(0xffu << (8 * (i & 3)))) | byte << (8 * (i & 3));
        }
    }
}

}  // namespace llvq
