// Dequantizer for codes whose class tables do not fit shared memory (the 72-bit code: 114 976 classes, up to
// seven unranking steps and nine distinct values per class).  The class-independent tables (Golay, Pascal,
// 14-slot subsets, deposit) are served from shared memory as on the fast path; class offsets and descriptors
// are read from global memory (they stay in L2).  Produces the point as 24 signed bytes.
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

// S3-S6 for any class of any supported code.  All 32 lanes of the warp call this together.
__device__ __forceinline__ void big_decode_local(const FastSmem& T, const DevCode& dc, int cls, uint64_t local, bool valid, Point& pt)
{
    const uint4* cd = reinterpret_cast<const uint4*>(dc.cls + (valid ? cls : 0));
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    const uint4 h0 = valid ? __ldg(cd) : zero4, h1 = valid ? __ldg(cd + 1) : zero4;
    const uint32_t parity = h0.x & 0xff, w = (h0.x >> 8) & 0xff, B = (h0.x >> 16) & 0xff, signpar = h0.x >> 24;
    const uint32_t nlev1 = h0.y & 0xff, nlev0 = (h0.y >> 8) & 0xff, fill1 = (h0.y >> 16) & 0xff, fill0 = h0.y >> 24;
    const uint32_t goff = h0.z & 0xffff, A = h0.z >> 16;
    const uint32_t nlev = nlev1 + nlev0;

    // S3: r fastest, then the sign word s, then the arrangement rank p
    uint64_t q = local;
    uint32_t r = 0;
    if (A == 4096u) { r = (uint32_t)local & 4095u; q = local >> 12; }
    else if (A > 1u) divmod_magic(local, A, ((uint64_t)h1.y << 32) | h1.x, q, r);
    const uint32_t s = (uint32_t)q & ((1u << B) - 1u);
    uint64_t p = q >> B;

    // S4: Golay codeword
    const uint32_t c = T.golay[goff + r];

    // S5: arrangement.  Group 1 on F1(c), then group 0 on F0(c) (odd classes: one group 0 on all positions).
    const bool odd = parity != 0u;
    const uint32_t F1 = odd ? 0u : c;
    const uint32_t F0 = ~F1 & 0xffffffu;
    uint32_t freem = F1;
    bool in_group0 = false;
    uint32_t bit1 = 0, nz0 = 0;
#pragma unroll
    for (int i = 0; i < 6; ++i) pt.w[i] = 0u;
    const int maxlev = __reduce_max_sync(kFullMask, nlev);
    for (int l = 0; l < maxlev; ++l) {
        if (!in_group0 && (uint32_t)l >= nlev1) {               // group 1 done: its last value fills what is left of F1
            place_value(pt, freem, fill1);
            if (fill1 & 2u) bit1 |= freem;
            freem = F0; in_group0 = true;
        }
        const bool active = (uint32_t)l < nlev;
        const uint4 L = active ? __ldg(cd + 2 + l) : zero4;
        const uint32_t k = L.y & 0xff, val = (L.y >> 8) & 0xff, n = (L.y >> 16) & 0xff;
        uint32_t rho = 0;
        if (active) {
            if ((p >> 32) == 0ull) {
                // the rank has shrunk to 32 bits (it only ever gets smaller): the high word of the 64-bit magic,
                // floor(2^32 / d) or one less, gives an estimate at most two too small
                const uint32_t p32 = (uint32_t)p;
                uint32_t q32 = __umulhi(p32, L.w);
                uint32_t r32 = p32 - q32 * L.x;
                if (r32 >= L.x) { r32 -= L.x; ++q32; }
                if (r32 >= L.x) { r32 -= L.x; ++q32; }
                rho = r32; p = q32;
            } else {
                uint64_t pq;
                divmod_magic(p, L.x, ((uint64_t)L.w << 32) | L.z, pq, rho);
                p = pq;
            }
        }
        const int top = __reduce_max_sync(kFullMask, n);
        const uint32_t rel = nth_subset(T, k, rho, top);
        const uint32_t a = deposit24(T.pd6, rel, freem);
        freem ^= a;
        place_value(pt, a, val);
        if (val & 2u) bit1 |= a;
        if (in_group0 && val) nz0 |= a;
    }
    if (!in_group0) {
        place_value(pt, freem, fill1);
        if (fill1 & 2u) bit1 |= freem;
        freem = F0;
    }
    place_value(pt, freem, fill0);
    if (fill0 & 2u) bit1 |= freem;
    if (fill0) nz0 |= freem;

    // S6: signs
    const uint32_t nf1 = w ? w - 1u : 0u;                       // free sign bits on F1
    const uint32_t s1 = s & ((1u << nf1) - 1u);
    const uint32_t src1 = s1 | (((__popc(s1) + signpar) & 1u) << nf1);     // last F1 position: sum = 0 mod 8
    const uint32_t neg_even = deposit24(T.pd6, src1, F1) | deposit24(T.pd6, s >> nf1, odd ? 0u : nz0);
    negate_at(pt, valid ? (odd ? (c ^ bit1) : neg_even) : 0u);
}

}  // namespace llvq
