// Device-side dequantizer: stored index field -> integer Leech-lattice point
// (App. A steps 1-4), one thread per block of 24 weights.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tables.h"

namespace llvq {

// Device view of one code's tables (all pointers are device memory owned by the context).
struct DevCode {
    const uint32_t* golay;          // [4096]
    const ClassDesc* cls;           // [nclasses]
    const uint64_t* off_lo;         // [nclasses + 1] low 64 bits of the class offsets
    const uint32_t* off_hi;         // [nclasses + 1] bits 64.. of the class offsets (W > 64 only)
    const uint32_t* pascal;         // [25 * 25]
    unsigned long long* bad_index;  // device counter of fields with I >= N
    uint32_t* flags;                // device error flags
    uint64_t n_lo, n_hi;            // N
    int nclasses;
    int W;
};

// A decoded point: 24 signed bytes, coordinate i in byte (i & 3) of word (i >> 2).
struct Point { uint32_t w[6]; };

// ---- S1: bit unpack --------------------------------------------------------
// Field b occupies stream bits [b*W, (b+1)*W).  Reads only the 32-bit words the field touches.
__device__ __forceinline__ void load_index(const uint32_t* __restrict__ s, uint64_t b, int W, uint64_t& lo, uint64_t& hi)
{
    uint64_t bp = b * (uint64_t)W;
    uint64_t wi = bp >> 5;
    int sh = (int)(bp & 31);
    int nw = (sh + W + 31) >> 5;                        // 1..4 words
    uint32_t w0 = __ldg(s + wi);
    uint32_t w1 = nw > 1 ? __ldg(s + wi + 1) : 0u;
    uint32_t w2 = nw > 2 ? __ldg(s + wi + 2) : 0u;
    uint32_t w3 = nw > 3 ? __ldg(s + wi + 3) : 0u;
    uint64_t a = ((uint64_t)w1 << 32) | w0, c = ((uint64_t)w3 << 32) | w2;
    if (sh) { lo = (a >> sh) | (c << (64 - sh)); hi = c >> sh; }
    else    { lo = a; hi = c; }
    if (W < 64) { lo &= (1ull << W) - 1; hi = 0; }
    else if (W == 64) hi = 0;
    else hi &= (1ull << (W - 64)) - 1;
}

// ---- S2: class lookup ------------------------------------------------------
// Largest j with offset[j] <= I; I < N is guaranteed by the caller.
__device__ __forceinline__ int find_class(const DevCode& dc, uint64_t lo, uint64_t hi, uint64_t& local)
{
    int a = 0, b = dc.nclasses - 1;
    if (dc.W <= 64) {
        while (a < b) {
            int mid = (a + b + 1) >> 1;
            if (__ldg(dc.off_lo + mid) <= lo) a = mid; else b = mid - 1;
        }
        local = lo - __ldg(dc.off_lo + a);
    } else {
        while (a < b) {
            int mid = (a + b + 1) >> 1;
            uint64_t ol = __ldg(dc.off_lo + mid); uint64_t oh = __ldg(dc.off_hi + mid);
            bool le = oh < hi || (oh == hi && ol <= lo);
            if (le) a = mid; else b = mid - 1;
        }
        local = lo - __ldg(dc.off_lo + a);            // class sizes fit 63 bits: the difference is exact mod 2^64
    }
    return a;
}

// q = p / d, r = p % d with magic = floor((2^64 - 1) / d): the estimate is at most one too small.
__device__ __forceinline__ void divmod_magic(uint64_t p, uint32_t d, uint64_t magic, uint64_t& q, uint32_t& r)
{
    q = __umul64hi(p, magic);
    uint64_t rem = p - q * d;
    if (rem >= d) { rem -= d; ++q; }
    r = (uint32_t)rem;
}

// ---- S5 helpers ------------------------------------------------------------
// The rho-th k-subset of {0..n-1} in combinatorial-number-system order, as a bit mask.
__device__ __forceinline__ uint32_t nth_subset(const uint32_t* __restrict__ pascal, int n, int k, uint32_t rho)
{
    uint32_t m = 0;
    int e = n;
    for (int t = k; t >= 1; --t) {
        uint32_t c;
        do { --e; c = __ldg(pascal + e * 25 + t); } while (c > rho);
        rho -= c;
        m |= 1u << e;
    }
    return m;
}

// Deposit the low bits of src into the set positions of mask, lowest first.
__device__ __forceinline__ uint32_t deposit_bits(uint32_t src, uint32_t mask)
{
    uint32_t out = 0;
    while (mask) {
        uint32_t low = mask & (0u - mask);
        if (src & 1u) out |= low;
        src >>= 1;
        mask ^= low;
    }
    return out;
}

// 4 mask bits -> 4 bytes holding 0 or 1.
__device__ __forceinline__ uint32_t spread4(uint32_t nib) { return (nib * 0x00204081u) & 0x01010101u; }

__device__ __forceinline__ void place_value(Point& pt, uint32_t mask, uint32_t val)
{
#pragma unroll
    for (int i = 0; i < 6; ++i) pt.w[i] += spread4((mask >> (4 * i)) & 15u) * val;
}

// ---- S3-S6: class-local index -> point --------------------------------------
__device__ __forceinline__ void decode_local(const DevCode& dc, int cls, uint64_t local, Point& pt)
{
    const uint4* cd = reinterpret_cast<const uint4*>(dc.cls + cls);
    uint4 h0 = __ldg(cd), h1 = __ldg(cd + 1);
    const uint32_t parity = h0.x & 0xff, w = (h0.x >> 8) & 0xff, B = (h0.x >> 16) & 0xff, signpar = h0.x >> 24;
    const uint32_t nlev1 = h0.y & 0xff, nlev0 = (h0.y >> 8) & 0xff, fill1 = (h0.y >> 16) & 0xff, fill0 = h0.y >> 24;
    const uint32_t goff = h0.z & 0xffff, A = h0.z >> 16;
    const uint64_t magicA = ((uint64_t)h1.y << 32) | h1.x;

    // S3: r fastest, then the sign word s, then the arrangement rank p
    uint64_t q; uint32_t r;
    if (A == 4096) { r = (uint32_t)local & 4095u; q = local >> 12; }
    else if (A == 1) { r = 0; q = local; }
    else divmod_magic(local, A, magicA, q, r);
    const uint32_t s = (uint32_t)q & ((1u << B) - 1u);
    uint64_t p = q >> B;

    // S4: Golay codeword
    const uint32_t c = __ldg(dc.golay + goff + r);

    // S5: arrangement.  Group 1 on F1(c), then group 0 on F0(c) (odd classes: one group on all positions).
#pragma unroll
    for (int i = 0; i < 6; ++i) pt.w[i] = 0;
    uint32_t bit1 = 0;                                 // positions whose absolute value has bit 1 set
    uint32_t nz0 = 0;                                  // nonzero positions of group 0
    uint32_t lev = 0;
    for (int group = 1; group >= 0; --group) {
        uint32_t freem = parity ? (group ? 0u : 0xFFFFFFu) : (group ? c : (~c & 0xFFFFFFu));
        const uint32_t nl = group ? nlev1 : nlev0;
        for (uint32_t i = 0; i < nl; ++i, ++lev) {
            uint4 L = __ldg(cd + 2 + lev);
            const uint32_t radix = L.x, k = L.y & 0xff, val = (L.y >> 8) & 0xff, n = (L.y >> 16) & 0xff;
            uint64_t pq; uint32_t rho;
            divmod_magic(p, radix, ((uint64_t)L.w << 32) | L.z, pq, rho);
            p = pq;
            uint32_t rel = nth_subset(dc.pascal, (int)n, (int)k, rho);
            uint32_t abs = deposit_bits(rel, freem);
            freem ^= abs;
            place_value(pt, abs, val);
            if (val & 2u) bit1 |= abs;
            if (!group) nz0 |= abs;
        }
        const uint32_t fill = group ? fill1 : fill0;
        place_value(pt, freem, fill);
        if (fill & 2u) bit1 |= freem;
        if (!group && fill) nz0 |= freem;
    }

    // S6: signs
    uint32_t neg;
    if (parity) {
        neg = c ^ bit1;                                // x_i = 1 mod 4 on F0, 3 mod 4 on F1
    } else {
        uint32_t nf1 = w ? w - 1u : 0u;                // free sign bits on F1
        uint32_t s1 = s & ((1u << nf1) - 1u);
        neg = deposit_bits(s1, c);
        if (w && ((__popc(s1) + signpar) & 1u)) neg |= 1u << (31 - __clz(c));   // last F1 position: sum = 0 mod 8
        neg |= deposit_bits(s >> nf1, nz0);
    }
#pragma unroll
    for (int i = 0; i < 6; ++i) {
        uint32_t sm = spread4((neg >> (4 * i)) & 15u);
        pt.w[i] = (pt.w[i] ^ (sm * 0xFFu)) + sm;        // bytewise negate; negated bytes are never zero
    }
}

// Full dequantizer for field b of a stream.  Invalid fields give the zero point and are counted.
__device__ __forceinline__ void decode_field(const DevCode& dc, const uint32_t* __restrict__ stream, uint64_t b, Point& pt)
{
    uint64_t lo, hi;
    load_index(stream, b, dc.W, lo, hi);
    if (hi > dc.n_hi || (hi == dc.n_hi && lo >= dc.n_lo)) {
#pragma unroll
        for (int i = 0; i < 6; ++i) pt.w[i] = 0;
        atomicAdd(dc.bad_index, 1ull);
        return;
    }
    uint64_t local;
    int cls = find_class(dc, lo, hi, local);
    decode_local(dc, cls, local, pt);
}

// ---- S7: gain ---------------------------------------------------------------
// bf16_rn(float(gain) * float(x)): the product is exact in binary32, one rounding.
__device__ __forceinline__ float coord(const Point& pt, int i)
{
    return (float)(int)(int8_t)(pt.w[i >> 2] >> (8 * (i & 3)));
}

__device__ __forceinline__ __nv_bfloat16 dequant(float gain, const Point& pt, int i)
{
    return __float2bfloat16_rn(gain * coord(pt, i));
}

__device__ __forceinline__ float gain_to_float(uint16_t bits)
{
    return __half2float(__ushort_as_half(bits));
}

}  // namespace llvq
