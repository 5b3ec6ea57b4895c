// Fast dequantizer for codes whose tables fit in shared memory (few classes,
// indices up to 64 bits): App. A steps 1-4 with every table lookup served from
// shared memory, one thread per block of 24 weights.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tables.h"

namespace llvq {

constexpr uint32_t kFullMask = 0xffffffffu;
constexpr int kPascalToBase14 = 2512;     // byte distance from pascal[t] to base14[t] in the table image

// Pointers into the CTA's copy of the table image.
struct FastSmem {
    const uint32_t* golay;
    const uint16_t* lut;
    const uint32_t* pascal;
    const uint32_t* base14;
    const uint16_t* r14;
    const uint8_t* pd6;
    const uint64_t* off;
    const uint32_t* desc;
    const uint64_t* recip64;  // images without class tables: reciprocals of the Pascal entries
    const uint32_t* recip32;
    uint32_t sub3;            // shared-window byte address of the table of small subsets, 0 when the kernel did not load it
    uint32_t lut_shift;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// with_small_subsets: the kernel loaded L.total_ext bytes of the image, not only L.total
__device__ __forceinline__ FastSmem fast_view(const uint8_t* smem, const FastLayout& L, bool with_small_subsets = false)
{
    FastSmem T;
    T.golay = reinterpret_cast<const uint32_t*>(smem + L.golay);
    T.lut = reinterpret_cast<const uint16_t*>(smem + L.lut);
    T.pascal = reinterpret_cast<const uint32_t*>(smem + L.pascal);
    T.base14 = reinterpret_cast<const uint32_t*>(smem + L.base14);
    T.r14 = reinterpret_cast<const uint16_t*>(smem + L.r14);
    T.pd6 = smem + L.pd6;
    T.off = reinterpret_cast<const uint64_t*>(smem + L.off);
    T.desc = reinterpret_cast<const uint32_t*>(smem + L.desc);
    T.recip64 = reinterpret_cast<const uint64_t*>(smem + L.recip64);
    T.recip32 = reinterpret_cast<const uint32_t*>(smem + L.recip32);
    T.sub3 = with_small_subsets ? smem_addr(smem + L.sub3) : 0u;
    T.lut_shift = L.lut_shift;
    return T;
}

// Copy the table image into shared memory with bulk asynchronous copies (TMA,
// no multicast) tracked by one mbarrier.  Every thread of the CTA must call this.
// Returns false (for the whole CTA) if the copy did not complete within the
// wait limit; the error flag is then set and the caller must return.
__device__ __forceinline__ bool fast_load_image(uint8_t* dst, const uint8_t* __restrict__ src, uint32_t bytes,
                                                uint64_t* bar, uint32_t* err_flags)
{
    const uint32_t bar_a = smem_addr(bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
        constexpr uint32_t kChunk = 32768;
        for (uint32_t o = 0; o < bytes; o += kChunk) {
            uint32_t n = bytes - o < kChunk ? bytes - o : kChunk;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(dst + o)), "l"(src + o), "r"(n), "r"(bar_a) : "memory");
        }
    }
    uint32_t done = 0;
    for (uint32_t it = 0; it < (1u << 20) && !done; ++it) {
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar_a), "r"(0u) : "memory");
    }
    if (!done) {
        atomicOr(err_flags, 1u);
        // the copy may still be writing this CTA's shared memory: give it the same limit once more before the caller returns
        for (uint32_t it = 0; it < (1u << 20) && !done; ++it) {
            asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                         : "=r"(done) : "r"(bar_a), "r"(0u) : "memory");
        }
        done = 0;
    }
    return __syncthreads_and((int)done) != 0;
}

// Deposit the low bits of src into the set bits of mask, lowest first (24-bit masks, 6 bits per lookup).
// r = a * b + c on the multiply-add pipe (the logic pipe is the busy one: sums of disjoint bit fields go here)
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}

__device__ __forceinline__ uint32_t deposit24(const uint8_t* pd6, uint32_t src, uint32_t mask)
{
    // how many source bits the lower groups consume: known from the mask alone, so the four lookups are independent
    const uint32_t c1 = __popc(mask & 0x3fu), c2 = __popc(mask & 0xfffu), c3 = __popc(mask & 0x3ffffu);
    // row of a lookup = the group's 6 mask bits times 64: for groups 1..3 that is a masked (shifted) copy of the mask
    const uint32_t r0 = pd6[mad_u32(mask & 0x3fu, 64u, src & 63u)];
    const uint32_t r1 = pd6[(mask & 0xfc0u) + ((src >> c1) & 63u)];
    const uint32_t r2 = pd6[((mask >> 6) & 0xfc0u) + ((src >> c2) & 63u)];
    const uint32_t r3 = pd6[((mask >> 12) & 0xfc0u) + ((src >> c3) & 63u)];
    return mad_u32(r3, 1u << 18, mad_u32(r2, 1u << 12, mad_u32(r1, 64u, r0)));
}

template <int kOff>
__device__ __forceinline__ uint32_t lds_at(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(kOff));
    return v;
}

// One slot decision: take slot kPos iff at least C(kPos, t) subsets come before (t = elements still to place).
template <int kPos>
__device__ __forceinline__ void subset_step(uint32_t& col, uint32_t& rho, uint32_t& m, int top)
{
    if (kPos < top) {                                   // warp-uniform
        const uint32_t cnt = lds_at<kPos * 100>(col);   // C(kPos, t); column 0 is stored as 0xffffffff: never taken
        if (rho >= cnt) { rho -= cnt; m |= 1u << kPos; col -= 4u; }
    }
}

__device__ __forceinline__ uint32_t nth_subset(const FastSmem& T, uint32_t k, uint32_t rho, int top)
{
    static_assert(kLowBits == 14, "the slot decisions below cover slots 23..14");
    uint32_t m = 0;
    // byte address (shared window) of C(0, t); it walks down one column each time an element is taken
    uint32_t col = smem_addr(T.pascal) + k * 4u;
    subset_step<23>(col, rho, m, top); subset_step<22>(col, rho, m, top); subset_step<21>(col, rho, m, top);
    subset_step<20>(col, rho, m, top); subset_step<19>(col, rho, m, top); subset_step<18>(col, rho, m, top);
    subset_step<17>(col, rho, m, top); subset_step<16>(col, rho, m, top); subset_step<15>(col, rho, m, top);
    subset_step<14>(col, rho, m, top);
    const uint32_t first = lds_at<kPascalToBase14>(col);   // base14[t] sits right after the 625-entry Pascal table
    return m | (uint32_t)T.r14[first + rho];
}

// The rho-th k-subset of up to 24 slots for k <= 3: one lookup behind a four-word directory (T.sub3 != 0).
__device__ __forceinline__ uint32_t small_subset(const FastSmem& T, uint32_t k, uint32_t rho)
{
    uint32_t first, m;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(first) : "r"(T.sub3 + k * 4u));
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(m) : "r"(T.sub3 + (first + rho) * 4u));
    return m;
}

// Deposit into a mask that is 24 ones with at most two holes: open a gap at each hole, lowest first.
__device__ __forceinline__ uint32_t deposit_two_holes(uint32_t src, uint32_t mask)
{
    uint32_t holes = ~mask & 0xffffffu;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint32_t b = holes & (0u - holes);          // lowest hole, or 0: then nothing moves
        const uint32_t low = b - 1u;
        src = (src & low) | ((src & ~low) << 1);
        holes ^= b;
    }
    return src;
}

// Result of the index -> point map in a form the consumers expand cheaply:
// three bit planes giving each position a value id (0..7), the table of
// absolute values per id, and the mask of negative positions.
struct Decoded {
    uint32_t p0, p1, p2;
    uint32_t neg;
    uint32_t vals_lo, vals_hi;     // absolute value of id 0..3 / 4..7, one byte each
};

// S2: class of index I (< N) and its class-local index.
__device__ __forceinline__ uint32_t fast_find_class(const FastSmem& T, uint64_t I, uint64_t& local)
{
    uint32_t cls = T.lut[(uint32_t)(I >> T.lut_shift)];
    while (I >= T.off[cls + 1]) ++cls;
    local = I - T.off[cls];
    return cls;
}

// S3-S6.  `mask` = the lanes of the warp that call this together.  kPar = -1: any class.  kPar = 1: all calling lanes
// hold odd classes.  kPar = 0: all calling lanes hold even classes of Golay weight 8, 12 or 16 (both slot groups have
// at most 16 slots).  The specialised forms drop the work the other parity needs (slot decisions above 16, sign deposits).
// Writes d only where `valid`: the caller presets it (zeros for "no block").
template <int kPar>
__device__ __forceinline__ void fast_decode_local(const FastSmem& T, uint32_t cls, uint64_t local, bool valid, uint32_t mask, Decoded& d)
{
    const uint4* D = reinterpret_cast<const uint4*>(T.desc + cls * kFastDescStride);
    const uint4 h = D[0], v = D[1], lw = D[2], mg = D[3];
    const uint32_t B = (h.x >> 8) & 0xff, flags = (h.x >> 16) & 0xff;
    const uint32_t nlev1 = kPar == 1 ? 0u : (h.x >> 24) & 0xf, nlev = valid ? h.x >> 28 : 0u;
    const uint32_t goff = h.y & 0xffff, A = h.y >> 16;
    const bool odd = kPar == 1 || (kPar == -1 && (flags & 1u));
    // the arrangement rank of every calling lane fits 32 bits (all but the largest class of the 48-bit code): no 64-bit division
    const bool rank32 = kPar != -1 && __all_sync(mask, !valid || (flags & kFastFlagRank32));

    // S3: r fastest, then the sign word s, then the arrangement rank p
    uint64_t q;
    uint32_t r;
    if (kPar == 1 || (kPar == -1 && A == 4096u)) { r = (uint32_t)local & 4095u; q = local >> 12; }
    else {
        q = __umul64hi(local, ((uint64_t)h.w << 32) | h.z);
        uint64_t rem = local - q * A;
        if (rem >= A) { rem -= A; ++q; }
        r = (uint32_t)rem;
    }
    const uint32_t s = kPar == 1 ? 0u : (uint32_t)q & ((1u << B) - 1u);
    const uint64_t p = kPar == 1 ? q : q >> B;

    // S4: Golay codeword
    const uint32_t c = T.golay[goff + r];

    // S5: arrangement.  Group 1 lives on F1(c), group 0 on F0(c); an odd class is one group 0 on all positions.
    const uint32_t F1 = odd ? 0u : c;
    const uint32_t F0 = ~F1 & 0xffffffu;
    uint32_t freem = kPar == 1 ? 0xffffffu : F1;
    bool in_group0 = kPar == 1;
    uint32_t p0 = 0, p1 = 0, p2 = 0, bit1 = 0, nz0 = 0;
    uint32_t p32 = (uint32_t)p;
    const uint32_t lwords[4] = {lw.x, lw.y, lw.z, lw.w};
    const uint32_t magics[4] = {0u, mg.x, mg.y, mg.z};
    const int maxlev = __reduce_max_sync(mask, nlev);
#pragma unroll
    for (int l = 0; l < kFastMaxLevels; ++l) {
        if (l < maxlev) {
            if (kPar != 1 && !in_group0 && (uint32_t)l >= nlev1) {     // group 1 done: its filler gets id 1
                p0 |= freem;
                if (kPar == -1 && (flags & 8u)) bit1 |= freem;
                freem = F0; in_group0 = true;
            }
            // a lane whose class has fewer steps finds radix 1, k = 0 and all-ones reciprocals in its descriptor: the
            // division returns remainder 0 and the rank unchanged, the empty subset is placed (lanes without a block run
            // the steps of class 0, their result is dropped)
            const uint32_t word = lwords[l];
            const uint32_t radix = word & 0x3fffffu;
            const uint32_t k = (word >> 22) & 31u;
            const uint32_t nfree = (mg.w >> (8 * l)) & 0xffu;            // slots free before this step (0: no step)
            uint32_t rho;
            if (l + 1 == maxlev) {
                // the last step of the warp: what is left of the rank is the step's own digit (lanes whose class has fewer steps
                // hold 0 here and place the empty subset), no division
                rho = p32;
            } else if (l == 0 && !rank32) {
                uint64_t qq = __umul64hi(p, ((uint64_t)v.w << 32) | v.z);
                uint64_t rem = p - qq * radix;
                if (rem >= radix) { rem -= radix; ++qq; }
                p32 = (uint32_t)qq; rho = (uint32_t)rem;
            } else {
                uint32_t qq = __umulhi(p32, l == 0 ? T.desc[cls * kFastDescStride + kFastDescMagic0] : magics[l]);
                uint32_t rem = p32 - qq * radix;
                if (rem >= radix) { rem -= radix; ++qq; }
                p32 = qq; rho = rem;
            }
            uint32_t rel;
            if (T.sub3 != 0u && __all_sync(mask, k <= (uint32_t)kSmallSubsetMaxK)) {
                rel = small_subset(T, k, rho);                          // few elements: one lookup whatever the number of slots
            } else {
                int top;
                if (kPar == 0) top = 16;
                else if (kPar == 1 && l == 0) top = 24;
                else top = __reduce_max_sync(mask, nfree);
                rel = nth_subset(T, k, rho, top);
            }
            uint32_t a;
            if (kPar == 1 && l == 0) a = rel;                           // odd, first step: every position is free
            else if (kPar == 1 && l == 1 && __all_sync(mask, k == 0u || nfree >= 22u)) a = deposit_two_holes(rel, freem);
            else a = deposit24(T.pd6, rel, freem);
            freem ^= a;
            constexpr int kId0 = kPar == 1 ? 1 : 2;                     // the value id of level l is 2 + l (odd classes alone: 1 + l)
            if ((l + kId0) & 1) p0 |= a;
            if ((l + kId0) & 2) p1 |= a;
            if ((l + kId0) & 4) p2 |= a;
            if (kPar != 0 && (word & (1u << 30))) bit1 |= a;
            if (kPar != 1 && in_group0 && (word >> 31)) nz0 |= a;
        }
    }
    if (kPar != 1 && !in_group0) {
        p0 |= freem;
        if (kPar == -1 && (flags & 8u)) bit1 |= freem;
        freem = F0;
    }
    if (kPar != 0 && (flags & 16u)) bit1 |= freem;              // filler of group 0 keeps id 0
    if (kPar != 1 && (flags & 4u)) nz0 |= freem;

    // S6: signs
    uint32_t neg;
    if (kPar == 1) {
        neg = c ^ bit1;                                         // 1 mod 4 on F0, 3 mod 4 on F1
    } else {
        // the bits of s go to the positions that carry a sign (F1 and the nonzero ones of F0) in ascending order, except the
        // last F1 position: its sign makes the sum 0 mod 8
        const uint32_t last_f1 = F1 ? 0x80000000u >> __clz(F1) : 0u;
        uint32_t neg_even = deposit24(T.pd6, s, (F1 | (odd ? 0u : nz0)) & ~last_f1);
        if ((__popc(neg_even & F1) + (flags >> 1)) & 1u) neg_even |= last_f1;
        neg = odd ? (c ^ bit1) : neg_even;
    }
    if (valid) {
        d.p0 = p0; d.p1 = p1; d.p2 = p2; d.neg = neg;
        if (kPar == 1) {
            const uint2 vo = *reinterpret_cast<const uint2*>(T.desc + cls * kFastDescStride + kFastDescValsOdd);
            d.vals_lo = vo.x; d.vals_hi = vo.y;
        } else {
            d.vals_lo = v.x; d.vals_hi = v.y;
        }
    }
}

__device__ __forceinline__ void fast_decode(const FastSmem& T, uint64_t I, bool valid, Decoded& d)
{
    d.p0 = d.p1 = d.p2 = d.neg = d.vals_lo = d.vals_hi = 0u;
    uint64_t local = 0;
    const uint32_t cls = valid ? fast_find_class(T, I, local) : 0u;
    fast_decode_local<-1>(T, cls, local, valid, kFullMask, d);
}

// ---- expansion helpers -------------------------------------------------------
// 8 mask bits -> 8 nibbles (bit i -> bit 4i).
__device__ __forceinline__ uint32_t nibspread8(uint32_t b)
{
    // each "x | x << s" is written as a multiplication (the two copies never overlap): it runs on the FMA pipe,
    // the integer ALU pipe is the busy one
    uint32_t x = (b * 0x1001u) & 0x000f000fu;
    x = (x * 65u) & 0x03030303u;
    x = (x * 9u) & 0x11111111u;
    return x;
}

// Value id of each position as a nibble string: sel[r] holds positions 8r..8r+7.
__device__ __forceinline__ void id_nibbles(const Decoded& d, uint32_t sel[3])
{
#pragma unroll
    for (int r = 0; r < 3; ++r)
        sel[r] = nibspread8((d.p0 >> (8 * r)) & 0xffu) | (nibspread8((d.p1 >> (8 * r)) & 0xffu) << 1) |
                 (nibspread8((d.p2 >> (8 * r)) & 0xffu) << 2);
}

// 4 mask bits -> the most significant bits of 4 bytes.
__device__ __forceinline__ uint32_t msbspread4(uint32_t nib) { return (nib * 0x10204080u) & 0x80808080u; }

// The 24 coordinates as signed bytes, coordinate i in byte (i & 3) of word (i >> 2).
__device__ __forceinline__ void expand_bytes(const Decoded& d, uint32_t out[6])
{
    uint32_t sel[3];
    id_nibbles(d, sel);
#pragma unroll
    for (int j = 0; j < 6; ++j) {
        const uint32_t s16 = (j & 1) ? sel[j >> 1] >> 16 : sel[j >> 1];
        const uint32_t a = __byte_perm(d.vals_lo, d.vals_hi, s16);
        const uint32_t sm = msbspread4((d.neg >> (4 * j)) & 15u) >> 7;     // bytes 0 / 1
        out[j] = (a ^ (sm * 0xffu)) + sm;                                     // negated bytes are never zero
    }
}

// The 24 dequantized weights bf16_rn(gain * x_i) as 12 packed pairs (weight 2j in the low half of w[j]).
// All lanes of the warp must call this together: when no lane uses a value id above 3 (codes with few distinct
// values per class) the third bit plane and the upper half of the value table are skipped.
__device__ __forceinline__ void expand_bf16(const Decoded& d, float gain, uint32_t w[12])
{
    const bool wide = __any_sync(kFullMask, d.p2 != 0u);
    // bf16(gain * a) for the value ids; float(a) by the 2^23 trick (a <= 28)
    uint32_t packed[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (i < 2 || wide) {
            const uint32_t src = i < 2 ? d.vals_lo : d.vals_hi;
            const float a0 = __uint_as_float(__byte_perm(src, 0x4b000000u, (i & 1) ? 0x7442 : 0x7440)) - 8388608.f;
            const float a1 = __uint_as_float(__byte_perm(src, 0x4b000000u, (i & 1) ? 0x7443 : 0x7441)) - 8388608.f;
            __nv_bfloat162 b = __floats2bfloat162_rn(gain * a0, gain * a1);
            packed[i] = *reinterpret_cast<uint32_t*>(&b);
        }
    }
    const uint32_t lo03 = __byte_perm(packed[0], packed[1], 0x6420), hi03 = __byte_perm(packed[0], packed[1], 0x7531);
    const uint32_t lo47 = __byte_perm(packed[2], packed[3], 0x6420), hi47 = __byte_perm(packed[2], packed[3], 0x7531);
    uint32_t sel[3];
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        sel[r] = nibspread8((d.p0 >> (8 * r)) & 0xffu) | (nibspread8((d.p1 >> (8 * r)) & 0xffu) << 1);
        if (wide) sel[r] |= nibspread8((d.p2 >> (8 * r)) & 0xffu) << 2;
    }
#pragma unroll
    for (int j = 0; j < 6; ++j) {
        const uint32_t s16 = (j & 1) ? sel[j >> 1] >> 16 : sel[j >> 1];
        const uint32_t lob = __byte_perm(lo03, lo47, s16);
        const uint32_t hib = __byte_perm(hi03, hi47, s16) ^ msbspread4((d.neg >> (4 * j)) & 15u);
        w[2 * j] = __byte_perm(lob, hib, 0x5140);
        w[2 * j + 1] = __byte_perm(lob, hib, 0x7362);
    }
}

}  // namespace llvq
