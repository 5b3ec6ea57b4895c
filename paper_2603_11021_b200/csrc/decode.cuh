// Pieces shared by all kernels: the device view of a code's tables, the stored-format bit unpacking (S1), the
// packed representation of a decoded point and the gain step (S7).
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tables.h"

namespace llvq {

// Device view of one code's class tables in global memory (pointers owned by the context).  Codes whose class
// tables fit shared memory use the copies inside the table image instead.
struct DevCode {
    const ClassDesc* cls;           // [nclasses] (codes whose tables fit shared memory: read by the encoder's indexing kernel)
    const BigDesc* big;             // [nclasses] compact records (codes whose class tables stay in global memory)
    const uint64_t* off_lo;         // [nclasses + 1] low 64 bits of the class offsets
    const uint32_t* off_hi;         // [nclasses + 1] bits 64.. of the class offsets
    const uint32_t* lut16;          // [65537] class of the first index of bucket (I >> (W - 16)), then the last class
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

// Field b of a stream of W-bit fields, W <= 64: at most three 32-bit words, the third only when the field reaches it.
__device__ __forceinline__ uint64_t load_field(const uint32_t* __restrict__ stream, uint64_t b, int W)
{
    const uint64_t bp = b * (uint64_t)W;
    const uint32_t* p = stream + (bp >> 5);
    const int sh = (int)(bp & 31);
    const int last = sh + W;                                     // bits of the field counted from the first word
    const uint32_t w0 = __ldg(p);
    const uint32_t w1 = last > 32 ? __ldg(p + 1) : 0u;
    const uint32_t w2 = last > 64 ? __ldg(p + 2) : 0u;
    uint64_t v = (((uint64_t)w1 << 32) | w0) >> sh;
    if (sh) v |= (uint64_t)w2 << (64 - sh);
    return W < 64 ? v & ((1ull << W) - 1) : v;
}

// The same in two steps, for a caller that requests the words well before it needs the field: the words as they are
// (x = words 0-1, y = word 2 | bit offset << 32), and the field from them.
__device__ __forceinline__ ulonglong2 load_field_words(const uint32_t* __restrict__ stream, uint64_t b, int W)
{
    const uint64_t bp = b * (uint64_t)W;
    const uint32_t* p = stream + (bp >> 5);
    const int sh = (int)(bp & 31);
    const int last = sh + W;
    const uint32_t w0 = __ldg(p);
    const uint32_t w1 = last > 32 ? __ldg(p + 1) : 0u;
    const uint32_t w2 = last > 64 ? __ldg(p + 2) : 0u;
    return make_ulonglong2(((unsigned long long)w1 << 32) | w0, (unsigned long long)w2 | (unsigned long long)sh << 32);
}

__device__ __forceinline__ uint64_t field_of_words(ulonglong2 w, int W)
{
    const int sh = (int)(w.y >> 32);
    uint64_t v = w.x >> sh;
    if (sh) v |= (w.y & 0xffffffffull) << (64 - sh);
    return W < 64 ? v & ((1ull << W) - 1) : v;
}

// q = p / d, r = p % d with magic = floor((2^64 - 1) / d): the estimate is at most one too small.
__device__ __forceinline__ void divmod_magic(uint64_t p, uint32_t d, uint64_t magic, uint64_t& q, uint32_t& r)
{
    q = __umul64hi(p, magic);
    uint64_t rem = p - q * d;
    if (rem >= d) { rem -= d; ++q; }
    r = (uint32_t)rem;
}

// 4 mask bits -> 4 bytes holding 0 or 1.
__device__ __forceinline__ uint32_t spread4(uint32_t nib) { return (nib * 0x00204081u) & 0x01010101u; }

// Write absolute value `val` at the positions of `mask` (positions not yet written).
__device__ __forceinline__ void place_value(Point& pt, uint32_t mask, uint32_t val)
{
#pragma unroll
    for (int i = 0; i < 6; ++i) pt.w[i] += spread4((mask >> (4 * i)) & 15u) * val;
}

// Negate the coordinates at the positions of `neg` (never zero coordinates).
__device__ __forceinline__ void negate_at(Point& pt, uint32_t neg)
{
#pragma unroll
    for (int i = 0; i < 6; ++i) {
        const uint32_t sm = spread4((neg >> (4 * i)) & 15u);
        pt.w[i] = (pt.w[i] ^ (sm * 0xFFu)) + sm;
    }
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

// A 16-bit read-only load that stays where it is written among the other volatile statements (the decoders' table
// reads): issued before a block is unranked, its result is first used when the weights are formed.
__device__ __forceinline__ uint16_t ldg_u16_here(const uint16_t* p)
{
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ float gain_to_float(uint16_t bits)
{
    return __half2float(__ushort_as_half(bits));
}

}  // namespace llvq
