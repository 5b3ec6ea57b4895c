// C ABI and kernels of the LLVQ dequantization library (see include/llvq.h).
#include "llvq.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "decode.cuh"
#include "fast.cuh"
#include "big.cuh"
#include "umma.cuh"
#include "tables.h"
#include "ctx.h"

using namespace llvq;

namespace {


// ===========================================================================
// Fast path (tables in shared memory).  Dynamic shared memory of every fast
// kernel: [table image | mbarrier (16 bytes) | kernel-specific staging].
// Persistent CTAs, one per SM.
// ===========================================================================
constexpr int kFastThreads = 1024;      // decode / dequant kernels
constexpr int kGemvThreads = 1024;     // upper bound; the launch picks the warp count that divides the units per CTA best

struct FastArgs {
    FastLayout L;
    const uint8_t* image;
    uint32_t* flags;
    unsigned long long* bad_index;
    uint64_t n_points;              // N when it fits 64 bits (fast path)
    DevCode dc;                     // class tables in global memory (big codes)
};

// One block of 24 weights, end to end, in the two forms the consumers use.  kBig selects the decoder for codes
// whose class tables live in global memory; otherwise everything is served from the shared-memory image.
// All 32 lanes of a warp call these together; `in` = the block exists.
template <bool kBig>
__device__ __forceinline__ void block_point(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                            uint64_t b, bool in, Point& pt)
{
    uint64_t lo = 0, hi = 0;
    if (in) load_index(stream, b, fa.dc.W, lo, hi);
    const bool valid = in && (hi < fa.dc.n_hi || (hi == fa.dc.n_hi && lo < fa.dc.n_lo));
    if (in && !valid) atomicAdd(fa.bad_index, 1ull);
    uint64_t local = 0;
    const int cls = valid ? big_find_class(fa.dc, lo, hi, local) : 0;
    big_decode_local(T, fa.dc, cls, local, valid, pt);
}

template <bool kBig>
__device__ __forceinline__ void block_bytes(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                            uint64_t b, bool in, uint32_t w[6])
{
    if (kBig) {
        Point pt;
        block_point<kBig>(fa, T, stream, b, in, pt);
#pragma unroll
        for (int i = 0; i < 6; ++i) w[i] = pt.w[i];
    } else {
        const uint64_t I = in ? load_field(stream, b, (int)fa.L.W) : 0ull;
        const bool valid = in && I < fa.n_points;
        if (in && !valid) atomicAdd(fa.bad_index, 1ull);
        Decoded d;
        fast_decode(T, I, valid, d);
        expand_bytes(d, w);
    }
}

template <bool kBig>
__device__ __forceinline__ void block_pairs(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                            const uint16_t* __restrict__ gain, uint64_t b, bool in, uint32_t w[12])
{
    const float g = in ? gain_to_float(__ldg(gain + b)) : 0.f;
    if (kBig) {
        Point pt;
        block_point<kBig>(fa, T, stream, b, in, pt);
#pragma unroll
        for (int j = 0; j < 12; ++j) {
            __nv_bfloat162 h = __halves2bfloat162(dequant(g, pt, 2 * j), dequant(g, pt, 2 * j + 1));
            w[j] = *reinterpret_cast<uint32_t*>(&h);
        }
    } else {
        const uint64_t I = in ? load_field(stream, b, (int)fa.L.W) : 0ull;
        const bool valid = in && I < fa.n_points;
        if (in && !valid) atomicAdd(fa.bad_index, 1ull);
        Decoded d;
        fast_decode(T, I, valid, d);
        expand_bf16(d, g, w);
    }
}

// Shape-gain form of the gain step (App. E "Shape-gain" with a scalar gain codebook): the stored field carries the
// shape index in its low W bits and a gain index above; the block gain is
// (row_scale * codebook[k]) / |x|, each operation in binary32, 1/|x| = 1/sqrt(16 m) taken from the class descriptor.
struct SgArgs {
    const float* codebook;      // [1 << bits]
    const float* row_scale;     // [rows] or null (= 1)
    int bits;
};

__device__ __forceinline__ void block_pairs_sg(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                               const SgArgs& sg, uint64_t b, int64_t row, bool in, uint32_t w[12])
{
    const uint64_t f = in ? load_field(stream, b, (int)fa.L.W + sg.bits) : 0ull;
    const uint64_t I = f & ((1ull << fa.L.W) - 1ull);                 // W < 64 whenever gain bits are present or not: checked on the host
    const uint32_t k = (uint32_t)(f >> fa.L.W);
    const bool valid = in && I < fa.n_points;
    if (in && !valid) atomicAdd(fa.bad_index, 1ull);
    uint64_t local = 0;
    const uint32_t cls = valid ? fast_find_class(T, I, local) : 0u;
    Decoded d;
    fast_decode_local<-1>(T, cls, local, valid, kFullMask, d);
    float g = 0.f;
    if (in) {
        const float scale = sg.row_scale ? __ldg(sg.row_scale + row) : 1.f;
        g = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + k)), __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
    }
    expand_bf16(d, g, w);
}

// Programmatic dependent launch: a GEMV kernel lets the next kernel of the stream start early (its thread blocks
// move in as soon as this kernel's finish) and itself waits for the previous kernel to complete only after it has
// loaded its table image, before it reads anything a predecessor may have written (x, the scratch, the counters).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Ask for the 128-byte lines of [p + first, p + last) in L2; the whole CTA calls this.
__device__ __forceinline__ void prefetch_span_l2(const void* p, uint64_t first, uint64_t last)
{
    const uint8_t* base = static_cast<const uint8_t*>(p);
    for (uint64_t o = (first & ~127ull) + (uint64_t)threadIdx.x * 128; o < last; o += (uint64_t)blockDim.x * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + o));
}

#define FAST_PROLOGUE()                                                                         \
    extern __shared__ __align__(128) uint8_t smem[];                                            \
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + fa.L.total);                              \
    uint8_t* staging = smem + fa.L.total + 16;                                                  \
    (void)staging;                                                                              \
    pdl_launch_dependents();                                                                    \
    if (!fast_load_image(smem, fa.image, fa.L.total, bar, fa.flags)) return;                    \
    pdl_wait();                                                                                 \
    const FastSmem T = fast_view(smem, fa.L);

template <bool kBig>
__global__ void __launch_bounds__(kFastThreads, 1)
decode_blocks_fast_kernel(FastArgs fa, const uint32_t* __restrict__ stream, uint64_t nblocks, uint2* __restrict__ out)
{
    FAST_PROLOGUE();
    const uint64_t ntiles = (nblocks + kFastThreads - 1) / kFastThreads;
    for (uint64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const uint64_t b = tile * kFastThreads + threadIdx.x;
        const bool in = b < nblocks;
        uint32_t w[6];
        block_bytes<kBig>(fa, T, stream, b, in, w);
        if (in) {
            out[b * 3 + 0] = make_uint2(w[0], w[1]);
            out[b * 3 + 1] = make_uint2(w[2], w[3]);
            out[b * 3 + 2] = make_uint2(w[4], w[5]);
        }
    }
}

// FLAT (bpr == 0): block b covers elements 24b.. of the flattened matrix.
// ROWWISE: block b = r * bpr + cb covers columns 24cb.. of row r.
template <bool kBig, bool kSg = false>
__global__ void __launch_bounds__(kFastThreads, 1)
dequant_fast_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ gain, SgArgs sg, uint64_t nblocks,
                    int64_t rows, int64_t cols, int64_t bpr, __nv_bfloat16* __restrict__ out, int64_t ld)
{
    FAST_PROLOGUE();
    const uint64_t ntiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const uint64_t total = (uint64_t)rows * (uint64_t)cols;
    for (uint64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const uint64_t b = tile * kFastThreads + threadIdx.x;
        const bool in = b < nblocks;
        uint32_t w[12];
        if (kSg) block_pairs_sg(fa, T, stream, sg, b, in ? (int64_t)(b / (uint64_t)bpr) : 0, in, w);   // ROWWISE only
        else block_pairs<kBig>(fa, T, stream, gain, b, in, w);        // whole warp: the decoders vote
        if (!in) continue;
        __nv_bfloat16* dst;
        int64_t left;
        if (bpr == 0) { dst = out + b * 24; left = (int64_t)(total - b * 24); }
        else { const int64_t r = (int64_t)(b / (uint64_t)bpr), cb = (int64_t)(b % (uint64_t)bpr); dst = out + r * ld + cb * 24; left = cols - cb * 24; }
        if (left >= 24 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
            uint4* d4 = reinterpret_cast<uint4*>(dst);
            d4[0] = make_uint4(w[0], w[1], w[2], w[3]);
            d4[1] = make_uint4(w[4], w[5], w[6], w[7]);
            d4[2] = make_uint4(w[8], w[9], w[10], w[11]);
        } else {
#pragma unroll
            for (int j = 0; j < 24; ++j)
                if (j < left) dst[j] = __ushort_as_bfloat16((unsigned short)(w[j >> 1] >> (16 * (j & 1))));
        }
    }
}

// Fused dequant + GEMV.  The work is cut into units of 8 rows x 4 column blocks, numbered row group major, and
// every CTA takes an equal contiguous range of units.  In a unit lane (g, t) = (lane / 4, lane % 4) decodes the
// block (row g, column block 4q + t); its 12 packed bf16 pairs are the A fragments (rows 0..7; rows 8..15 are
// zero) of six m16n8k16 tensor-core MMAs whose B fragment carries the matching 4 x 24 activations (the same in
// all 8 columns), accumulating in binary32.  Row sums are collected in shared memory; a row group that is
// split between CTAs is finished through a zero-kept global scratch and an arrival counter.
constexpr int kGemvGroupRows = 8;        // rows per unit
constexpr int kGemvGroupsPerPass = 128;  // row groups whose sums a CTA keeps in shared memory at a time

__device__ __forceinline__ void mma_bf16_16816(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// CTA that owns unit u when G CTAs split U units into ranges [c*U/G, (c+1)*U/G).
__device__ __forceinline__ int64_t unit_owner(int64_t u, int64_t U, int64_t G) { return ((u + 1) * G - 1) / U; }

// Where a GEMV kernel puts y.  Row-sharded over several GPUs (each rank owns a band of output rows, x is the same
// everywhere), a rank writes its band straight into every rank's copy of the full vector: `y` is this rank's copy
// and `peer` the other ranks' copies mapped into this process, every pointer already advanced to the band's first
// row.  The stores to a peer travel over NVLink as plain remote writes.  n_peer = 0 is the single-GPU case.
constexpr int64_t kPairSlotOffset = 64ll * 65536;      // floats: the 64-bit slots of finish_pass lie behind the binary32 scratch rows
constexpr int kMaxShardPeers = 7;
struct YOut {
    void* y;
    void* peer[kMaxShardPeers];
    int n_peer;
    // optional: one word per peer that receives `epoch` once the whole grid has stored its rows (done = the
    // context's arrival counter, zero between launches)
    uint32_t* flag[kMaxShardPeers];
    uint32_t* done;
    uint32_t epoch;
    int n_flag;
};

template <bool kOutBf16, bool kShard>
__device__ __forceinline__ void store_y(const YOut& yo, int64_t row, float v)
{
    if (kOutBf16) {
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        reinterpret_cast<__nv_bfloat16*>(yo.y)[row] = h;
        if (!kShard) return;                              // the single-GPU instantiations carry none of what follows
#pragma unroll
        for (int p = 0; p < kMaxShardPeers; ++p)          // static indices: the struct stays in the parameter bank
            if (p < yo.n_peer) reinterpret_cast<__nv_bfloat16*>(yo.peer[p])[row] = h;
    } else {
        reinterpret_cast<float*>(yo.y)[row] = v;
        if (!kShard) return;
#pragma unroll
        for (int p = 0; p < kMaxShardPeers; ++p)
            if (p < yo.n_peer) reinterpret_cast<float*>(yo.peer[p])[row] = v;
    }
}

// Stages x for a GEMV CTA: xs[cb * 12 + j] = the bf16 pair (x[24 cb + 2j], x[24 cb + 2j + 1]), zero beyond k_in; `words`
// = 12 x the number of column blocks staged.  16-byte loads where x allows them.
__device__ __forceinline__ void stage_x(uint32_t* xs, const uint16_t* __restrict__ x, int64_t k_in, int64_t words)
{
    if ((reinterpret_cast<uintptr_t>(x) & 15) == 0) {
        const int64_t full = k_in / 8;                                       // whole groups of 8 elements
        for (int64_t v = threadIdx.x; v < words / 4; v += blockDim.x) {
            uint4 q = make_uint4(0u, 0u, 0u, 0u);
            if (v < full) q = __ldg(reinterpret_cast<const uint4*>(x) + v);
            else {
                uint32_t t[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t e = 8 * v + 2 * j;
                    const uint32_t lo = e < k_in ? __ldg(x + e) : 0u, hi = e + 1 < k_in ? __ldg(x + e + 1) : 0u;
                    t[j] = lo | hi << 16;
                }
                q = make_uint4(t[0], t[1], t[2], t[3]);
            }
            reinterpret_cast<uint4*>(xs)[v] = q;
        }
        return;
    }
    for (int64_t i = threadIdx.x; i < words; i += blockDim.x) {
        const int64_t e = 2 * i;
        const uint32_t lo = e < k_in ? __ldg(x + e) : 0u, hi = e + 1 < k_in ? __ldg(x + e + 1) : 0u;
        xs[i] = lo | hi << 16;
    }
}

// End of a pass of a GEMV CTA over row groups rg0..rg1 (8 rows each; the CTA owns units [u_begin, u_end) of U, nq
// units per row group, G CTAs): row_sum(i) is the CTA's sum for row i of the pass.  One warp per row group, lanes
// 0..7 its rows, no CTA-wide barrier inside.  A group the CTA covers completely is final.  A group it shares with
// neighbouring CTAs goes through the scratch row in global memory: add, make the add visible, count the arrival;
// whoever arrives last reads the total, writes y and leaves scratch and counter zero for the next launch (groups shared
// by exactly two CTAs take a shorter way, below).
// The caller puts a __syncthreads() before (sums complete) and after (sums may be cleared) the call.
template <bool kOutBf16, bool kShard, typename RowSum>
__device__ __forceinline__ void finish_pass(const YOut& yo, int64_t rg0, int64_t rg1, int64_t nq, int64_t u_begin, int64_t u_end,
                                            int64_t U, int64_t G, int64_t n_out, float* __restrict__ scratch,
                                            uint32_t* __restrict__ counters, RowSum row_sum)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = (int)(blockDim.x >> 5);
    for (int64_t rg = rg0 + warp; rg <= rg1; rg += nwarps) {
        const bool whole = u_begin <= rg * nq && (rg + 1) * nq <= u_end;
        const int64_t row = rg * kGemvGroupRows + lane;
        const bool mine = lane < kGemvGroupRows && row < n_out;
        const float part = lane < kGemvGroupRows ? row_sum((rg - rg0) * kGemvGroupRows + lane) : 0.f;
        if (whole) {
            if (mine) {
                store_y<kOutBf16, kShard>(yo, row, part);
                if (kShard) __threadfence_system();
            }
            continue;
        }
        const uint32_t parts = (uint32_t)(unit_owner((rg + 1) * nq - 1, U, G) - unit_owner(rg * nq, U, G) + 1);
        if (parts == 2u) {
            // two CTAs share the group (the usual case): one compare-and-swap on a 64-bit slot carries both the sum
            // and the arrival.  Whoever finds the slot empty leaves (its sum, 1) there; the other gets that back from
            // its failed swap, adds its own sum, stores y and empties the slot.  One round trip each, no fence.
            if (mine) {
                unsigned long long* slot = reinterpret_cast<unsigned long long*>(scratch + kPairSlotOffset) + row;
                const unsigned long long seen = atomicCAS(slot, 0ull, (unsigned long long)__float_as_uint(part) | 1ull << 32);
                if (seen != 0ull) {
                    store_y<kOutBf16, kShard>(yo, row, __fadd_rn(__uint_as_float((uint32_t)seen), part));
                    __stcg(slot, 0ull);
                    if (kShard) __threadfence_system();
                }
            }
            continue;
        }
        if (mine) atomicAdd(scratch + row, part);
        __threadfence();                               // every lane's add is performed before ...
        __syncwarp();
        uint32_t is_last = 0u;
        if (lane == 0) {
            __threadfence();                           // ... lane 0 counts the arrival
            is_last = atomicAdd(counters + rg, 1u) == parts - 1u;
        }
        is_last = __shfl_sync(kFullMask, is_last, 0);
        if (is_last) {
            __threadfence();
            if (mine) {
                store_y<kOutBf16, kShard>(yo, row, __ldcg(scratch + row));
                __stcg(scratch + row, 0.f);
                if (kShard) __threadfence_system();
            }
            if (lane == 0) counters[rg] = 0u;
        }
    }
}

// Last step of a row-sharded GEMV CTA (all threads call it, after their last store to y): counts the CTA in; the CTA
// that completes the grid raises the epoch in every peer's flag word.  The remote stores of y are fenced at system
// scope by the threads that made them (finish_pass) and once more, cumulatively, by the thread that counts.
__device__ __forceinline__ void shard_arrive(const YOut& yo)
{
    if (yo.n_flag == 0) return;
    __syncthreads();
    if (threadIdx.x != 0) return;
    __threadfence_system();
    if (atomicAdd(yo.done, 1u) != gridDim.x - 1u) return;
    atomicExch(yo.done, 0u);
    __threadfence_system();
#pragma unroll
    for (int p = 0; p < kMaxShardPeers; ++p)
        if (p < yo.n_flag) asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(yo.flag[p]), "r"(yo.epoch) : "memory");
}

template <bool kBig, bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_fast_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ gain, SgArgs sg,
                 int64_t n_out, int64_t k_in, int64_t bpr, const uint16_t* __restrict__ x, YOut yo,
                 float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    FAST_PROLOGUE();
    const int64_t nq = (bpr + 3) / 4;                               // units along K
    uint32_t* xs = reinterpret_cast<uint32_t*>(staging);            // [nq * 4][12] packed bf16 pairs of x
    float* acc = reinterpret_cast<float*>(xs + nq * 48);            // [kGemvGroupsPerPass][8]
    stage_x(xs, x, k_in, nq * 48);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int kWarps = (int)(blockDim.x >> 5);
    const int64_t groups = (n_out + kGemvGroupRows - 1) / kGemvGroupRows;
    const int64_t U = groups * nq, G = gridDim.x;
    const int64_t u_begin = blockIdx.x * U / G, u_end = (blockIdx.x + 1) * U / G;
    const int64_t rg_first = u_begin / nq, rg_last = u_begin < u_end ? (u_end - 1) / nq : rg_first - 1;   // no units: no pass
    for (int64_t rg0 = rg_first; rg0 <= rg_last; rg0 += kGemvGroupsPerPass) {
        const int64_t rg1 = min(rg0 + kGemvGroupsPerPass - 1, rg_last);
        for (int i = threadIdx.x; i < kGemvGroupsPerPass * kGemvGroupRows; i += (int)blockDim.x) acc[i] = 0.f;
        __syncthreads();
        const int64_t p_begin = max(u_begin, rg0 * nq), p_end = min(u_end, (rg1 + 1) * nq);
        int64_t rg = (p_begin + warp) / nq, kq = (p_begin + warp) - rg * nq;      // walked along with u: no division per unit
        for (int64_t u = p_begin + warp; u < p_end; u += kWarps, kq += kWarps) {
            while (kq >= nq) { kq -= nq; ++rg; }
            const int64_t cb = kq * 4 + t;
            const int64_t row = rg * kGemvGroupRows + g;
            const bool in = row < n_out && cb < bpr;
            const uint64_t b = (uint64_t)(row * bpr + cb);
            uint32_t w[12];
            if (kSg) block_pairs_sg(fa, T, stream, sg, b, row, in, w);
            else block_pairs<kBig>(fa, T, stream, gain, b, in, w);
            const uint4* xb = reinterpret_cast<const uint4*>(xs + cb * 12);
            const uint4 x0 = xb[0], x1 = xb[1], x2 = xb[2];
            const uint32_t xv[12] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w};
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int q = 0; q < 6; ++q)
                mma_bf16_16816(c, w[2 * q], 0u, w[2 * q + 1], 0u, xv[2 * q], xv[2 * q + 1]);
            if (t == 0) atomicAdd(&acc[(rg - rg0) * kGemvGroupRows + g], c[0]);
        }
        __syncthreads();
        // row groups this CTA covers completely are final; the (at most two) split ones go through the scratch
        finish_pass<kOutBf16, kShard>(yo, rg0, rg1, nq, u_begin, u_end, U, G, n_out, scratch, counters, [&](int64_t r) { return acc[r]; });
        __syncthreads();                                   // the sums are read above: the next pass may clear them only now
    }
    if (kShard) shard_arrive(yo);
}

constexpr uint32_t kKindEven = 0u, kKindOdd = 1u, kKindOther = 2u, kKindNull = 3u;   // decoder form a class needs

// ===========================================================================
// Sorted layout for the fused GEMV (llvq_sort_blocks / llvq_gemv_sorted).
// The work is cut exactly as in gemv_fast_kernel: units of 8 rows x 4 column blocks, row group major, an equal
// contiguous range of units per CTA (for the CTA count of this device).  Inside a CTA's range the units are taken
// in segments of up to kSortSegUnits units, and the blocks of a segment are stored sorted by the decoder form
// their class needs (odd / even with Golay weight 8, 12, 16 / other) and its number of unranking steps (most
// expensive first), so that the 32 lanes of a warp run the same form with the same trip count.  Each block is a
// 64-bit entry: the stored index I unchanged in the low 48 bits, its position in the segment (unit * 32 + lane)
// in the high 16 bits; entries that do not exist (ragged edges) or are out of range carry I = 2^48 - 1.
// All of App. A runs in the GEMV kernel.  A warp takes 32 consecutive entries, each lane unranks its block and
// multiplies it with its own slice of x (binary32 FMAs), and adds the partial row sum to the CTA's row sums.
// ===========================================================================
constexpr int kSortSegUnits = 2048;                  // 65536 blocks
constexpr int kSortThreads = 1024;
constexpr int kSortAccCopies = 4;                    // copies of the row sums in shared memory (a power of two)
constexpr unsigned long long kSortIndexMask = (1ull << 48) - 1ull;

// Calls f(tu0, tu1, rg0, rg1, first, last) for every segment [tu0, tu1) of CTA `cta` (of G) in order; rg0..rg1 = row
// groups of the pass the segment belongs to (a pass covers at most kGemvGroupsPerPass row groups); first / last =
// the segment opens / closes its pass.
template <typename F>
__device__ __forceinline__ void for_each_sorted_segment(int64_t U, int64_t G, int64_t nq, int64_t cta, F f, int seg_units = kSortSegUnits)
{
    const int64_t u_begin = cta * U / G, u_end = (cta + 1) * U / G;
    if (u_begin >= u_end) return;
    const int64_t rg_first = u_begin / nq, rg_last = (u_end - 1) / nq;
    for (int64_t rg0 = rg_first; rg0 <= rg_last; rg0 += kGemvGroupsPerPass) {
        const int64_t rg1 = min(rg0 + kGemvGroupsPerPass - 1, rg_last);
        const int64_t p_begin = max(u_begin, rg0 * nq), p_end = min(u_end, (rg1 + 1) * nq);
        for (int64_t tu0 = p_begin; tu0 < p_end; tu0 += seg_units)
            f(tu0, min(tu0 + (int64_t)seg_units, p_end), rg0, rg1, tu0 == p_begin, tu0 + seg_units >= p_end);
    }
}

__global__ void __launch_bounds__(kSortThreads, 1)
sort_blocks_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ sort_rank, int gain_bits, int64_t n_out,
                   int64_t bpr, unsigned long long* __restrict__ out)
{
    FAST_PROLOGUE();
    __shared__ uint32_t hist[1024], cursor[1024];                  // one bin per class, in sort order; bin 1023 = no block
    const int64_t nq = (bpr + 3) / 4;
    const int64_t groups = (n_out + kGemvGroupRows - 1) / kGemvGroupRows;
    const int64_t U = groups * nq, G = gridDim.x;
    for_each_sorted_segment(U, G, nq, blockIdx.x, [&](int64_t tu0, int64_t tu1, int64_t, int64_t, bool, bool) {
        const int entries = (int)(tu1 - tu0) * 32;
        hist[threadIdx.x] = 0; cursor[threadIdx.x] = 0;
        __syncthreads();
        // key and field of entry i of the segment; count = the first pass (out-of-range fields are counted once)
        auto entry_of = [&](int i, bool count, unsigned long long& field) {
            const int64_t u = tu0 + (i >> 5);
            const int lane = i & 31;
            const int64_t rg = u / nq, kq = u - rg * nq;
            const int64_t row = rg * kGemvGroupRows + (lane >> 2), cb = kq * 4 + (lane & 3);
            field = kSortIndexMask;
            if (row >= n_out || cb >= bpr) return 1023u;
            const uint64_t f = load_field(stream, (uint64_t)(row * bpr + cb), (int)fa.L.W + gain_bits);   // shape index | gain index << W
            const uint64_t I = f & ((1ull << fa.L.W) - 1ull);
            if (I >= fa.n_points) { if (count) atomicAdd(fa.bad_index, 1ull); return 1023u; }
            uint64_t local;
            field = f;
            return (uint32_t)__ldg(sort_rank + fast_find_class(T, I, local));
        };
        for (int i = threadIdx.x; i < entries; i += kSortThreads) {
            unsigned long long field;
            atomicAdd(&hist[entry_of(i, true, field)], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (int k = 0; k < 1024; ++k) { const uint32_t c = hist[k]; hist[k] = run; run += c; }
        }
        __syncthreads();
        // the entries are visited column-block major (all row groups of a column unit, then the next unit): the blocks
        // of a bin then come out roughly ordered by column block, and the 32 lanes of a GEMV warp read few different
        // slices of x
        const int64_t rg_a = tu0 / nq, nrg = (tu1 - 1) / nq - rg_a + 1;
        for (int64_t e = threadIdx.x; e < nq * nrg * 32; e += kSortThreads) {
            const int64_t kq = e / (nrg * 32), rem = e - kq * (nrg * 32);
            const int64_t u = (rg_a + (rem >> 5)) * nq + kq;
            if (u < tu0 || u >= tu1) continue;
            const int i = (int)(u - tu0) * 32 + (int)(rem & 31);
            unsigned long long field;
            const uint32_t key = entry_of(i, false, field);
            const uint32_t slot = hist[key] + atomicAdd(&cursor[key], 1u);
            out[tu0 * 32 + slot] = field | (unsigned long long)i << 48;
        }
        __syncthreads();
    });
}

// App. A steps 2-4 for one entry of a sorted layout: class lookup, then the unranker form the class needs.  The
// lanes of a warp call this together; after sorting they almost always share the form (and the class).
__device__ __forceinline__ void decode_known_class(const FastSmem& T, uint32_t cls, uint64_t local, bool valid, Decoded& r)
{
    const uint32_t h = T.desc[cls * kFastDescStride];
    const uint32_t w8 = h & 0xffu;
    const uint32_t kind = !valid ? kKindNull : ((h & (1u << 16)) ? kKindOdd : ((w8 == 8u || w8 == 12u || w8 == 16u) ? kKindEven : kKindOther));
    Decoded d;
    r.p0 = r.p1 = r.p2 = r.neg = r.vals_lo = r.vals_hi = 0u;
    if (__any_sync(kFullMask, kind == kKindOdd)) {
        const bool mine = kind == kKindOdd;
        fast_decode_local<1>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, d);
        if (mine) r = d;
    }
    if (__any_sync(kFullMask, kind == kKindEven)) {
        const bool mine = kind == kKindEven;
        fast_decode_local<0>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, d);
        if (mine) r = d;
    }
    if (__any_sync(kFullMask, kind == kKindOther)) {
        const bool mine = kind == kKindOther;
        fast_decode_local<-1>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, d);
        if (mine) r = d;
    }
}

__device__ __forceinline__ uint32_t decode_sorted_entry(const FastArgs& fa, const FastSmem& T, uint64_t I, bool valid, Decoded& r)
{
    uint64_t local = 0;
    const uint32_t cls = valid ? fast_find_class(T, I, local) : 0u;
    decode_known_class(T, cls, local, valid, r);
    return cls;
}

template <bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_sorted_kernel(FastArgs fa, const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, SgArgs sg,
                   int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, const uint16_t* __restrict__ x, YOut yo,
                   float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    FAST_PROLOGUE();
    const int64_t nq = (bpr + 3) / 4;
    uint32_t* xs = reinterpret_cast<uint32_t*>(staging);            // [nq * 4][12] packed bf16 pairs of x
    float* acc = reinterpret_cast<float*>(xs + nq * 48);            // [kSortAccCopies][kGemvGroupsPerPass][8]: warps spread their adds over the copies
    uint32_t* last_flag = reinterpret_cast<uint32_t*>(acc + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows);
    uint32_t* next_chunk = last_flag + 1;
    stage_x(xs, x, k_in, nq * 48);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t kWarps = blockDim.x >> 5;
    const int64_t groups = (n_out + kGemvGroupRows - 1) / kGemvGroupRows;
    const int64_t U = groups * nq, G = gridDim.x;
    const uint32_t nq32 = (uint32_t)nq;

    for_each_sorted_segment(U, G, nq, blockIdx.x, [&](int64_t tu0, int64_t tu1, int64_t rg0, int64_t rg1, bool first, bool last) {
        if (first)
            for (int i = threadIdx.x; i < kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows; i += (int)blockDim.x) acc[i] = 0.f;
        if (threadIdx.x == 0) *next_chunk = kWarps;
        __syncthreads();
        const int64_t rg_a = tu0 / nq;
        const uint32_t kq_a = (uint32_t)(tu0 - rg_a * nq), rg_off = (uint32_t)(rg_a - rg0);
        const uint32_t nchunks = (uint32_t)(tu1 - tu0);
        const unsigned long long* seg = sorted + tu0 * 32 + lane;
        uint32_t ch = (uint32_t)warp;
        unsigned long long e = ch < nchunks ? __ldg(seg + (uint64_t)ch * 32) : 0ull;
        while (ch < nchunks) {
            // chunks are handed out dynamically (their cost depends on the form); the next entry is fetched ahead
            uint32_t nxt = 0;
            if (lane == 0) nxt = atomicAdd(next_chunk, 1u);
            nxt = __shfl_sync(kFullMask, nxt, 0);
            const unsigned long long e_next = nxt < nchunks ? __ldg(seg + (uint64_t)nxt * 32) : 0ull;
            const uint64_t field = e & kSortIndexMask;
            const uint64_t I = kSg ? field & ((1ull << fa.L.W) - 1ull) : field;     // shape-gain form: gain index above the shape index
            const uint32_t pos = (uint32_t)(e >> 48);
            const bool valid = field != kSortIndexMask && I < fa.n_points;
            // where the block sits: unit = pos / 32 of the segment, (row, column block) = lane of the unit
            const uint32_t v = kq_a + (pos >> 5);
            uint32_t q = __umulhi(v, nq_magic), kq = v - q * nq32;
            if (kq >= nq32) { kq -= nq32; ++q; }
            const uint32_t rloc = (rg_off + q) * kGemvGroupRows + ((pos >> 2) & 7u);      // row inside the pass
            const uint32_t cb = kq * 4u + (pos & 3u);
            float gn = 0.f;
            if (!kSg && valid) gn = gain_to_float(__ldg(gain + ((int64_t)rg0 * kGemvGroupRows + rloc) * bpr + cb));
            Decoded r;
            const uint32_t cls = decode_sorted_entry(fa, T, I, valid, r);
            if (kSg && valid) {
                const float scale = sg.row_scale ? __ldg(sg.row_scale + (int64_t)rg0 * kGemvGroupRows + rloc) : 1.f;
                gn = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + (uint32_t)(field >> fa.L.W))),
                               __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
            }
            uint32_t w[12];
            expand_bf16(r, gn, w);
            const uint4* xb = reinterpret_cast<const uint4*>(xs + cb * 12u);
            const uint4 x0 = xb[0], x1 = xb[1], x2 = xb[2];
            const uint32_t xv[12] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w};
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < 12; ++j) {                        // bf16 x bf16 products are exact in binary32
                s0 = fmaf(__uint_as_float(w[j] << 16), __uint_as_float(xv[j] << 16), s0);
                s1 = fmaf(__uint_as_float(w[j] & 0xffff0000u), __uint_as_float(xv[j] & 0xffff0000u), s1);
            }
            if (valid) atomicAdd(&acc[(warp & (kSortAccCopies - 1)) * (kGemvGroupsPerPass * kGemvGroupRows) + rloc], s0 + s1);
            ch = nxt; e = e_next;
        }
        __syncthreads();
        if (!last) return;
        // end of the pass: row groups this CTA covers completely are final; the split ones go through the scratch
        auto row_sum = [&](int64_t r) {
            float v = 0.f;
#pragma unroll
            for (int c = 0; c < kSortAccCopies; ++c) v += acc[c * (kGemvGroupsPerPass * kGemvGroupRows) + r];
            return v;
        };
        const int64_t ub = blockIdx.x * U / G, ue = (blockIdx.x + 1) * U / G;     // recomputed here: nothing 64-bit lives across the main loop
        finish_pass<kOutBf16, kShard>(yo, rg0, rg1, nq, ub, ue, U, G, n_out, scratch, counters, row_sum);
        __syncthreads();                                   // the sums are read above: the next pass may clear them only now
    });
    if (kShard) shard_arrive(yo);
}

// ===========================================================================
// Fused GEMV on the stored stream with the blocks binned inside the kernel: the work split of gemv_fast_kernel, but a
// CTA first looks up the class of every block of a segment of up to kBinSegUnits units (S1-S2), orders the
// (class-local index, class, position) triples by the sorted layout's key with a counting sort in shared memory,
// and then proceeds like gemv_sorted_kernel on those entries (S3-S8): a warp takes 32 consecutive entries, runs
// the one unranker form they need and each lane forms its own dot product.
// ===========================================================================
constexpr int kBinSegUnits = 256;                    // at most 8192 blocks per segment (halved while shared memory is short)
constexpr int kBinPerThread = kBinSegUnits * 32 / kSortThreads;   // 8

template <bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_bin_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ sort_rank, const uint16_t* __restrict__ gain, SgArgs sg,
                int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, int seg_units, const uint16_t* __restrict__ x, YOut yo,
                float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    FAST_PROLOGUE();
    const int64_t nq = (bpr + 3) / 4;
    uint32_t* xs = reinterpret_cast<uint32_t*>(staging);            // [nq * 4][12] packed bf16 pairs of x
    float* acc = reinterpret_cast<float*>(xs + nq * 48);            // [kSortAccCopies][kGemvGroupsPerPass][8]
    uint32_t* last_flag = reinterpret_cast<uint32_t*>(acc + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows);
    uint32_t* next_chunk = last_flag + 1;
    uint32_t* hist = last_flag + 4;                                  // [1024] bins in sort order; later their first slots
    uint32_t* cursor = hist + 1024;                                  // [1024]
    unsigned long long* ent = reinterpret_cast<unsigned long long*>(cursor + 1024);   // [seg_units * 32] class-local index | position << 48
    uint16_t* ent_cls = reinterpret_cast<uint16_t*>(ent + seg_units * 32);            // [seg_units * 32] class (| gain index << 10), 0xffff = no block
    stage_x(xs, x, k_in, nq * 48);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t kWarps = blockDim.x >> 5;
    const int64_t groups = (n_out + kGemvGroupRows - 1) / kGemvGroupRows;
    const int64_t U = groups * nq, G = gridDim.x;
    const int64_t u_begin = blockIdx.x * U / G, u_end = (blockIdx.x + 1) * U / G;
    const uint32_t nq32 = (uint32_t)nq;
    if (u_begin < u_end) {
        // the rows of the row groups this CTA touches are one contiguous span of the index stream and of the gains:
        // request it from DRAM now, the binning phases then read it from L2
        const uint64_t b_first = (uint64_t)(u_begin / nq) * kGemvGroupRows * (uint64_t)bpr;
        const uint64_t b_last = (uint64_t)min(((u_end - 1) / nq + 1) * kGemvGroupRows, n_out) * (uint64_t)bpr;
        const uint64_t wf = (uint64_t)fa.L.W + (kSg ? (uint64_t)sg.bits : 0ull);
        prefetch_span_l2(stream, b_first * wf / 8, (b_last * wf + 7) / 8);
        if (!kSg) prefetch_span_l2(gain, b_first * 2, b_last * 2);
    }
    for_each_sorted_segment(U, G, nq, blockIdx.x, [&](int64_t tu0, int64_t tu1, int64_t rg0, int64_t rg1, bool first, bool last) {
        if (first)
            for (int i = threadIdx.x; i < kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows; i += (int)blockDim.x) acc[i] = 0.f;
        hist[threadIdx.x] = 0; cursor[threadIdx.x] = 0;
        if (threadIdx.x == 0) *next_chunk = kWarps;
        __syncthreads();
        const int64_t rg_a = tu0 / nq;
        const uint32_t kq_a = (uint32_t)(tu0 - rg_a * nq), rg_off = (uint32_t)(rg_a - rg0);
        const int entries = (int)(tu1 - tu0) * 32;
        // ---- S1-S2 for the whole segment and the histogram of the sort keys
        unsigned long long mine_ent[kBinPerThread];
        uint32_t mine_key[kBinPerThread];
#pragma unroll
        for (int q = 0; q < kBinPerThread; ++q) {
            const int i = (int)threadIdx.x + q * kSortThreads;
            mine_key[q] = 0xffffffffu; mine_ent[q] = 0ull;
            if (i < entries) {
                const uint32_t pos = (uint32_t)i;
                const uint32_t v = kq_a + (pos >> 5);
                uint32_t qd = __umulhi(v, nq_magic), kq = v - qd * nq32;
                if (kq >= nq32) { kq -= nq32; ++qd; }
                const int64_t row = (rg_a + qd) * kGemvGroupRows + ((pos >> 2) & 7u), cb = (int64_t)kq * 4 + (pos & 3u);
                uint32_t key = 1023u, cls = 0xffffu;
                uint64_t local = 0;
                if (row < n_out && cb < bpr) {
                    const uint64_t f = load_field(stream, (uint64_t)(row * bpr + cb), (int)fa.L.W + (kSg ? sg.bits : 0));
                    const uint64_t I = kSg ? f & ((1ull << fa.L.W) - 1ull) : f;
                    if (I < fa.n_points) {
                        cls = fast_find_class(T, I, local);
                        key = __ldg(sort_rank + cls);
                        if (kSg) cls |= (uint32_t)(f >> fa.L.W) << 10;           // the gain index rides with the class
                    } else atomicAdd(fa.bad_index, 1ull);
                }
                mine_key[q] = key | cls << 16;
                mine_ent[q] = local | (unsigned long long)pos << 48;
                atomicAdd(&hist[key], 1u);
            }
        }
        __syncthreads();
        // exclusive prefix sum of the 1024 bins: one bin per thread
        {
            const uint32_t c = hist[threadIdx.x];
            uint32_t incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(kFullMask, incl, o); if (lane >= o) incl += t; }
            if (lane == 31) cursor[warp] = incl;                       // warp totals, parked in the cursor array for a moment
            __syncthreads();
            uint32_t before = 0;
            for (int w2 = 0; w2 < warp; ++w2) before += cursor[w2];
            __syncthreads();
            hist[threadIdx.x] = before + incl - c;
            cursor[threadIdx.x] = 0;
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kBinPerThread; ++q) {
            if (mine_key[q] != 0xffffffffu) {
                const uint32_t key = mine_key[q] & 0xffffu;
                const uint32_t slot = hist[key] + atomicAdd(&cursor[key], 1u);
                ent[slot] = mine_ent[q];
                ent_cls[slot] = (uint16_t)(mine_key[q] >> 16);
            }
        }
        __syncthreads();
        // ---- S3-S8 on the ordered entries
        const uint32_t nchunks = (uint32_t)(tu1 - tu0);
        const uint16_t* gain_pass = gain + rg0 * kGemvGroupRows * bpr;
        for (uint32_t ch = (uint32_t)warp; ch < nchunks;) {
            uint32_t nxt = 0;
            if (lane == 0) nxt = atomicAdd(next_chunk, 1u);
            nxt = __shfl_sync(kFullMask, nxt, 0);
            const unsigned long long e = ent[ch * 32 + lane];
            const uint32_t cls16 = ent_cls[ch * 32 + lane];
            const bool valid = cls16 != 0xffffu;
            const uint32_t pos = (uint32_t)(e >> 48);
            const uint32_t v = kq_a + (pos >> 5);
            uint32_t q = __umulhi(v, nq_magic), kq = v - q * nq32;
            if (kq >= nq32) { kq -= nq32; ++q; }
            const uint32_t rloc = (rg_off + q) * kGemvGroupRows + ((pos >> 2) & 7u);
            const uint32_t cb = kq * 4u + (pos & 3u);
            const uint32_t cls = valid ? (kSg ? cls16 & 1023u : cls16) : 0u;
            float gn = 0.f;
            if (valid) {
                if (kSg) {
                    const float scale = sg.row_scale ? __ldg(sg.row_scale + (int64_t)rg0 * kGemvGroupRows + rloc) : 1.f;
                    gn = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + (cls16 >> 10))), __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
                } else {
                    gn = gain_to_float(__ldg(gain_pass + (int64_t)rloc * bpr + cb));
                }
            }
            Decoded r;
            decode_known_class(T, cls, e & ((1ull << 48) - 1ull), valid, r);
            uint32_t w[12];
            expand_bf16(r, gn, w);
            const uint4* xb = reinterpret_cast<const uint4*>(xs + cb * 12u);
            const uint4 x0 = xb[0], x1 = xb[1], x2 = xb[2];
            const uint32_t xv[12] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w};
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < 12; ++j) {
                s0 = fmaf(__uint_as_float(w[j] << 16), __uint_as_float(xv[j] << 16), s0);
                s1 = fmaf(__uint_as_float(w[j] & 0xffff0000u), __uint_as_float(xv[j] & 0xffff0000u), s1);
            }
            if (valid) atomicAdd(&acc[(warp & (kSortAccCopies - 1)) * (kGemvGroupsPerPass * kGemvGroupRows) + rloc], s0 + s1);
            ch = nxt;
        }
        __syncthreads();
        if (!last) return;
        auto row_sum = [&](int64_t r) {
            float v = 0.f;
#pragma unroll
            for (int c = 0; c < kSortAccCopies; ++c) v += acc[c * (kGemvGroupsPerPass * kGemvGroupRows) + r];
            return v;
        };
        const int64_t ub = blockIdx.x * U / G, ue = (blockIdx.x + 1) * U / G;     // recomputed here: nothing 64-bit lives across the main loop
        finish_pass<kOutBf16, kShard>(yo, rg0, rg1, nq, ub, ue, U, G, n_out, scratch, counters, row_sum);
        __syncthreads();
    }, seg_units);
    if (kShard) shard_arrive(yo);
}

// ===========================================================================
// llvq_gemm_small_batch: Y[b][i] = sum_k X[b][k] W[i][k] on the tensor cores.
// A work item is a tile of 128 output rows x a range of K stages (96 columns = 4 blocks of 24 per row).
// Per stage every thread of a 512-thread group dequantizes one block into the group's shared-memory A tile
// (bf16, K-major core-matrix layout), the matching slice of X goes into its B tile, and one thread issues
// six tcgen05 MMAs (M = 128, N = padded batch, K = 16) into the group's accumulator in tensor memory.
// The two groups of a CTA take alternate stages, so two stages are in flight.
// Split-K partial sums are added into a zero-initialised binary32 scratch [npad][n_out]; the last item
// of a row tile converts it to bf16 and clears it again.
// ===========================================================================
constexpr int kGemmThreads = 1024;
constexpr int kGemmGroupThreads = 512;
constexpr int kGemmRows = 128;
constexpr int kStageBlocks = 4;                       // column blocks per stage
constexpr int kStageK = kStageBlocks * 24;            // 96
constexpr int kMaxScratchRows = 65536;
constexpr int kCounterWords = 64 * kMaxScratchRows / 8;      // the word after them counts the CTAs of a row-sharded GEMV that have finished
constexpr uint32_t kTmemCols = 128;

struct GemmArgs {
    int64_t n_out, k_in, bpr;
    int batch, npad;
    int nstages, split;
    const uint16_t* x;
    uint16_t* y;               // Y [batch][y_ld] bf16, at the first row of this launch's rows
    int64_t y_ld;
    const YOut* shard;         // row-sharded launch: the peers' copies and flags (device memory), else null
    float* scratch;            // [npad][scratch_ld] binary32, all zero on entry and on exit
    int64_t scratch_ld;        // row tiles * 128
    uint32_t* counters;        // [row tiles], zero on entry and on exit
};

__global__ void put_shard_kernel(YOut yo, YOut* dst)
{
    if (threadIdx.x == 0) *dst = yo;
}

// One element of Y; a row-sharded launch also writes it into the peers' copies (their description sits in device
// memory so that the ordinary launch's parameters stay as small as they were).
template <bool kShard>
__device__ __forceinline__ void gemm_store(const GemmArgs& ga, int n, int64_t orow, float v)
{
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const int64_t at = (int64_t)n * ga.y_ld + orow;
    reinterpret_cast<__nv_bfloat16*>(ga.y)[at] = h;
    if (kShard) {
        const int np = ga.shard->n_peer;
        for (int p = 0; p < np; ++p) reinterpret_cast<__nv_bfloat16*>(ga.shard->peer[p])[at] = h;
    }
}

__device__ __forceinline__ void group_barrier(int group)
{
    asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "n"(kGemmGroupThreads) : "memory");
}

template <bool kBig, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ gain, SgArgs sg, GemmArgs ga)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t img_bytes = fa.L.total;
    uint64_t* bar_img = reinterpret_cast<uint64_t*>(smem + img_bytes);
    uint64_t* bar_free = bar_img + 1;                                     // [2]: the MMAs reading group h's buffers are done
    uint64_t* bar_done = bar_img + 3;                                     // [2]: group h's accumulator of this item is complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_img + 5);
    uint32_t* last_flag = tmem_slot + 1;
    const uint32_t a_off = (img_bytes + 64 + 1023) & ~1023u;
    uint8_t* a_buf = smem + a_off;                                        // [2 groups] x 24576
    uint8_t* b_buf = a_buf + 2 * kGemmRows * kStageK * 2;                  // [2 groups] x npad * 192
    const uint32_t b_stage = (uint32_t)ga.npad * kStageK * 2;

    pdl_launch_dependents();
    if (!fast_load_image(smem, fa.image, fa.L.total, bar_img, fa.flags)) return;
    pdl_wait();
    const FastSmem T = fast_view(smem, fa.L);
    // Two groups of 512 threads fill alternate stages, each into its own buffers and its own accumulator
    // (TMEM columns [64 h, 64 h + npad)); the epilogue adds the two accumulators.
    const int group = threadIdx.x / kGemmGroupThreads, gtid = threadIdx.x % kGemmGroupThreads;
    const int gwarp = gtid >> 5, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(&bar_free[0], 1); mbar_init(&bar_free[1], 1); mbar_init(&bar_done[0], 1); mbar_init(&bar_done[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t idesc = instr_desc_bf16_m128((uint32_t)ga.npad);
    uint8_t* const a_mine = a_buf + group * (kGemmRows * kStageK * 2);
    uint8_t* const b_mine = b_buf + group * b_stage;

    const int64_t row_tiles = (ga.n_out + kGemmRows - 1) / kGemmRows;
    const int64_t items = row_tiles * ga.split;
    uint32_t uses = 0;                                  // stages this group has filled so far
    uint32_t done[2] = {0, 0};                          // completed accumulations per group
    bool timeout = false;
    for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int64_t rt = item / ga.split;
        const int f = (int)(item % ga.split);
        const int s_begin = (int)((int64_t)f * ga.nstages / ga.split), s_end = (int)((int64_t)(f + 1) * ga.nstages / ga.split);
        const int64_t row = rt * kGemmRows + gwarp * 8 + (lane & 7);
        for (int s = s_begin + group; s < s_end; s += 2, ++uses) {
            // ---- A: dequantize one block of 24 weights
            const int64_t cb = (int64_t)s * kStageBlocks + (lane >> 3);
            const bool in = row < ga.n_out && cb < ga.bpr;
            const uint64_t b = in ? (uint64_t)(row * ga.bpr + cb) : 0ull;
            uint32_t w[12];
            if (kSg) block_pairs_sg(fa, T, stream, sg, b, row, in, w);
            else block_pairs<kBig>(fa, T, stream, gain, b, in, w);
            // the MMAs of this group's previous stage read its buffers: wait for them only now, with the block already unranked
            if (uses > 0 && !mbar_wait(&bar_free[group], (uses - 1u) & 1u)) timeout = true;
            uint8_t* a_dst = a_mine + gwarp * 128 + (lane & 7) * 16;
#pragma unroll
            for (int j = 0; j < 3; ++j)
                *reinterpret_cast<uint4*>(a_dst + (3 * (lane >> 3) + j) * 2048) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            // ---- B: the slice of X, 16-byte chunks (8 values along K)
            for (int i = gtid; i < ga.npad * (kStageK / 8); i += kGemmGroupThreads) {
                const int kc = i / ga.npad, n = i % ga.npad;
                const int64_t k = (int64_t)s * kStageK + kc * 8;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (n < ga.batch && k < ga.k_in) v = __ldg(reinterpret_cast<const uint4*>(ga.x + (int64_t)n * ga.k_in + k));
                *reinterpret_cast<uint4*>(b_mine + (uint32_t)kc * ga.npad * 16 + n * 16) = v;
            }
            fence_async_smem();
            group_barrier(group);
            if (gtid == 0) {
                tc_fence_after();
                const uint32_t a_addr = smem_u32(a_mine), b_addr = smem_u32(b_mine);
#pragma unroll
                for (int j = 0; j < kStageK / 16; ++j)
                    umma_bf16(tmem + 64u * group, smem_desc(a_addr + j * 4096, 2048, 128),
                              smem_desc(b_addr + j * 2 * ga.npad * 16, ga.npad * 16, 128), idesc, (s > s_begin + group || j > 0) ? 1u : 0u);
                umma_commit(&bar_free[group]);
                if (s + 2 >= s_end) umma_commit(&bar_done[group]);
            }
        }
        // ---- epilogue: accumulators -> scratch (split-K) or Y
        const bool has0 = s_end > s_begin, has1 = s_end > s_begin + 1;
        if (warp < 4) {
            if (has0 && !mbar_wait(&bar_done[0], done[0] & 1u)) timeout = true;
            if (has1 && !mbar_wait(&bar_done[1], done[1] & 1u)) timeout = true;
            tc_fence_after();
            const int64_t orow = rt * kGemmRows + warp * 32 + lane;
            for (int c0 = 0; c0 < ga.npad && has0; c0 += 16) {
                float v[16], v1[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (has1) {
                    tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + 64u + (uint32_t)c0, v1);
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += v1[i];
                }
                if (orow < ga.n_out) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int n = c0 + i;
                        if (n < ga.batch) {
                            if (ga.split == 1) gemm_store<kShard>(ga, n, orow, v[i]);
                            else atomicAdd(ga.scratch + (int64_t)n * ga.scratch_ld + orow, v[i]);
                        }
                    }
                }
            }
            tc_fence_before();
        }
        done[0] += has0; done[1] += has1;
        if (ga.split > 1) {
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) *last_flag = (atomicAdd(ga.counters + rt, 1u) == (uint32_t)ga.split - 1u);
            __syncthreads();
            if (*last_flag) {
                __threadfence();
                for (int i = threadIdx.x; i < kGemmRows * ga.batch; i += kGemmThreads) {
                    const int n = i / kGemmRows;
                    const int64_t orow = rt * kGemmRows + (i % kGemmRows);
                    if (orow < ga.n_out) {
                        float* sp = ga.scratch + (int64_t)n * ga.scratch_ld + orow;
                        gemm_store<kShard>(ga, n, orow, __ldcg(sp));
                        __stcg(sp, 0.f);
                    }
                }
                if (threadIdx.x == 0) ga.counters[rt] = 0u;
            }
        }
        __syncthreads();
    }
    if (timeout) atomicOr(fa.flags, 1u);
    if (kShard) {
        __threadfence_system();                           // this thread's stores to the peers' copies, before the CTA counts itself in
        shard_arrive(*ga.shard);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ===========================================================================
// Sorted layout for the small-batch GEMM (llvq_sort_blocks_gemm / llvq_gemm_small_batch_sorted).
// A domain is 128 rows x 8 column blocks (1024 blocks, two 96-column MMA stages); the stream holds the domains
// row tile major, each domain's blocks ordered like the GEMV's sorted layout (decoder form, unranking steps,
// class), one 64-bit entry per block: the stored index unchanged (48 bits) + position in the domain (row * 8 +
// column block, 10 bits, stored in the high 16).  The kernel runs the whole CTA on one accumulator: per
// iteration it unranks one domain (padded batch > 32) or two (warp w takes the w-th chunk of the first and the
// (31-w)-th of the second: both are ordered from expensive to cheap, so the pairs balance), writing the bf16
// weights straight to their place in the K-major A tiles, then one thread issues the tcgen05 MMAs of those stages.
// ===========================================================================
constexpr int kDomBlocks = 8;                          // column blocks per domain
constexpr int kDomEntries = kGemmRows * kDomBlocks;    // 1024
constexpr int kDomStages = 2;                          // 96-column MMA stages per domain

__global__ void __launch_bounds__(kDomEntries, 1)
sort_blocks_gemm_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ sort_rank, int gain_bits, int64_t n_out,
                        int64_t bpr, int64_t ndomains, unsigned long long* __restrict__ out)
{
    FAST_PROLOGUE();
    __shared__ uint32_t hist[1024], cursor[1024];
    const int64_t nd = (bpr + kDomBlocks - 1) / kDomBlocks;
    for (int64_t dom = blockIdx.x; dom < ndomains; dom += gridDim.x) {
        hist[threadIdx.x] = 0; cursor[threadIdx.x] = 0;
        __syncthreads();
        const int64_t rt = dom / nd, d = dom - rt * nd;
        const int i = threadIdx.x;
        const int64_t row = rt * kGemmRows + (i >> 3), cb = d * kDomBlocks + (i & 7);
        unsigned long long field = kSortIndexMask;
        uint32_t key = 1023u;
        if (row < n_out && cb < bpr) {
            const uint64_t f = load_field(stream, (uint64_t)(row * bpr + cb), (int)fa.L.W + gain_bits);   // shape index | gain index << W
            const uint64_t I = f & ((1ull << fa.L.W) - 1ull);
            if (I < fa.n_points) {
                uint64_t local;
                field = f;
                key = __ldg(sort_rank + fast_find_class(T, I, local));
            } else {
                atomicAdd(fa.bad_index, 1ull);
            }
        }
        atomicAdd(&hist[key], 1u);
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (int k = 0; k < 1024; ++k) { const uint32_t c = hist[k]; hist[k] = run; run += c; }
        }
        __syncthreads();
        const uint32_t slot = hist[key] + atomicAdd(&cursor[key], 1u);
        out[dom * kDomEntries + slot] = field | (unsigned long long)i << 48;
        __syncthreads();
    }
}

// The same layout for codes whose class tables live in global memory (72-bit indices): 128-bit entries, x = the low 64
// bits of the stored index, y = its bits 64.. (8 bits) | class << 8 (24 bits) | position in the domain << 32 (10 bits);
// bit 63 of y marks "no block" (ragged edge or index out of range).  The class rides along so that the GEMM kernel does
// not search for it again; the blocks of a domain are ordered by unranking steps (most first), then by class, so that
// the lanes of a warp run the same trip counts and read neighbouring class descriptors.
constexpr unsigned long long kBigNoBlock = 1ull << 63;

__global__ void __launch_bounds__(kDomEntries, 1)
sort_blocks_gemm_big_kernel(FastArgs fa, const uint32_t* __restrict__ stream, int64_t n_out, int64_t bpr, int64_t ndomains,
                            ulonglong2* __restrict__ out)
{
    __shared__ uint32_t keys[kDomEntries];
    __shared__ unsigned long long ex[kDomEntries], ey[kDomEntries];
    const int64_t nd = (bpr + kDomBlocks - 1) / kDomBlocks;
    const int i = threadIdx.x;
    for (int64_t dom = blockIdx.x; dom < ndomains; dom += gridDim.x) {
        const int64_t rt = dom / nd, d = dom - rt * nd;
        const int64_t row = rt * kGemmRows + (i >> 3), cb = d * kDomBlocks + (i & 7);
        unsigned long long x = 0ull, y = kBigNoBlock | (unsigned long long)i << 32;
        uint32_t key = 0x7ffffc00u | (uint32_t)i;                   // no block: after everything else
        if (row < n_out && cb < bpr) {
            uint64_t lo, hi;
            load_index(stream, (uint64_t)(row * bpr + cb), fa.dc.W, lo, hi);
            if (hi < fa.dc.n_hi || (hi == fa.dc.n_hi && lo < fa.dc.n_lo)) {
                uint64_t local;
                const uint32_t cls = (uint32_t)big_find_class(fa.dc, lo, hi, local);
                const uint32_t h0y = __ldg(reinterpret_cast<const uint32_t*>(fa.dc.cls + cls) + 1);
                const uint32_t nlev = (h0y & 0xff) + ((h0y >> 8) & 0xff);
                x = lo;
                y = (hi & 0xffull) | (unsigned long long)cls << 8 | (unsigned long long)i << 32;
                key = (15u - min(nlev, 15u)) << 27 | cls << 10 | (uint32_t)i;
            } else {
                atomicAdd(fa.bad_index, 1ull);
            }
        }
        keys[i] = key; ex[i] = x; ey[i] = y;
        __syncthreads();
        for (int k = 2; k <= kDomEntries; k <<= 1)                   // bitonic sort of the 1024 keys
            for (int j = k >> 1; j > 0; j >>= 1) {
                const int o = i ^ j;
                if (o > i) {
                    const uint32_t a = keys[i], b = keys[o];
                    if ((a > b) == ((i & k) == 0)) { keys[i] = b; keys[o] = a; }
                }
                __syncthreads();
            }
        const uint32_t src = keys[i] & 1023u;
        out[dom * kDomEntries + i] = make_ulonglong2(ex[src], ey[src]);
        __syncthreads();
    }
}

template <bool kBig, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_sorted_kernel(FastArgs fa, const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, SgArgs sg, GemmArgs ga, int dpi)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t img_bytes = fa.L.total;
    uint64_t* bar_img = reinterpret_cast<uint64_t*>(smem + img_bytes);
    uint64_t* bar_free = bar_img + 1;                                     // the MMAs reading the A / B buffers are done
    uint64_t* bar_done = bar_img + 2;                                     // the accumulator of this item is complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_img + 5);
    uint32_t* last_flag = tmem_slot + 1;
    const uint32_t a_off = (img_bytes + 64 + 1023) & ~1023u;
    constexpr uint32_t kAStage = kGemmRows * kStageK * 2;                  // 24576
    uint8_t* a_buf = smem + a_off;                                        // [dpi * 2 stages] x 24576
    const uint32_t b_stage = (uint32_t)ga.npad * kStageK * 2;
    uint8_t* b_buf = a_buf + (uint32_t)dpi * kDomStages * kAStage;         // [dpi * 2 stages] x npad * 192

    pdl_launch_dependents();
    if (!fast_load_image(smem, fa.image, fa.L.total, bar_img, fa.flags)) return;
    pdl_wait();
    const FastSmem T = fast_view(smem, fa.L);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(bar_free, 1); mbar_init(bar_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t idesc = instr_desc_bf16_m128((uint32_t)ga.npad);
    const int64_t row_tiles = (ga.n_out + kGemmRows - 1) / kGemmRows;
    const int64_t nd = ga.nstages;                                         // domains per row tile
    // every CTA takes an equal contiguous range of the row_tiles * nd domains (row tile major); the parts of a row
    // tile that end up in different CTAs are summed through the scratch, as in the GEMV
    const int64_t D = row_tiles * nd, G = gridDim.x;
    const int64_t dom_begin = blockIdx.x * D / G, dom_end = (blockIdx.x + 1) * D / G;
    uint32_t uses = 0, done = 0;
    bool timeout = false;
    for (int64_t rt = dom_begin / nd; rt * nd < dom_end; ++rt) {
        const int d_begin = (int)(max(dom_begin, rt * nd) - rt * nd), d_end = (int)(min(dom_end, (rt + 1) * nd) - rt * nd);
        const uint32_t parts = (uint32_t)(unit_owner((rt + 1) * nd - 1, D, G) - unit_owner(rt * nd, D, G) + 1);   // CTAs that share this row tile
        // the entries of an iteration are requested one iteration ahead (they come from DRAM)
        const ulonglong2 no_entry = make_ulonglong2(kSortIndexMask, kBigNoBlock);
        auto entry_at = [&](int d, int q) {
            if (d + q >= d_end) return no_entry;
            // warp 0 also issues the MMAs of every iteration: it takes the cheapest chunk of each domain (the last), the other
            // warps pair chunk w - 1 of the first domain with chunk 31 - w of the second
            const int chunk = warp == 0 ? 31 : (q == 0 ? warp - 1 : 31 - warp);
            const int64_t at = (rt * nd + d + q) * kDomEntries + chunk * 32 + lane;
            if (kBig) return __ldg(reinterpret_cast<const ulonglong2*>(sorted) + at);
            return make_ulonglong2(__ldg(sorted + at), 0ull);
        };
        ulonglong2 e0 = entry_at(d_begin, 0), e1 = dpi > 1 ? entry_at(d_begin, 1) : no_entry;
        for (int d0 = d_begin; d0 < d_end; d0 += dpi, ++uses) {
            const int nd_now = min(dpi, d_end - d0);
            const ulonglong2 cur0 = e0, cur1 = e1;
            e0 = entry_at(d0 + dpi, 0);
            if (dpi > 1) e1 = entry_at(d0 + dpi, 1);
            // ---- A: every warp unranks one chunk of 32 sorted entries per domain
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (q >= nd_now) break;
                const ulonglong2 e = q == 0 ? cur0 : cur1;
                const uint64_t field = e.x & kSortIndexMask;
                const uint64_t I = kSg ? field & ((1ull << fa.L.W) - 1ull) : field;     // shape-gain form: gain index above the shape index
                const uint32_t pos = kBig ? (uint32_t)(e.y >> 32) & 1023u : (uint32_t)(e.x >> 48);
                const bool valid = kBig ? !(e.y >> 63) : (field != kSortIndexMask && I < fa.n_points);
                const uint32_t r = pos >> 3, c = pos & 7u;
                const int64_t row = rt * kGemmRows + r, cb = (int64_t)(d0 + q) * kDomBlocks + c;
                float gn = (!kSg && valid) ? gain_to_float(__ldg(gain + row * ga.bpr + cb)) : 0.f;
                uint32_t w[12];
                if (kBig) {
                    const int cls = valid ? (int)((uint32_t)(e.y >> 8) & 0xffffffu) : 0;
                    const uint64_t local = valid ? e.x - __ldg(fa.dc.off_lo + cls) : 0ull;     // class sizes fit 63 bits: exact mod 2^64
                    Point pt;
                    big_decode_local(T, fa.dc, cls, local, valid, pt);
#pragma unroll
                    for (int j = 0; j < 12; ++j) {
                        __nv_bfloat162 h = __halves2bfloat162(dequant(gn, pt, 2 * j), dequant(gn, pt, 2 * j + 1));
                        w[j] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
                    Decoded dec;
                    const uint32_t cls = decode_sorted_entry(fa, T, I, valid, dec);
                    if (kSg && valid) {
                        const float scale = sg.row_scale ? __ldg(sg.row_scale + row) : 1.f;
                        gn = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + (uint32_t)(field >> fa.L.W))),
                                       __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
                    }
                    expand_bf16(dec, gn, w);
                }
                // the previous MMAs read the buffers: wait for them only now, with the first chunk already unranked
                if (q == 0 && uses > 0 && !mbar_wait(bar_free, (uses - 1u) & 1u)) timeout = true;
                uint8_t* a_dst = a_buf + (uint32_t)(q * kDomStages + (c >> 2)) * kAStage + (r >> 3) * 128u + (r & 7u) * 16u + 3u * (c & 3u) * 2048u;
#pragma unroll
                for (int j = 0; j < 3; ++j)
                    *reinterpret_cast<uint4*>(a_dst + j * 2048) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            }
            // ---- B: the slice of X of these stages, 16-byte chunks (8 values along K)
            const int kchunks = nd_now * kDomStages * (kStageK / 8);
            for (int i = threadIdx.x; i < ga.npad * kchunks; i += kGemmThreads) {
                const int kc = i / ga.npad, n = i % ga.npad;
                const int64_t k = (int64_t)d0 * kDomBlocks * 24 + (int64_t)kc * 8;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (n < ga.batch && k < ga.k_in) v = __ldg(reinterpret_cast<const uint4*>(ga.x + (int64_t)n * ga.k_in + k));
                *reinterpret_cast<uint4*>(b_buf + (uint32_t)(kc / (kStageK / 8)) * b_stage + (uint32_t)(kc % (kStageK / 8)) * ga.npad * 16 + n * 16) = v;
            }
            fence_async_smem();
            __syncthreads();
            if (threadIdx.x == 0) {
                tc_fence_after();
                const uint32_t a_addr = smem_u32(a_buf), b_addr = smem_u32(b_buf);
                for (int st = 0; st < nd_now * kDomStages; ++st)
#pragma unroll
                    for (int j = 0; j < kStageK / 16; ++j)
                        umma_bf16(tmem, smem_desc(a_addr + st * kAStage + j * 4096, 2048, 128),
                                  smem_desc(b_addr + st * b_stage + j * 2 * ga.npad * 16, ga.npad * 16, 128), idesc,
                                  (d0 > d_begin || st > 0 || j > 0) ? 1u : 0u);
                umma_commit(bar_free);
                if (d0 + dpi >= d_end) umma_commit(bar_done);
            }
        }
        // ---- epilogue: accumulator -> scratch (split-K) or Y
        const bool has = d_end > d_begin;
        if (warp < 4 && has) {
            if (!mbar_wait(bar_done, done & 1u)) timeout = true;
            tc_fence_after();
            const int64_t orow = rt * kGemmRows + warp * 32 + lane;
            for (int c0 = 0; c0 < ga.npad; c0 += 16) {
                float v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (orow < ga.n_out) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int n = c0 + i;
                        if (n < ga.batch) {
                            if (parts == 1u) gemm_store<kShard>(ga, n, orow, v[i]);
                            else atomicAdd(ga.scratch + (int64_t)n * ga.scratch_ld + orow, v[i]);
                        }
                    }
                }
            }
            tc_fence_before();
        }
        done += has;
        if (parts > 1u) {
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) *last_flag = (atomicAdd(ga.counters + rt, 1u) == parts - 1u);
            __syncthreads();
            if (*last_flag) {
                __threadfence();
                for (int i = threadIdx.x; i < kGemmRows * ga.batch; i += kGemmThreads) {
                    const int n = i / kGemmRows;
                    const int64_t orow = rt * kGemmRows + (i % kGemmRows);
                    if (orow < ga.n_out) {
                        float* sp = ga.scratch + (int64_t)n * ga.scratch_ld + orow;
                        gemm_store<kShard>(ga, n, orow, __ldcg(sp));
                        __stcg(sp, 0.f);
                    }
                }
                if (threadIdx.x == 0) ga.counters[rt] = 0u;
            }
        }
        __syncthreads();
    }
    if (timeout) atomicOr(fa.flags, 1u);
    if (kShard) {
        __threadfence_system();                           // this thread's stores to the peers' copies, before the CTA counts itself in
        shard_arrive(*ga.shard);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// The same product for padded batch <= 32, where two domains' tiles fit: the two buffer sets alternate between
// consecutive domains and nobody waits for the whole CTA.  Warps 1..31 unrank: the chunks of 32 sorted entries of a
// row tile are handed out by a ticket counter (ticket t = chunk t % 32 of the tile's domain t / 32, so from expensive
// to cheap inside a domain), a warp always holding its next ticket with that chunk's entries already requested.
// It unranks the chunk, waits (rarely) until the MMAs that read this buffer two domains ago are done, writes its
// part of A and arrives on the buffer's "full" barrier.  Warp 0 stages the X slice of the next domain, arrives too,
// and its first thread issues the MMAs of a domain as soon as that barrier completes.
// kStored: the same structure on the stored stream (`sorted` then points at it): a chunk is 32 consecutive blocks of the
// domain in natural order (4 rows x 8 column blocks), unranked by the any-class decoder.
template <bool kBig, bool kSg = false, bool kShard = false, bool kStored = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_pipe_kernel(FastArgs fa, const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, SgArgs sg, GemmArgs ga,
                 int b_double)
{
    static_assert(!(kStored && kBig && kSg), "no shape-gain form for the codes with tables in global memory");
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t img_bytes = fa.L.total;
    uint64_t* bar_img = reinterpret_cast<uint64_t*>(smem + img_bytes);
    uint64_t* bar_full = bar_img + 1;                                     // [2] 32 chunks of A and the X slice are in the buffer
    uint64_t* bar_free = bar_img + 3;                                     // [2] the MMAs reading the buffer are done
    uint64_t* bar_done = bar_img + 5;                                     // the accumulator of this row tile is complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_img + 6);
    uint32_t* last_flag = tmem_slot + 1;
    uint32_t* ticket = tmem_slot + 2;                                     // next chunk ticket of the row tile in progress
    const uint32_t a_off = (img_bytes + 64 + 1023) & ~1023u;
    constexpr uint32_t kAStage = kGemmRows * kStageK * 2;                  // 24576
    uint8_t* a_buf = smem + a_off;                                        // [2 buffers][2 stages] x 24576
    const uint32_t b_stage = (uint32_t)ga.npad * kStageK * 2;
    uint8_t* b_buf = a_buf + 2u * kDomStages * kAStage;                    // [2 buffers, or 1][2 stages] x npad * 192
    constexpr uint32_t kWorkers = kGemmThreads / 32 - 1;                   // 31 unranking warps

    pdl_launch_dependents();
    if (!fast_load_image(smem, fa.image, fa.L.total, bar_img, fa.flags)) return;
    pdl_wait();
    const FastSmem T = fast_view(smem, fa.L);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(bar_full, 33); mbar_init(bar_full + 1, 33);             // 32 chunks + the X slice
        mbar_init(bar_free, 1); mbar_init(bar_free + 1, 1); mbar_init(bar_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t idesc = instr_desc_bf16_m128((uint32_t)ga.npad);
    const int64_t row_tiles = (ga.n_out + kGemmRows - 1) / kGemmRows;
    const int64_t nd = ga.nstages;                                         // domains per row tile
    const int64_t D = row_tiles * nd, G = gridDim.x;
    const int64_t dom_begin = blockIdx.x * D / G, dom_end = (blockIdx.x + 1) * D / G;
    uint32_t g_base = 0, done = 0;                                         // domains this CTA has finished (domain g uses buffer g & 1 for the (g >> 1)-th time)
    bool timeout = false;
    const ulonglong2 no_entry = make_ulonglong2(kSortIndexMask, kBigNoBlock);
    auto arrive_full = [&](uint32_t b) {
        fence_async_smem();
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar_full + b)) : "memory");
    };

    for (int64_t rt = dom_begin / nd; rt * nd < dom_end; ++rt) {
        const int d_begin = (int)(max(dom_begin, rt * nd) - rt * nd), d_end = (int)(min(dom_end, (rt + 1) * nd) - rt * nd);
        const uint32_t parts = (uint32_t)(unit_owner((rt + 1) * nd - 1, D, G) - unit_owner(rt * nd, D, G) + 1);   // CTAs that share this row tile
        const uint32_t n_dom = (uint32_t)(d_end - d_begin), n_tickets = n_dom * 32u;
        if (threadIdx.x == 0) *ticket = kWorkers;                          // the first tickets are the workers' own numbers
        __syncthreads();
        if (warp == 0) {
            // ---- X slices and MMAs
            // the slice of domain j of this tile, 16-byte chunks (8 values along K).  With two X buffers it may be written once
            // the MMAs of two domains ago are done; with one (wide batches: no room for two), only after the previous domain's
            auto stage_b = [&](uint32_t j) {
                const uint32_t gd = g_base + j, b = gd & 1u, bx = b_double ? b : 0u;
                if (b_double) { if (gd >= 2u && !mbar_wait(bar_free + b, ((gd >> 1) - 1u) & 1u)) timeout = true; }
                else if (gd >= 1u && !mbar_wait(bar_free + ((gd - 1u) & 1u), ((gd - 1u) >> 1) & 1u)) timeout = true;
                const int64_t k0 = (int64_t)(d_begin + (int)j) * kDomBlocks * 24;
                for (int n = lane; n < ga.npad; n += 32) {
                    const uint16_t* xr = ga.x + (int64_t)n * ga.k_in + k0;
                    uint8_t* dst = b_buf + bx * kDomStages * b_stage + n * 16;
#pragma unroll 4
                    for (int kc = 0; kc < kDomStages * (kStageK / 8); ++kc) {        // 24 asynchronous 16-byte copies per row, zero-filled outside X
                        const bool in = n < ga.batch && k0 + kc * 8 < ga.k_in;
                        const uint32_t to = smem_u32(dst + (uint32_t)(kc / (kStageK / 8)) * b_stage + (uint32_t)(kc % (kStageK / 8)) * ga.npad * 16);
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(to), "l"(in ? xr + kc * 8 : ga.x), "r"(in ? 16u : 0u) : "memory");
                    }
                }
                asm volatile("cp.async.wait_all;" ::: "memory");
                arrive_full(b);
            };
            if (n_dom > 0) stage_b(0);
            for (uint32_t j = 0; j < n_dom; ++j) {
                if (b_double && j + 1 < n_dom) stage_b(j + 1);
                const uint32_t gd = g_base + j, b = gd & 1u, bx = b_double ? b : 0u;
                if (lane == 0) {
                    if (!mbar_wait(bar_full + b, (gd >> 1) & 1u)) timeout = true;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(a_buf) + b * kDomStages * kAStage, b_addr = smem_u32(b_buf) + bx * kDomStages * b_stage;
                    for (int st = 0; st < kDomStages; ++st)
#pragma unroll
                        for (int jj = 0; jj < kStageK / 16; ++jj)
                            umma_bf16(tmem, smem_desc(a_addr + st * kAStage + jj * 4096, 2048, 128),
                                      smem_desc(b_addr + st * b_stage + jj * 2 * ga.npad * 16, ga.npad * 16, 128), idesc,
                                      (j > 0 || st > 0 || jj > 0) ? 1u : 0u);
                    umma_commit(bar_free + b);
                    if (j + 1 == n_dom) umma_commit(bar_done);
                }
                __syncwarp();
                if (!b_double && j + 1 < n_dom) stage_b(j + 1);
            }
        } else {
            // ---- A: unrank chunks until the tile's tickets are gone
            auto entry_of = [&](uint32_t t) {
                if (t >= n_tickets) return no_entry;
                if (kStored && kBig) {                                       // the index itself, in the form of the sorted layout's entries
                    const uint32_t pos = (t & 31u) * 32u + lane;
                    const int64_t row = rt * kGemmRows + (pos >> 3), cb = (int64_t)(d_begin + (int)(t >> 5)) * kDomBlocks + (pos & 7u);
                    uint64_t lo = 0, hi = kBigNoBlock;
                    if (row < ga.n_out && cb < ga.bpr) load_index(reinterpret_cast<const uint32_t*>(sorted), (uint64_t)(row * ga.bpr + cb), fa.dc.W, lo, hi);
                    return make_ulonglong2(lo, hi | (unsigned long long)pos << 32);
                }
                if (kStored) {                                               // the field itself, its position in the high 16 bits
                    const uint32_t pos = (t & 31u) * 32u + lane;
                    const int64_t row = rt * kGemmRows + (pos >> 3), cb = (int64_t)(d_begin + (int)(t >> 5)) * kDomBlocks + (pos & 7u);
                    unsigned long long f = kSortIndexMask;
                    if (row < ga.n_out && cb < ga.bpr)
                        f = load_field(reinterpret_cast<const uint32_t*>(sorted), (uint64_t)(row * ga.bpr + cb), (int)fa.L.W + (kSg ? sg.bits : 0));
                    return make_ulonglong2(f | (unsigned long long)pos << 48, 0ull);
                }
                const int64_t at = (rt * nd + d_begin + (int)(t >> 5)) * kDomEntries + (t & 31u) * 32u + lane;
                if (kBig) return __ldg(reinterpret_cast<const ulonglong2*>(sorted) + at);
                return make_ulonglong2(__ldg(sorted + at), 0ull);
            };
            uint32_t tk = (uint32_t)warp - 1u;
            ulonglong2 e = entry_of(tk);
            while (tk < n_tickets) {
                uint32_t tk_next = 0;
                if (lane == 0) tk_next = atomicAdd(ticket, 1u);
                tk_next = __shfl_sync(kFullMask, tk_next, 0);
                const ulonglong2 e_next = entry_of(tk_next);                // requested a chunk ahead (it comes from DRAM)
                const uint32_t j = tk >> 5, gd = g_base + j, b = gd & 1u;
                const int d = d_begin + (int)j;
                const uint64_t field = e.x & kSortIndexMask;
                const uint64_t I = kSg ? field & ((1ull << fa.L.W) - 1ull) : field;     // shape-gain form: gain index above the shape index
                const uint32_t pos = kBig ? (uint32_t)(e.y >> 32) & 1023u : (uint32_t)(e.x >> 48);
                bool valid = kBig ? !(e.y >> 63) : (field != kSortIndexMask && I < fa.n_points);
                if (kStored && kBig && valid) {                               // the stored index may be out of range: count it, treat it as no block
                    const uint64_t hi = e.y & 0xffull;
                    valid = hi < fa.dc.n_hi || (hi == fa.dc.n_hi && e.x < fa.dc.n_lo);
                    if (!valid) atomicAdd(fa.bad_index, 1ull);
                }
                const uint32_t r = pos >> 3, c = pos & 7u;
                const int64_t row = rt * kGemmRows + r, cb = (int64_t)d * kDomBlocks + c;
                float gn = (!kSg && valid) ? gain_to_float(__ldg(gain + row * ga.bpr + cb)) : 0.f;
                uint32_t w[12];
                if (kBig) {
                    int cls = 0;
                    uint64_t local = 0;
                    if (kStored) { if (valid) cls = big_find_class(fa.dc, e.x, e.y & 0xffull, local); }
                    else if (valid) {
                        cls = (int)((uint32_t)(e.y >> 8) & 0xffffffu);
                        local = e.x - __ldg(fa.dc.off_lo + cls);                 // class sizes fit 63 bits: exact mod 2^64
                    }
                    Point pt;
                    big_decode_local(T, fa.dc, cls, local, valid, pt);
#pragma unroll
                    for (int jj = 0; jj < 12; ++jj) {
                        __nv_bfloat162 h = __halves2bfloat162(dequant(gn, pt, 2 * jj), dequant(gn, pt, 2 * jj + 1));
                        w[jj] = *reinterpret_cast<uint32_t*>(&h);
                    }
                } else {
                    Decoded dec;
                    uint32_t cls;
                    if (kStored) {
                        if (field != kSortIndexMask && !valid) atomicAdd(fa.bad_index, 1ull);
                        uint64_t local = 0;
                        cls = valid ? fast_find_class(T, I, local) : 0u;
                        fast_decode_local<-1>(T, cls, local, valid, kFullMask, dec);
                    } else {
                        cls = decode_sorted_entry(fa, T, I, valid, dec);
                    }
                    if (kSg && valid) {
                        const float scale = sg.row_scale ? __ldg(sg.row_scale + row) : 1.f;
                        gn = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + (uint32_t)(field >> fa.L.W))),
                                       __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
                    }
                    expand_bf16(dec, gn, w);
                }
                // the MMAs of two domains ago read this buffer: wait for them only now, with the chunk already unranked
                if (gd >= 2u && !mbar_wait(bar_free + b, ((gd >> 1) - 1u) & 1u)) timeout = true;
                uint8_t* a_dst = a_buf + (b * kDomStages + (c >> 2)) * kAStage + (r >> 3) * 128u + (r & 7u) * 16u + 3u * (c & 3u) * 2048u;
#pragma unroll
                for (int jj = 0; jj < 3; ++jj)
                    *reinterpret_cast<uint4*>(a_dst + jj * 2048) = make_uint4(w[4 * jj], w[4 * jj + 1], w[4 * jj + 2], w[4 * jj + 3]);
                arrive_full(b);
                tk = tk_next; e = e_next;
            }
        }
        g_base += n_dom;
        const bool has = d_end > d_begin;
        // ---- epilogue: accumulator -> scratch (split-K) or Y
        if (warp < 4 && has) {
            if (!mbar_wait(bar_done, done & 1u)) timeout = true;
            tc_fence_after();
            const int64_t orow = rt * kGemmRows + warp * 32 + lane;
            for (int c0 = 0; c0 < ga.npad; c0 += 16) {
                float v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (orow < ga.n_out) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int n = c0 + i;
                        if (n < ga.batch) {
                            if (parts == 1u) gemm_store<kShard>(ga, n, orow, v[i]);
                            else atomicAdd(ga.scratch + (int64_t)n * ga.scratch_ld + orow, v[i]);
                        }
                    }
                }
            }
            tc_fence_before();
        }
        done += has;
        if (parts > 1u) {
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) *last_flag = (atomicAdd(ga.counters + rt, 1u) == parts - 1u);
            __syncthreads();
            if (*last_flag) {
                __threadfence();
                for (int i = threadIdx.x; i < kGemmRows * ga.batch; i += kGemmThreads) {
                    const int n = i / kGemmRows;
                    const int64_t orow = rt * kGemmRows + (i % kGemmRows);
                    if (orow < ga.n_out) {
                        float* sp = ga.scratch + (int64_t)n * ga.scratch_ld + orow;
                        gemm_store<kShard>(ga, n, orow, __ldcg(sp));
                        __stcg(sp, 0.f);
                    }
                }
                if (threadIdx.x == 0) ga.counters[rt] = 0u;
            }
        }
        __syncthreads();
    }
    if (timeout) atomicOr(fa.flags, 1u);
    if (kShard) {
        __threadfence_system();                           // this thread's stores to the peers' copies, before the CTA counts itself in
        shard_arrive(*ga.shard);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

FastArgs fast_args(const llvq_ctx* ctx)
{
    FastArgs fa;
    fa.L = ctx->fl; fa.image = ctx->d_image; fa.flags = ctx->dev.flags; fa.bad_index = ctx->dev.bad_index;
    fa.n_points = ctx->dev.n_lo;
    fa.dc = ctx->dev;
    return fa;
}

// Launch with programmatic stream serialization allowed (see pdl_wait above).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename K>
bool set_smem(K kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

int check_common(const llvq_ctx* ctx, const void* d_idx)
{
    if (!ctx || !d_idx || ctx->device < 0) return LLVQ_EINVAL;
    if (!aligned(d_idx, 16)) return LLVQ_EALIGN;
    return LLVQ_OK;
}

int launch_status();

int check_gemm_args(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                    const uint16_t* d_x_bf16, int batch, const uint16_t* d_y_bf16)
{
    if (ctx && ctx->device >= 0 && n_out == 0 && batch >= 1 && batch <= 64) return LLVQ_OK;   // nothing to do: pointers may be null
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_gain_f16 || !d_x_bf16 || !d_y_bf16 || n_out < 0 || k_in < 0 || batch < 1 || batch > 64) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2) || !aligned(d_x_bf16, 16) || !aligned(d_y_bf16, 2) || (k_in & 7)) return LLVQ_EALIGN;
    return LLVQ_OK;
}

// Enqueue gemm_sorted_kernel on a stream sorted by llvq_sort_blocks_gemm.
int launch_gemm_domains(const llvq_ctx* ctx, const void* p, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                        const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, float* scratch, uint32_t* counters, void* stream,
                        const YOut* yo = nullptr, int64_t y_ld = 0, const SgArgs* sg = nullptr)
{
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    GemmArgs ga;
    ga.y = d_y_bf16; ga.y_ld = n_out; ga.shard = nullptr;
    if (yo) {                                             // the description travels ahead of the kernel on the same stream
        ga.y = static_cast<uint16_t*>(yo->y); ga.y_ld = y_ld; ga.shard = static_cast<const YOut*>(ctx->d_shard);
        put_shard_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(*yo, static_cast<YOut*>(ctx->d_shard));   // by value: safe under stream capture
    }
    ga.n_out = n_out; ga.k_in = k_in; ga.bpr = (k_in + 23) / 24;
    ga.batch = batch; ga.npad = (batch + 15) / 16 * 16;
    ga.nstages = (int)((ga.bpr + kDomBlocks - 1) / kDomBlocks);              // domains per row tile
    ga.x = d_x_bf16; ga.scratch = scratch; ga.counters = counters;
    int dpi = ga.npad <= 32 ? 2 : 1;                                         // gemm_sorted_kernel: domains unranked per iteration (shared memory decides)
    const int64_t row_tiles = (n_out + kGemmRows - 1) / kGemmRows;
    ga.scratch_ld = row_tiles * kGemmRows;
    ga.split = 1;                                                             // unused: the kernel balances domains over the CTAs itself
    const unsigned grid = (unsigned)std::min<int64_t>(row_tiles * ga.nstages, ctx->sm_count);
    // gemm_pipe_kernel: two A buffer sets and two X buffer sets, or one X set when two do not fit; else the kernel with the block barrier
    const size_t head = (ctx->fl.total + 64 + 1023) & ~size_t(1023), a_set = (size_t)kDomStages * kGemmRows * kStageK * 2,
                 x_set = (size_t)kDomStages * ga.npad * kStageK * 2;
    int pipe = 0, b_double = 0;
    size_t smem = head + (size_t)dpi * (a_set + x_set);
    if (!ctx->fast) {}                                   // the 72-bit code gains nothing from the pipeline (measured): it keeps the kernel below
    else if (head + 2 * a_set + 2 * x_set <= 227 * 1024) { pipe = 1; b_double = 1; smem = head + 2 * a_set + 2 * x_set; }
    else if (head + 2 * a_set + x_set <= 227 * 1024) { pipe = 1; smem = head + 2 * a_set + x_set; }
    if (smem > 227 * 1024) return LLVQ_EUNSUPPORTED;
#define LLVQ_LAUNCH_DOMAINS(BIG, SG, SH)                                                                                      \
    do {                                                                                                                     \
        if (pipe) {                                                                                                          \
            if (!set_smem(gemm_pipe_kernel<BIG, SG, SH>, smem)) return LLVQ_ECUDA;                                            \
            if (launch_pdl(gemm_pipe_kernel<BIG, SG, SH>, grid, (unsigned)kGemmThreads, smem, (cudaStream_t)stream, fast_args(ctx), \
                           static_cast<const unsigned long long*>(p), d_gain_f16, sga, ga, b_double) != cudaSuccess) return LLVQ_ECUDA; \
        } else {                                                                                                             \
            if (!set_smem(gemm_sorted_kernel<BIG, SG, SH>, smem)) return LLVQ_ECUDA;                                          \
            if (launch_pdl(gemm_sorted_kernel<BIG, SG, SH>, grid, (unsigned)kGemmThreads, smem, (cudaStream_t)stream, fast_args(ctx), \
                           static_cast<const unsigned long long*>(p), d_gain_f16, sga, ga, dpi) != cudaSuccess) return LLVQ_ECUDA; \
        }                                                                                                                    \
    } while (0)
    const SgArgs sga = sg ? *sg : SgArgs{};
    if (yo) {                                            // row-sharded: stored-gain form only
        if (sg) return LLVQ_EUNSUPPORTED;
        if (ctx->fast) LLVQ_LAUNCH_DOMAINS(false, false, true); else LLVQ_LAUNCH_DOMAINS(true, false, true);
    } else if (sg) {
        LLVQ_LAUNCH_DOMAINS(false, true, false);
    } else if (ctx->fast) {
        LLVQ_LAUNCH_DOMAINS(false, false, false);
    } else {
        LLVQ_LAUNCH_DOMAINS(true, false, false);
    }
#undef LLVQ_LAUNCH_DOMAINS
    return launch_status();
}

// Enqueue the small-batch GEMM with the given split-K scratch ([npad][row tiles * 128] floats) and counters
// ([row tiles]); both must be zero when the kernel starts and are zero again when it ends.
int launch_gemm(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, float* scratch, uint32_t* counters, void* stream,
                const SgArgs* sg = nullptr, const YOut* yo = nullptr, int64_t y_ld = 0)
{
    if (n_out == 0) return LLVQ_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (k_in == 0) return cudaMemsetAsync(d_y_bf16, 0, (size_t)n_out * batch * 2, st) == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
    GemmArgs ga;
    ga.y = d_y_bf16; ga.y_ld = n_out; ga.shard = nullptr;
    if (yo) {                                             // the description travels ahead of the kernel on the same stream
        ga.y = static_cast<uint16_t*>(yo->y); ga.y_ld = y_ld; ga.shard = static_cast<const YOut*>(ctx->d_shard);
        put_shard_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(*yo, static_cast<YOut*>(ctx->d_shard));   // by value: safe under stream capture
    }
    ga.n_out = n_out; ga.k_in = k_in; ga.bpr = (k_in + 23) / 24;
    ga.batch = batch; ga.npad = (batch + 15) / 16 * 16;
    ga.nstages = (int)((ga.bpr + kStageBlocks - 1) / kStageBlocks);
    ga.x = d_x_bf16; ga.scratch = scratch; ga.counters = counters;
    // split K so that the work items fill the SMs evenly, keeping at least four stages per item
    const int64_t row_tiles = (n_out + kGemmRows - 1) / kGemmRows;
    ga.scratch_ld = row_tiles * kGemmRows;
    int best = 1; double best_eff = 0.0;
    for (int f = 1; f <= 64 && f * 4 <= std::max(ga.nstages, 4); ++f) {
        const int64_t items = row_tiles * f;
        const double eff = (double)items / (double)(((items + ctx->sm_count - 1) / ctx->sm_count) * ctx->sm_count);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = f; }
    }
    ga.split = best;
    const int64_t items = row_tiles * ga.split;
    const unsigned grid = (unsigned)std::min<int64_t>(items, ctx->sm_count);
    const size_t img = ctx->fl.total;
    const size_t smem = ((img + 64 + 1023) & ~size_t(1023)) + 2 * kGemmRows * kStageK * 2 + 2 * (size_t)ga.npad * kStageK * 2;
    if (smem > 227 * 1024) return LLVQ_EUNSUPPORTED;
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    if (yo && sg) return LLVQ_EUNSUPPORTED;              // row-sharded: stored-gain form only
    {
        // the kernel without a block barrier (see gemm_pipe_kernel), if its buffers fit
        const size_t head = (img + 64 + 1023) & ~size_t(1023), a_set = (size_t)kDomStages * kGemmRows * kStageK * 2,
                     x_set = (size_t)kDomStages * ga.npad * kStageK * 2;
        const int b_double = head + 2 * a_set + 2 * x_set <= 227 * 1024;
        const size_t smem_pipe = head + 2 * a_set + (b_double ? 2 : 1) * x_set;
        if (smem_pipe <= 227 * 1024 && (ctx->fast || ga.npad <= 32)) {    // 72-bit code at wide batches: slower than gemm_kernel (measured)
            GemmArgs gp = ga;
            gp.nstages = (int)((ga.bpr + kDomBlocks - 1) / kDomBlocks);        // domains per row tile
            gp.split = 1;
            const unsigned grid_pipe = (unsigned)std::min<int64_t>(row_tiles * gp.nstages, ctx->sm_count);
            const unsigned long long* words = static_cast<const unsigned long long*>(d_idx);
            const SgArgs sga = sg ? *sg : SgArgs{};
#define LLVQ_LAUNCH_PIPE_STORED(BIG, SG, SH)                                                                                    \
    do {                                                                                                                        \
        if (!set_smem(gemm_pipe_kernel<BIG, SG, SH, true>, smem_pipe)) return LLVQ_ECUDA;                                        \
        if (launch_pdl(gemm_pipe_kernel<BIG, SG, SH, true>, grid_pipe, (unsigned)kGemmThreads, smem_pipe, st, fast_args(ctx), words, \
                       d_gain_f16, sga, gp, b_double) != cudaSuccess) return LLVQ_ECUDA;                                        \
    } while (0)
            if (!ctx->fast) { if (yo) LLVQ_LAUNCH_PIPE_STORED(true, false, true); else LLVQ_LAUNCH_PIPE_STORED(true, false, false); }
            else if (yo) LLVQ_LAUNCH_PIPE_STORED(false, false, true);
            else if (sg) LLVQ_LAUNCH_PIPE_STORED(false, true, false);
            else LLVQ_LAUNCH_PIPE_STORED(false, false, false);
#undef LLVQ_LAUNCH_PIPE_STORED
            return launch_status();
        }
    }
    if (yo) {
        if (ctx->fast) {
            if (!set_smem(gemm_kernel<false, false, true>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemm_kernel<false, false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
        } else {
            if (!set_smem(gemm_kernel<true, false, true>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemm_kernel<true, false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
        }
    } else if (sg) {
        if (!set_smem(gemm_kernel<false, true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx), idx, d_gain_f16, *sg, ga) != cudaSuccess) return LLVQ_ECUDA;
    } else if (ctx->fast) {
        if (!set_smem(gemm_kernel<false, false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<false, false>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(gemm_kernel<true, false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<true, false>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
    }
    return launch_status();
}

int launch_status()
{
    return cudaGetLastError() == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}

}  // namespace

extern "C" {

int llvq_create(llvq_ctx** out, int m_lo, int m_hi, int device)
{
    if (!out) return LLVQ_EINVAL;
    *out = nullptr;
    llvq_ctx* ctx = new (std::nothrow) llvq_ctx();
    if (!ctx) return LLVQ_ECUDA;
    if (!build_tables(m_lo, m_hi, ctx->host)) { delete ctx; return LLVQ_EUNSUPPORTED; }
    ctx->device = device;
    if (device < 0) { *out = ctx; return LLVQ_OK; }      // host-only context: table queries, no kernels
    DeviceGuard guard(device);
    if (!guard.ok) { delete ctx; return LLVQ_ECUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return LLVQ_ECUDA; }
    ctx->sm_count = prop.multiProcessorCount;

    const HostTables& h = ctx->host;
    const size_t ncls = h.desc.size();
    std::vector<uint64_t> off_lo(ncls + 1);
    std::vector<uint32_t> off_hi(ncls + 1);
    for (size_t j = 0; j <= ncls; ++j) { off_lo[j] = (uint64_t)h.offset[j]; off_hi[j] = (uint32_t)(h.offset[j] >> 64); }
    std::vector<uint8_t> image;
    ctx->fast = build_fast_image(h, ctx->fl, image, true);
    if (!ctx->fast && !build_fast_image(h, ctx->fl, image, false)) { delete ctx; return LLVQ_EUNSUPPORTED; }
    std::vector<uint32_t> lut16;
    build_bucket_table(h, lut16);

    // encoder tables (point -> index), for codes the encoder supports
    std::vector<uint64_t> hkeys; std::vector<uint32_t> hcls;
    std::vector<uint16_t> pos12(4096, 0xffff);
    ctx->can_encode = m_lo == 2 && m_hi >= 6 && h.W <= 64 && build_class_hash(h, hkeys, hcls);
    if (ctx->can_encode) {
        for (uint32_t j = 0; j < 4096; ++j) {
            uint16_t& slot = pos12[h.golay[j] & 0xfffu];
            if (slot != 0xffff) ctx->can_encode = false;       // the low 12 bits must identify the codeword
            slot = (uint16_t)j;
        }
    }
    if (!ctx->can_encode) { hkeys.clear(); hcls.clear(); }
    uint64_t sigs[64];
    for (int a = 0; a < 64; ++a) sigs[a] = sig_of_value(a);

    // one blob: [off_hi | off_lo | classes | bucket table | error words | table image | encoder tables | counters | scratch], 256-byte aligned parts
    auto up = [](size_t v) { return (v + 255) & ~size_t(255); };
    size_t o_offhi = 0;
    size_t o_offlo = up(o_offhi + (ncls + 1) * 4);
    size_t o_cls = up(o_offlo + (ncls + 1) * 8);
    size_t o_lut = up(o_cls + ncls * sizeof(ClassDesc));
    size_t o_err = up(o_lut + lut16.size() * 4);
    size_t o_img = up(o_err + 256);
    size_t o_gol = up(o_img + image.size());
    size_t o_p12 = up(o_gol + 4096 * 4);
    size_t o_sig = up(o_p12 + 4096 * 2);
    size_t o_hk = up(o_sig + sizeof sigs);
    size_t o_hc = up(o_hk + hkeys.size() * 8);
    size_t o_srk = up(o_hc + hcls.size() * 4);
    // order of the classes in the sorted GEMV layout: decoder form, then unranking steps (most first), then class
    std::vector<uint16_t> sort_rank;
    if (ctx->fast && ncls <= 1023) {
        std::vector<uint32_t> order(ncls);
        auto form_key = [&](uint32_t j) {
            const ClassDesc& d = h.desc[j];
            const uint32_t kind = d.parity ? 0u : ((d.w == 8 || d.w == 12 || d.w == 16) ? 1u : 2u);
            return kind * 16u + (15u - (uint32_t)(d.nlev1 + d.nlev0));
        };
        for (uint32_t j = 0; j < ncls; ++j) order[j] = j;
        std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return form_key(a) < form_key(b); });
        sort_rank.resize(ncls);
        for (uint32_t r = 0; r < ncls; ++r) sort_rank[order[r]] = (uint16_t)r;
    }
    size_t o_cnt = up(o_srk + sort_rank.size() * 2);
    size_t o_scr = up(o_cnt + (size_t)(kCounterWords + 16) * 4 + 256);   // ... and the peers' description of a row-sharded GEMM   // one counter per group of 8 rows (GEMV) / per 128-row tile (GEMM), then the grid arrival counter
    static_assert(kPairSlotOffset == 64ll * kMaxScratchRows, "the pair slots start where the scratch rows end");
    size_t total = o_scr + (size_t)64 * kMaxScratchRows * (4 + 8);       // binary32 scratch rows, then one 64-bit pair slot per GEMV row
    std::vector<uint8_t> blob(o_cnt, 0);
    std::memcpy(blob.data() + o_offhi, off_hi.data(), (ncls + 1) * 4);
    std::memcpy(blob.data() + o_offlo, off_lo.data(), (ncls + 1) * 8);
    std::memcpy(blob.data() + o_cls, h.desc.data(), ncls * sizeof(ClassDesc));
    std::memcpy(blob.data() + o_lut, lut16.data(), lut16.size() * 4);
    std::memcpy(blob.data() + o_img, image.data(), image.size());
    std::memcpy(blob.data() + o_gol, h.golay.data(), 4096 * 4);
    std::memcpy(blob.data() + o_p12, pos12.data(), 4096 * 2);
    std::memcpy(blob.data() + o_sig, sigs, sizeof sigs);
    if (!hkeys.empty()) {
        std::memcpy(blob.data() + o_hk, hkeys.data(), hkeys.size() * 8);
        std::memcpy(blob.data() + o_hc, hcls.data(), hcls.size() * 4);
    }
    if (!sort_rank.empty()) std::memcpy(blob.data() + o_srk, sort_rank.data(), sort_rank.size() * 2);
    if (cudaMalloc(&ctx->d_blob, total) != cudaSuccess) { delete ctx; return LLVQ_ECUDA; }
    if (cudaMemcpy(ctx->d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(static_cast<uint8_t*>(ctx->d_blob) + o_cnt, 0, total - o_cnt) != cudaSuccess) {
        cudaFree(ctx->d_blob); delete ctx; return LLVQ_ECUDA;
    }
    uint8_t* d = static_cast<uint8_t*>(ctx->d_blob);
    ctx->dev.off_hi = reinterpret_cast<const uint32_t*>(d + o_offhi);
    ctx->dev.off_lo = reinterpret_cast<const uint64_t*>(d + o_offlo);
    ctx->dev.cls = reinterpret_cast<const ClassDesc*>(d + o_cls);
    ctx->dev.lut16 = reinterpret_cast<const uint32_t*>(d + o_lut);
    ctx->d_err = reinterpret_cast<unsigned long long*>(d + o_err);
    ctx->dev.bad_index = ctx->d_err;
    ctx->dev.flags = reinterpret_cast<uint32_t*>(d + o_err + 8);
    ctx->dev.n_lo = (uint64_t)h.N; ctx->dev.n_hi = (uint64_t)(h.N >> 64);
    ctx->dev.nclasses = (int)ncls;
    ctx->dev.W = h.W;
    ctx->d_image = d + o_img;
    ctx->d_golay = reinterpret_cast<const uint32_t*>(d + o_gol);
    ctx->d_sort_rank = sort_rank.empty() ? nullptr : reinterpret_cast<const uint16_t*>(d + o_srk);
    ctx->enc.pos_by_low12 = reinterpret_cast<const uint16_t*>(d + o_p12);
    ctx->enc.sig_of_value = reinterpret_cast<const uint64_t*>(d + o_sig);
    ctx->enc.hash_key = reinterpret_cast<const uint64_t*>(d + o_hk);
    ctx->enc.hash_cls = reinterpret_cast<const uint32_t*>(d + o_hc);
    ctx->enc.hash_mask = hkeys.empty() ? 0u : (uint32_t)(hkeys.size() - 1);
    ctx->d_counters = reinterpret_cast<uint32_t*>(d + o_cnt);
    ctx->d_scratch = reinterpret_cast<float*>(d + o_scr);
    ctx->d_shard = d + o_cnt + (size_t)(kCounterWords + 16) * 4;
    static_assert(sizeof(YOut) <= 256, "the space reserved behind the counters");
    *out = ctx;
    return LLVQ_OK;
}

void llvq_destroy(llvq_ctx* ctx)
{
    if (!ctx) return;
    if (ctx->d_blob) {
        DeviceGuard guard(ctx->device);
        cudaFree(ctx->d_blob);
    }
    delete ctx;
}

int llvq_index_bits(const llvq_ctx* ctx) { return ctx ? ctx->host.W : -1; }

int llvq_num_points(const llvq_ctx* ctx, uint64_t lo_hi[2])
{
    if (!ctx || !lo_hi) return LLVQ_EINVAL;
    lo_hi[0] = (uint64_t)ctx->host.N; lo_hi[1] = (uint64_t)(ctx->host.N >> 64);
    return LLVQ_OK;
}

int llvq_num_classes(const llvq_ctx* ctx) { return ctx ? (int)ctx->host.desc.size() : -1; }

size_t llvq_index_bytes(const llvq_ctx* ctx, uint64_t nblocks)
{
    if (!ctx) return 0;
    unsigned __int128 bits = (unsigned __int128)nblocks * (unsigned)ctx->host.W;
    unsigned __int128 bytes = (bits + 7) / 8;
    return (size_t)((bytes + 15) / 16 * 16);
}

// Host-only: description of class j (for tests of the table generator).
// info = {m, parity, w, B, nvalues}; values/mults hold up to 24 entries.
int llvq_class_info(const llvq_ctx* ctx, int j, int info[5], uint64_t* A, uint64_t card[2], uint64_t offset[2],
                    int values[24], int mults[24])
{
    if (!ctx || j < 0 || j >= (int)ctx->host.info.size() || !info || !A || !card || !offset || !values || !mults) return LLVQ_EINVAL;
    const ClassInfo& c = ctx->host.info[j];
    info[0] = c.m; info[1] = c.parity; info[2] = c.w; info[3] = c.B; info[4] = (int)c.values.size();
    *A = c.A;
    card[0] = (uint64_t)c.card; card[1] = (uint64_t)(c.card >> 64);
    offset[0] = (uint64_t)c.offset; offset[1] = (uint64_t)(c.offset >> 64);
    for (size_t i = 0; i < c.values.size(); ++i) { values[i] = c.values[i]; mults[i] = c.mults[i]; }
    return LLVQ_OK;
}

// Host-only: copy of the sorted Golay table (4096 words).
int llvq_golay_table(const llvq_ctx* ctx, uint32_t out[4096])
{
    if (!ctx || !out) return LLVQ_EINVAL;
    std::memcpy(out, ctx->host.golay.data(), 4096 * 4);
    return LLVQ_OK;
}

int llvq_decode_blocks(const llvq_ctx* ctx, const void* d_idx, uint64_t nblocks, int8_t* d_points, void* stream)
{
    if (ctx && ctx->device >= 0 && nblocks == 0) return LLVQ_OK;      // nothing to do: pointers may be null
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_points) return LLVQ_EINVAL;
    if (!aligned(d_points, 8)) return LLVQ_EALIGN;
    if (nblocks > (1ull << 40)) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    if (ctx->fast) {
        if (!set_smem(decode_blocks_fast_kernel<false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(decode_blocks_fast_kernel<false>, g, (unsigned)kFastThreads, smem, (cudaStream_t)stream, fast_args(ctx), idx, nblocks,
                       reinterpret_cast<uint2*>(d_points)) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(decode_blocks_fast_kernel<true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(decode_blocks_fast_kernel<true>, g, (unsigned)kFastThreads, smem, (cudaStream_t)stream, fast_args(ctx), idx, nblocks,
                       reinterpret_cast<uint2*>(d_points)) != cudaSuccess) return LLVQ_ECUDA;
    }
    return launch_status();
}

int llvq_dequant_matrix(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16,
                        int64_t rows, int64_t cols, int layout, uint16_t* d_w_bf16, int64_t ld, void* stream)
{
    if (ctx && ctx->device >= 0 && (rows == 0 || cols == 0)) return LLVQ_OK;      // nothing to do: pointers may be null
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_gain_f16 || !d_w_bf16 || rows < 0 || cols < 0 || ld < cols) return LLVQ_EINVAL;
    if (layout != LLVQ_LAYOUT_FLAT && layout != LLVQ_LAYOUT_ROWWISE) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2) || !aligned(d_w_bf16, 2)) return LLVQ_EALIGN;
    if (rows == 0 || cols == 0) return LLVQ_OK;
    if (rows > (1ll << 31) || cols > (1ll << 31)) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (layout == LLVQ_LAYOUT_FLAT && ld != cols) return LLVQ_EINVAL;
    const int64_t bpr = layout == LLVQ_LAYOUT_FLAT ? 0 : (cols + 23) / 24;
    const uint64_t nblocks = layout == LLVQ_LAYOUT_FLAT ? ((uint64_t)rows * (uint64_t)cols + 23) / 24 : (uint64_t)rows * (uint64_t)bpr;
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(d_w_bf16);
    if (ctx->fast) {
        if (!set_smem(dequant_fast_kernel<false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(dequant_fast_kernel<false, false>, g, (unsigned)kFastThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, (uint64_t)nblocks,
                       rows, cols, bpr, w, ld) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(dequant_fast_kernel<true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(dequant_fast_kernel<true, false>, g, (unsigned)kFastThreads, smem, st, fast_args(ctx), idx, d_gain_f16, SgArgs{}, (uint64_t)nblocks,
                       rows, cols, bpr, w, ld) != cudaSuccess) return LLVQ_ECUDA;
    }
    return launch_status();
}

// Checks the destinations of a GEMV: every pointer present and aligned for the output type.
static int check_yout(const YOut& yo, int y_dtype)
{
    if (y_dtype != LLVQ_F32 && y_dtype != LLVQ_BF16) return LLVQ_EINVAL;
    if (!yo.y || yo.n_peer < 0 || yo.n_peer > kMaxShardPeers) return LLVQ_EINVAL;
    const size_t a = y_dtype == LLVQ_F32 ? 4 : 2;
    if (!aligned(yo.y, a)) return LLVQ_EALIGN;
    for (int p = 0; p < yo.n_peer; ++p) {
        if (!yo.peer[p]) return LLVQ_EINVAL;
        if (!aligned(yo.peer[p], a)) return LLVQ_EALIGN;
    }
    return LLVQ_OK;
}

static YOut single_y(void* d_y)
{
    YOut yo{};
    yo.y = d_y;
    return yo;
}

// Shared by llvq_gemv, llvq_gemv_sg and llvq_gemv_rowshard: exactly one of d_gain_f16 / sg is used.
static int gemv_common(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, const SgArgs* sg, int64_t n_out, int64_t k_in,
                       const uint16_t* d_x_bf16, const YOut& yo, int y_dtype, void* stream)
{
    if (!d_x_bf16 || n_out < 0 || k_in < 0) return LLVQ_EINVAL;
    if (int e = check_yout(yo, y_dtype)) return e;
    if (!aligned(d_x_bf16, 2)) return LLVQ_EALIGN;
    if (n_out == 0) return LLVQ_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (k_in == 0) {
        const size_t bytes = (size_t)n_out * (y_dtype == LLVQ_F32 ? 4 : 2);
        if (cudaMemsetAsync(yo.y, 0, bytes, st) != cudaSuccess) return LLVQ_ECUDA;
        for (int p = 0; p < yo.n_peer; ++p)
            if (cudaMemsetAsync(yo.peer[p], 0, bytes, st) != cudaSuccess) return LLVQ_ECUDA;
        return LLVQ_OK;
    }
    const int64_t bpr = (k_in + 23) / 24;
    const int64_t nq = (bpr + 3) / 4;
    const size_t smem = ctx->fl.total + 16 + (size_t)nq * 48 * 4 + kGemvGroupsPerPass * kGemvGroupRows * 4 + 16;
    if (smem > 227 * 1024 || n_out > 64ll * kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    const int64_t units = ((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
    const unsigned g = (unsigned)std::min<int64_t>(units, ctx->sm_count);
    // warps per CTA: the count in [28, 32] that wastes the fewest warp slots on the units of one CTA
    const int64_t upc = (units + g - 1) / g;
    int warps = 32; double best_eff = 0.0;
    for (int w = 32; w >= 28; --w) {
        const double eff = (double)upc / (double)(((upc + w - 1) / w) * w);
        if (eff > best_eff + 1e-9) { best_eff = eff; warps = w; }
    }
    const unsigned threads = 32u * (unsigned)warps;
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    const FastArgs fa = fast_args(ctx);
    const SgArgs sga = sg ? *sg : SgArgs{};
    const bool shard = yo.n_peer > 0 || yo.n_flag > 0;                  // row-sharded launch: stored-gain form only
    if (shard && sg) return LLVQ_EUNSUPPORTED;
    // fast-path codes with many classes (mixed warps are what costs there): the kernel that bins the blocks of a segment by
    // class before unranking them; codes with a handful of classes keep the direct kernel
    int seg_units = kBinSegUnits;
    auto bin_bytes = [&](int su) {
        return ctx->fl.total + 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16 + 2 * 1024 * 4 + (size_t)su * 32 * (8 + 2);
    };
    // (smaller segments sort too few blocks to pay for the sort: the direct kernel takes over when 8192 do not fit)
    const size_t smem_bin = bin_bytes(seg_units);
    if ((!sg || sg->bits <= 5) && ctx->fast && ctx->d_sort_rank && ctx->host.desc.size() >= 64 && ctx->host.W <= 48 && smem_bin <= 227 * 1024 &&
        nq < (1ll << 24)) {
        const uint32_t magic = nq == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)nq);
#define LLVQ_LAUNCH_BIN(BF16, SG, SH)                                                                                      \
    do {                                                                                                                   \
        if (!set_smem(gemv_bin_kernel<BF16, SG, SH>, smem_bin)) return LLVQ_ECUDA;                                          \
        if (launch_pdl(gemv_bin_kernel<BF16, SG, SH>, g, (unsigned)kSortThreads, smem_bin, st, fa, idx, ctx->d_sort_rank, d_gain_f16, sga, n_out, k_in, \
                       bpr, magic, seg_units, d_x_bf16, yo, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA; \
    } while (0)
        if (shard)   { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_BIN(true, false, true); else LLVQ_LAUNCH_BIN(false, false, true); }
        else if (sg) { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_BIN(true, true, false); else LLVQ_LAUNCH_BIN(false, true, false); }
        else         { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_BIN(true, false, false); else LLVQ_LAUNCH_BIN(false, false, false); }
#undef LLVQ_LAUNCH_BIN
        return launch_status();
    }
#define LLVQ_LAUNCH_GEMV(BIG, BF16, SG, SH)                                                                        \
    do {                                                                                                           \
        if (!set_smem(gemv_fast_kernel<BIG, BF16, SG, SH>, smem)) return LLVQ_ECUDA;                               \
        if (launch_pdl(gemv_fast_kernel<BIG, BF16, SG, SH>, g, threads, smem, st, fa, idx, d_gain_f16, sga, n_out, k_in, bpr, d_x_bf16, yo, \
                       ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;                         \
    } while (0)
    if (shard && ctx->fast) { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_GEMV(false, true, false, true); else LLVQ_LAUNCH_GEMV(false, false, false, true); }
    else if (shard)         { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_GEMV(true, true, false, true);  else LLVQ_LAUNCH_GEMV(true, false, false, true); }
    else if (sg)            { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_GEMV(false, true, true, false);  else LLVQ_LAUNCH_GEMV(false, false, true, false); }
    else if (ctx->fast)     { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_GEMV(false, true, false, false); else LLVQ_LAUNCH_GEMV(false, false, false, false); }
    else                    { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_GEMV(true, true, false, false);  else LLVQ_LAUNCH_GEMV(true, false, false, false); }
#undef LLVQ_LAUNCH_GEMV
    return launch_status();
}

int llvq_gemv(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
              const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;                     // nothing to do: pointers may be null
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_gain_f16) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2)) return LLVQ_EALIGN;
    return gemv_common(ctx, d_idx, d_gain_f16, nullptr, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

// Argument checks of the shape-gain entry points.
static int check_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook, const float* d_row_scale)
{
    if (int e = check_common(ctx, d_fields)) return e;
    if (gain_bits < 0 || gain_bits > 8 || !d_codebook) return LLVQ_EINVAL;
    if (!aligned(d_codebook, 4) || !aligned(d_row_scale, 4)) return LLVQ_EALIGN;
    if (!ctx->fast || ctx->host.W + gain_bits > 64 || ctx->host.W > 63) return LLVQ_EUNSUPPORTED;
    return LLVQ_OK;
}

size_t llvq_field_bytes(const llvq_ctx* ctx, uint64_t nblocks, int gain_bits)
{
    if (!ctx || gain_bits < 0 || gain_bits > 8) return 0;
    unsigned __int128 bits = (unsigned __int128)nblocks * (unsigned)(ctx->host.W + gain_bits);
    return (size_t)(((bits + 7) / 8 + 15) / 16 * 16);
}

int llvq_dequant_matrix_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32,
                           const float* d_row_scale_f32, int64_t rows, int64_t cols, uint16_t* d_w_bf16, int64_t ld, void* stream)
{
    if (ctx && ctx->device >= 0 && (rows == 0 || cols == 0)) return LLVQ_OK;      // nothing to do: pointers may be null
    if (int e = check_sg(ctx, d_fields, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    if (!d_w_bf16 || rows < 0 || cols < 0 || ld < cols) return LLVQ_EINVAL;
    if (!aligned(d_w_bf16, 2)) return LLVQ_EALIGN;
    if (rows > (1ll << 31) || cols > (1ll << 31)) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const int64_t bpr = (cols + 23) / 24;
    const uint64_t nblocks = (uint64_t)rows * (uint64_t)bpr;
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    if (!set_smem(dequant_fast_kernel<false, true>, smem)) return LLVQ_ECUDA;
    dequant_fast_kernel<false, true><<<g, kFastThreads, smem, (cudaStream_t)stream>>>(
        fast_args(ctx), static_cast<const uint32_t*>(d_fields), nullptr, SgArgs{d_codebook_f32, d_row_scale_f32, gain_bits},
        nblocks, rows, cols, bpr, reinterpret_cast<__nv_bfloat16*>(d_w_bf16), ld);
    return launch_status();
}

int llvq_gemv_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32, const float* d_row_scale_f32,
                 int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;                     // nothing to do: pointers may be null
    if (int e = check_sg(ctx, d_fields, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    const SgArgs sg{d_codebook_f32, d_row_scale_f32, gain_bits};
    return gemv_common(ctx, d_fields, nullptr, &sg, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

// Sorted layout (see the comment at sort_blocks_kernel).  Available for fast-path codes whose indices fit 48 bits
// with 2^48 - 1 left over as the "no block" marker.
static bool sortable(const llvq_ctx* ctx, int64_t k_in)
{
    if (!ctx->fast || !ctx->d_sort_rank || ctx->host.W > 48 || ctx->host.N >= (u128)kSortIndexMask) return false;
    const int64_t nq = ((k_in + 23) / 24 + 3) / 4;
    const size_t smem = ctx->fl.total + 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16;
    return smem <= 227 * 1024 && nq < (1ll << 24);
}

size_t llvq_sorted_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in)
{
    if (!ctx || ctx->device < 0 || n_out <= 0 || k_in <= 0 || !sortable(ctx, k_in)) return 0;
    const int64_t nq = ((k_in + 23) / 24 + 3) / 4;
    return (size_t)(((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq) * 32 * 8;
}

static int sort_blocks_common(const llvq_ctx* ctx, const void* d_fields, int gain_bits, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    if (int e = check_common(ctx, d_fields)) return e;
    if (!d_sorted || n_out <= 0 || k_in <= 0 || gain_bits < 0 || gain_bits > 8) return LLVQ_EINVAL;
    if (!aligned(d_sorted, 16)) return LLVQ_EALIGN;
    if (!sortable(ctx, k_in) || ctx->host.W + gain_bits > 48 || n_out > 64ll * kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const int64_t bpr = (k_in + 23) / 24, nq = (bpr + 3) / 4;
    const int64_t units = ((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
    const unsigned g = (unsigned)std::min<int64_t>(units, ctx->sm_count);
    const size_t smem = ctx->fl.total + 16;
    if (!set_smem(sort_blocks_kernel, smem)) return LLVQ_ECUDA;
    sort_blocks_kernel<<<g, kSortThreads, smem, (cudaStream_t)stream>>>(fast_args(ctx), static_cast<const uint32_t*>(d_fields), ctx->d_sort_rank, gain_bits,
                                                                       n_out, bpr, static_cast<unsigned long long*>(d_sorted));
    return launch_status();
}

int llvq_sort_blocks(const llvq_ctx* ctx, const void* d_idx, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    return sort_blocks_common(ctx, d_idx, 0, n_out, k_in, d_sorted, stream);
}

int llvq_sort_blocks_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    return sort_blocks_common(ctx, d_fields, gain_bits, n_out, k_in, d_sorted, stream);
}

// Exactly one of d_gain_f16 / sg is used.
static int gemv_sorted_common(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, const SgArgs* sg, int64_t n_out, int64_t k_in,
                              const uint16_t* d_x_bf16, const YOut& yo, int y_dtype, void* stream)
{
    if (!d_x_bf16 || n_out < 0 || k_in <= 0) return LLVQ_EINVAL;
    if (int e = check_yout(yo, y_dtype)) return e;
    if (!aligned(d_x_bf16, 2)) return LLVQ_EALIGN;
    if (!sortable(ctx, k_in) || n_out > 64ll * kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t bpr = (k_in + 23) / 24, nq = (bpr + 3) / 4;
    const int64_t units = ((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
    const unsigned g = (unsigned)std::min<int64_t>(units, ctx->sm_count);
    const size_t smem = ctx->fl.total + 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16;
    const uint32_t magic = nq == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)nq);
    const unsigned long long* sp = static_cast<const unsigned long long*>(d_sorted);
    const SgArgs sga = sg ? *sg : SgArgs{};
#define LLVQ_LAUNCH_SORTED(BF16, SG, SH)                                                                                \
    do {                                                                                                                \
        if (!set_smem(gemv_sorted_kernel<BF16, SG, SH>, smem)) return LLVQ_ECUDA;                                        \
        if (launch_pdl(gemv_sorted_kernel<BF16, SG, SH>, g, (unsigned)kSortThreads, smem, st, fast_args(ctx), sp, d_gain_f16, sga, n_out, k_in, bpr, \
                       magic, d_x_bf16, yo, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;          \
    } while (0)
    const bool shard = yo.n_peer > 0 || yo.n_flag > 0;                  // row-sharded launch: stored-gain form only
    if (shard && sg) return LLVQ_EUNSUPPORTED;
    if (shard)   { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_SORTED(true, false, true); else LLVQ_LAUNCH_SORTED(false, false, true); }
    else if (sg) { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_SORTED(true, true, false); else LLVQ_LAUNCH_SORTED(false, true, false); }
    else         { if (y_dtype == LLVQ_BF16) LLVQ_LAUNCH_SORTED(true, false, false); else LLVQ_LAUNCH_SORTED(false, false, false); }
#undef LLVQ_LAUNCH_SORTED
    return launch_status();
}

int llvq_gemv_sorted(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                     const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;
    if (int e = check_common(ctx, d_sorted)) return e;
    if (!d_gain_f16) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2)) return LLVQ_EALIGN;
    return gemv_sorted_common(ctx, d_sorted, d_gain_f16, nullptr, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

int llvq_gemv_sorted_sg(const llvq_ctx* ctx, const void* d_sorted, int gain_bits, const float* d_codebook_f32, const float* d_row_scale_f32,
                        int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;
    if (int e = check_sg(ctx, d_sorted, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    if (ctx->host.W + gain_bits > 48) return LLVQ_EUNSUPPORTED;
    const SgArgs sg{d_codebook_f32, d_row_scale_f32, gain_bits};
    return gemv_sorted_common(ctx, d_sorted, nullptr, &sg, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

// Row-sharded GEMV: the destinations of one rank's band.  d_y_all[0..n_dest) are the ranks' full-length copies of y
// (own_slot = this rank's own copy), the band starts at row row0; d_flag_words (optional) = for every destination
// the word that receives `epoch` when the band is in place (the own slot's entry is not used).
static int shard_yout(const llvq_ctx* ctx, void* const* d_y_all, int n_dest, int own_slot, int64_t row0, int y_dtype,
                      uint32_t* const* d_flag_words, uint32_t epoch, YOut* yo)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    if (!d_y_all || n_dest < 1 || n_dest > kMaxShardPeers + 1 || own_slot < 0 || own_slot >= n_dest || row0 < 0) return LLVQ_EINVAL;
    if (y_dtype != LLVQ_F32 && y_dtype != LLVQ_BF16) return LLVQ_EINVAL;
    const size_t es = y_dtype == LLVQ_F32 ? 4 : 2;
    *yo = YOut{};
    for (int d = 0; d < n_dest; ++d) {
        if (!d_y_all[d]) return LLVQ_EINVAL;
        if (!aligned(d_y_all[d], es)) return LLVQ_EALIGN;
        void* at = static_cast<unsigned char*>(d_y_all[d]) + (size_t)row0 * es;
        if (d == own_slot) { yo->y = at; continue; }
        yo->peer[yo->n_peer++] = at;
        if (d_flag_words) {
            if (!d_flag_words[d]) return LLVQ_EINVAL;
            if (!aligned(d_flag_words[d], 4)) return LLVQ_EALIGN;
            yo->flag[yo->n_flag++] = d_flag_words[d];
        }
    }
    yo->done = ctx->d_counters + kCounterWords;
    yo->epoch = epoch;
    return LLVQ_OK;
}

// A band without rows still has to tell the peers that it is done with the step.
static int signal_only(const llvq_ctx* ctx, const YOut& yo, void* stream)
{
    if (yo.n_flag == 0) return LLVQ_OK;
    return llvq_signal_ranks(ctx, yo.flag, yo.n_flag, yo.epoch, stream);
}

int llvq_gemv_rowshard(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                       const uint16_t* d_x_bf16, void* const* d_y_all, int n_dest, int own_slot, int64_t row0, int y_dtype,
                       uint32_t* const* d_flag_words, uint32_t epoch, void* stream)
{
    YOut yo;
    if (int e = shard_yout(ctx, d_y_all, n_dest, own_slot, row0, y_dtype, d_flag_words, epoch, &yo)) return e;
    if (n_rows == 0) return signal_only(ctx, yo, stream);
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_gain_f16) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2)) return LLVQ_EALIGN;
    if (k_in == 0) {                                   // y = 0 by copies, no kernel to raise the flags
        if (int e = gemv_common(ctx, d_idx, d_gain_f16, nullptr, n_rows, k_in, d_x_bf16, yo, y_dtype, stream)) return e;
        return signal_only(ctx, yo, stream);
    }
    return gemv_common(ctx, d_idx, d_gain_f16, nullptr, n_rows, k_in, d_x_bf16, yo, y_dtype, stream);
}

int llvq_gemv_sorted_rowshard(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                              const uint16_t* d_x_bf16, void* const* d_y_all, int n_dest, int own_slot, int64_t row0, int y_dtype,
                              uint32_t* const* d_flag_words, uint32_t epoch, void* stream)
{
    YOut yo;
    if (int e = shard_yout(ctx, d_y_all, n_dest, own_slot, row0, y_dtype, d_flag_words, epoch, &yo)) return e;
    if (n_rows == 0) return signal_only(ctx, yo, stream);
    if (int e = check_common(ctx, d_sorted)) return e;
    if (!d_gain_f16) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2)) return LLVQ_EALIGN;
    return gemv_sorted_common(ctx, d_sorted, d_gain_f16, nullptr, n_rows, k_in, d_x_bf16, yo, y_dtype, stream);
}

// Sorted layout of the small-batch GEMM (see the comment at sort_blocks_gemm_kernel).
static bool gemm_sortable(const llvq_ctx* ctx)
{
    if (!ctx->fast) return ctx->host.W <= 72 && ctx->dev.nclasses < (1 << 17);     // 128-bit entries: 72-bit index + class + position
    return ctx->d_sort_rank && ctx->host.W <= 48 && ctx->host.N < (u128)kSortIndexMask;
}

size_t llvq_sorted_gemm_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in)
{
    if (!ctx || ctx->device < 0 || n_out <= 0 || k_in <= 0 || !gemm_sortable(ctx)) return 0;
    const int64_t bpr = (k_in + 23) / 24;
    return (size_t)(((n_out + kGemmRows - 1) / kGemmRows) * ((bpr + kDomBlocks - 1) / kDomBlocks)) * kDomEntries * (ctx->fast ? 8 : 16);
}

static int sort_blocks_gemm_common(const llvq_ctx* ctx, const void* d_idx, int gain_bits, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_sorted || n_out <= 0 || k_in <= 0 || gain_bits < 0 || gain_bits > 8) return LLVQ_EINVAL;
    if (!aligned(d_sorted, 16)) return LLVQ_EALIGN;
    if (!gemm_sortable(ctx) || (gain_bits > 0 && !ctx->fast) || (ctx->fast && ctx->host.W + gain_bits > 48)) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const int64_t bpr = (k_in + 23) / 24;
    const int64_t ndomains = ((n_out + kGemmRows - 1) / kGemmRows) * ((bpr + kDomBlocks - 1) / kDomBlocks);
    const unsigned g = (unsigned)std::min<int64_t>(ndomains, 4ll * ctx->sm_count);
    if (!ctx->fast) {
        sort_blocks_gemm_big_kernel<<<g, kDomEntries, 0, (cudaStream_t)stream>>>(fast_args(ctx), static_cast<const uint32_t*>(d_idx), n_out, bpr,
                                                                                 ndomains, static_cast<ulonglong2*>(d_sorted));
        return launch_status();
    }
    const size_t smem = ctx->fl.total + 16;
    if (!set_smem(sort_blocks_gemm_kernel, smem)) return LLVQ_ECUDA;
    sort_blocks_gemm_kernel<<<g, kDomEntries, smem, (cudaStream_t)stream>>>(fast_args(ctx), static_cast<const uint32_t*>(d_idx), ctx->d_sort_rank,
                                                                           gain_bits, n_out, bpr, ndomains, static_cast<unsigned long long*>(d_sorted));
    return launch_status();
}

int llvq_sort_blocks_gemm(const llvq_ctx* ctx, const void* d_idx, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    return sort_blocks_gemm_common(ctx, d_idx, 0, n_out, k_in, d_sorted, stream);
}

int llvq_sort_blocks_gemm_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, int64_t n_out, int64_t k_in, void* d_sorted, void* stream)
{
    return sort_blocks_gemm_common(ctx, d_fields, gain_bits, n_out, k_in, d_sorted, stream);
}

int llvq_gemm_small_batch_sorted_sg(const llvq_ctx* ctx, const void* d_sorted, int gain_bits, const float* d_codebook_f32,
                                    const float* d_row_scale_f32, int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16, int batch,
                                    uint16_t* d_y_bf16, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;
    if (int e = check_sg(ctx, d_sorted, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    if (!d_x_bf16 || !d_y_bf16 || n_out < 0 || k_in < 0 || batch < 1 || batch > 64) return LLVQ_EINVAL;
    if (!aligned(d_x_bf16, 16) || !aligned(d_y_bf16, 2) || (k_in & 7)) return LLVQ_EALIGN;
    if (!gemm_sortable(ctx) || ctx->host.W + gain_bits > 48 || n_out > kMaxScratchRows || k_in <= 0) return LLVQ_EUNSUPPORTED;
    const SgArgs sg{d_codebook_f32, d_row_scale_f32, gain_bits};
    return launch_gemm_domains(ctx, d_sorted, nullptr, n_out, k_in, d_x_bf16, batch, d_y_bf16, ctx->d_scratch, ctx->d_counters, stream,
                               nullptr, 0, &sg);
}

int llvq_gemm_small_batch_sorted(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                                 const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, void* stream)
{
    if (int e = check_gemm_args(ctx, d_sorted, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16)) return e;
    if (n_out == 0) return LLVQ_OK;
    if (!gemm_sortable(ctx) || n_out > kMaxScratchRows || k_in <= 0) return LLVQ_EUNSUPPORTED;
    return launch_gemm_domains(ctx, d_sorted, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16, ctx->d_scratch, ctx->d_counters, stream);
}

int llvq_gemm_small_batch_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32, const float* d_row_scale_f32,
                             int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0 && batch >= 1 && batch <= 64) return LLVQ_OK;   // nothing to do: pointers may be null
    if (int e = check_sg(ctx, d_fields, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    if (!d_x_bf16 || !d_y_bf16 || n_out < 0 || k_in < 0 || batch < 1 || batch > 64) return LLVQ_EINVAL;
    if (!aligned(d_x_bf16, 16) || !aligned(d_y_bf16, 2) || (k_in & 7)) return LLVQ_EALIGN;
    if (n_out > kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    const SgArgs sg{d_codebook_f32, d_row_scale_f32, gain_bits};
    return launch_gemm(ctx, d_fields, nullptr, n_out, k_in, d_x_bf16, batch, d_y_bf16, ctx->d_scratch, ctx->d_counters, stream, &sg);
}

int llvq_gemm_small_batch(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                          const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, void* stream)
{
    if (int e = check_gemm_args(ctx, d_idx, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16)) return e;
    if (n_out > kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    return launch_gemm(ctx, d_idx, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16, ctx->d_scratch, ctx->d_counters, stream);
}

// Row-sharded small-batch GEMM: the band's columns [row0, row0 + n_rows) of every rank's Y [batch][n_out_total].
static int gemm_rowshard(const llvq_ctx* ctx, const void* d_stream, bool sorted, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                         const uint16_t* d_x_bf16, int batch, void* const* d_y_all, int n_dest, int own_slot, int64_t row0,
                         int64_t n_out_total, uint32_t* const* d_flag_words, uint32_t epoch, void* stream)
{
    YOut yo;
    if (int e = shard_yout(ctx, d_y_all, n_dest, own_slot, row0, LLVQ_BF16, d_flag_words, epoch, &yo)) return e;
    if (n_rows < 0 || n_out_total < row0 + n_rows) return LLVQ_EINVAL;
    if (n_rows == 0) return signal_only(ctx, yo, stream);
    if (int e = check_gemm_args(ctx, d_stream, d_gain_f16, n_rows, k_in, d_x_bf16, batch, static_cast<const uint16_t*>(yo.y))) return e;
    if (n_rows > kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    if (k_in == 0) {                                   // Y = 0 by copies, no kernel to raise the flags
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return LLVQ_ECUDA;
        for (int p = -1; p < yo.n_peer; ++p)
            if (cudaMemset2DAsync(p < 0 ? yo.y : yo.peer[p], (size_t)n_out_total * 2, 0, (size_t)n_rows * 2, (size_t)batch,
                                  (cudaStream_t)stream) != cudaSuccess) return LLVQ_ECUDA;
        return signal_only(ctx, yo, stream);
    }
    if (sorted) {
        if (!gemm_sortable(ctx)) return LLVQ_EUNSUPPORTED;
        return launch_gemm_domains(ctx, d_stream, d_gain_f16, n_rows, k_in, d_x_bf16, batch, nullptr, ctx->d_scratch, ctx->d_counters, stream,
                                   &yo, n_out_total);
    }
    return launch_gemm(ctx, d_stream, d_gain_f16, n_rows, k_in, d_x_bf16, batch, nullptr, ctx->d_scratch, ctx->d_counters, stream, nullptr,
                       &yo, n_out_total);
}

int llvq_gemm_small_batch_rowshard(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                                   const uint16_t* d_x_bf16, int batch, void* const* d_y_all, int n_dest, int own_slot, int64_t row0,
                                   int64_t n_out_total, uint32_t* const* d_flag_words, uint32_t epoch, void* stream)
{
    return gemm_rowshard(ctx, d_idx, false, d_gain_f16, n_rows, k_in, d_x_bf16, batch, d_y_all, n_dest, own_slot, row0, n_out_total,
                         d_flag_words, epoch, stream);
}

int llvq_gemm_small_batch_sorted_rowshard(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                                          const uint16_t* d_x_bf16, int batch, void* const* d_y_all, int n_dest, int own_slot, int64_t row0,
                                          int64_t n_out_total, uint32_t* const* d_flag_words, uint32_t epoch, void* stream)
{
    return gemm_rowshard(ctx, d_sorted, true, d_gain_f16, n_rows, k_in, d_x_bf16, batch, d_y_all, n_dest, own_slot, row0, n_out_total,
                         d_flag_words, epoch, stream);
}


// ---------------------------------------------------------------------------
// llvq_gemm_small_batch_noalloc: the small-batch GEMM for callers that must not allocate.
// Its split-K scratch is this fixed array, which every GPU that loads the library carries
// until the process exits.  Layout: [row-tile counters: 512 bytes][binary32 partial sums: 1 MiB].
// ---------------------------------------------------------------------------
constexpr int kNoallocMaxRowTiles = 128;                          // 128 tiles x 128 rows = 16384 output rows
constexpr size_t kNoallocCounterBytes = kNoallocMaxRowTiles * sizeof(uint32_t);
constexpr size_t kNoallocScratchFloats = 262144;                  // padded batch x padded rows must fit: 1 MiB
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocCounterBytes + kNoallocScratchFloats * sizeof(float)];

int llvq_gemm_small_batch_noalloc(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                                  const uint16_t* d_x_bf16, int batch, uint16_t* d_y_bf16, void* stream)
{
    if (int e = check_gemm_args(ctx, d_idx, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16)) return e;
    const int64_t row_tiles = (n_out + kGemmRows - 1) / kGemmRows;
    const int64_t npad = (batch + 15) / 16 * 16;
    if (row_tiles > kNoallocMaxRowTiles || npad * row_tiles * kGemmRows > (int64_t)kNoallocScratchFloats) return LLVQ_EUNSUPPORTED;
    if (n_out == 0) return LLVQ_OK;
    if (ctx->device >= 64) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    // The array's name is only a host-side handle: ask the runtime, once per device and with that device
    // current, for the address the kernels can use.
    static std::mutex lock;
    static unsigned char* device_ptr[64] = {nullptr};
    unsigned char* base;
    {
        std::lock_guard<std::mutex> hold(lock);
        if (!device_ptr[ctx->device]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return LLVQ_ECUDA;
            device_ptr[ctx->device] = static_cast<unsigned char*>(p);
        }
        base = device_ptr[ctx->device];
    }
    // The array keeps whatever the previous call (or an aborted one) left: clear the part this call uses.
    const size_t used = kNoallocCounterBytes + (size_t)(npad * row_tiles * kGemmRows) * sizeof(float);
    if (cudaMemsetAsync(base, 0, used, (cudaStream_t)stream) != cudaSuccess) return LLVQ_ECUDA;
    return launch_gemm(ctx, d_idx, d_gain_f16, n_out, k_in, d_x_bf16, batch, d_y_bf16,
                       reinterpret_cast<float*>(base + kNoallocCounterBytes), reinterpret_cast<uint32_t*>(base), stream);
}

// Waits, with a small iteration limit, on an mbarrier that nothing ever arrives at, then records the expiry the
// same way the real kernels do.  Exercises the "bounded wait -> error flag -> normal return" path without any fault.
__global__ void selftest_wait_kernel(uint32_t* flags)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const uint32_t a = smem_u32(&bar);
    uint32_t done = 0;
    for (uint32_t it = 0; it < 64u && !done; ++it) {
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(a), "r"(0u) : "memory");
    }
    if (!done && threadIdx.x == 0) atomicOr(flags, (uint32_t)LLVQ_FLAG_WAIT_TIMEOUT);
}

int llvq_selftest_wait_timeout(llvq_ctx* ctx, void* stream)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->dev.flags);
    return launch_status();
}

int llvq_last_error(llvq_ctx* ctx, void* stream, uint64_t* n_bad_index, uint32_t* flags)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long host[2] = {0, 0};
    if (cudaMemcpyAsync(host, ctx->d_err, 16, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaMemsetAsync(ctx->d_err, 0, 16, st) != cudaSuccess) return LLVQ_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LLVQ_ECUDA;
    if (n_bad_index) *n_bad_index = host[0];
    if (flags) *flags = (uint32_t)host[1];
    return LLVQ_OK;
}

}  // extern "C"
