// The fused dequant + GEMV kernels: the direct kernel (tensor-core reduction), the sorted layout (sort kernel and
// consumer) and the kernel that bins a segment's blocks by class itself.  Included by gemv.cu and gemm.cu inside their
// unnamed namespaces, after kernels_common.cuh.
#pragma once

// Fused dequant + GEMV.  The work is cut into units of 8 rows x 4 column blocks, numbered row group major, and
// every CTA takes an equal contiguous range of units.  In a unit lane (g, t) = (lane / 4, lane % 4) decodes the
// block (row g, column block 4q + t); its 12 packed bf16 pairs are the A fragments (rows 0..7; rows 8..15 are
// zero) of six m16n8k16 tensor-core MMAs whose B fragment carries the matching 4 x 24 activations (the same in
// all 8 columns), accumulating in binary32.  Row sums are collected in shared memory; a row group that is
// split between CTAs is finished through a zero-kept global scratch and an arrival counter.

__device__ __forceinline__ void mma_bf16_16816(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// CTA that owns unit u when G CTAs split U units into ranges [c*U/G, (c+1)*U/G).
__device__ __forceinline__ int64_t unit_owner(int64_t u, int64_t U, int64_t G) { return ((u + 1) * G - 1) / U; }

template <bool kOutBf16, bool kShard>
__device__ __forceinline__ void store_y(const YOut& yo, int64_t row, float v)
{
    if (kOutBf16) {
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        reinterpret_cast<__nv_bfloat16*>(yo.y)[row] = h;
        if (kShard) {                                     // the single-GPU instantiations carry none of this
#pragma unroll
            for (int p = 0; p < kMaxShardPeers; ++p)      // static indices: the struct stays in the parameter bank
                if (p < yo.n_peer) reinterpret_cast<__nv_bfloat16*>(yo.peer[p])[row] = h;
        }
    } else {
        reinterpret_cast<float*>(yo.y)[row] = v;
        if (kShard) {
#pragma unroll
            for (int p = 0; p < kMaxShardPeers; ++p)
                if (p < yo.n_peer) reinterpret_cast<float*>(yo.peer[p])[row] = v;
        }
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
// slot0 (a multiple of 8) = first scratch row / pair slot of this matrix when one launch works on several matrices.
template <bool kOutBf16, bool kShard, typename RowSum>
__device__ __forceinline__ void finish_pass(const YOut& yo, int64_t rg0, int64_t rg1, int64_t nq, int64_t u_begin, int64_t u_end,
                                            int64_t U, int64_t G, int64_t n_out, float* __restrict__ scratch,
                                            uint32_t* __restrict__ counters, RowSum row_sum, int64_t slot0 = 0, int warp_of = -1, int nwarps_of = 0)
{
    // by default the warps of the CTA share the row groups; warp_of / nwarps_of let a subset of the warps (one warp) do it
    const int warp = warp_of >= 0 ? warp_of : (int)(threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int nwarps = warp_of >= 0 ? nwarps_of : (int)(blockDim.x >> 5);
    for (int64_t rg = rg0 + warp; rg <= rg1; rg += nwarps) {
        const bool whole = u_begin <= rg * nq && (rg + 1) * nq <= u_end;
        const int64_t row = rg * kGemvGroupRows + lane;
        const bool mine = lane < kGemvGroupRows && row < n_out;
        const float part = lane < kGemvGroupRows ? row_sum((rg - rg0) * kGemvGroupRows + lane) : 0.f;
        if (whole) {
            if (mine) {
                store_y<kOutBf16, kShard>(yo, row, part);
            }
            continue;
        }
        const uint32_t parts = (uint32_t)(unit_owner((rg + 1) * nq - 1, U, G) - unit_owner(rg * nq, U, G) + 1);
        if (parts == 2u) {
            // two CTAs share the group (the usual case): one compare-and-swap on a 64-bit slot carries both the sum
            // and the arrival.  Whoever finds the slot empty leaves (its sum, 1) there; the other gets that back from
            // its failed swap, adds its own sum, stores y and empties the slot.  One round trip each, no fence.
            if (mine) {
                unsigned long long* slot = reinterpret_cast<unsigned long long*>(scratch + kPairSlotOffset) + slot0 + row;
                const unsigned long long seen = atomicCAS(slot, 0ull, (unsigned long long)__float_as_uint(part) | 1ull << 32);
                if (seen != 0ull) {
                    store_y<kOutBf16, kShard>(yo, row, __fadd_rn(__uint_as_float((uint32_t)seen), part));
                    __stcg(slot, 0ull);
                }
            }
            continue;
        }
        if (mine) atomicAdd(scratch + slot0 + row, part);
        __threadfence();                               // every lane's add is performed before ...
        __syncwarp();
        uint32_t is_last = 0u;
        if (lane == 0) {
            __threadfence();                           // ... lane 0 counts the arrival
            is_last = atomicAdd(counters + slot0 / kGemvGroupRows + rg, 1u) == parts - 1u;
        }
        is_last = __shfl_sync(kFullMask, is_last, 0);
        if (is_last) {
            __threadfence();
            if (mine) {
                store_y<kOutBf16, kShard>(yo, row, __ldcg(scratch + slot0 + row));
                __stcg(scratch + slot0 + row, 0.f);
            }
            if (lane == 0) counters[slot0 / kGemvGroupRows + rg] = 0u;
        }
    }
}

// Last step of a row-sharded GEMV CTA (all threads call it, after their last store to y): counts the CTA in; the CTA
// that completes the grid raises the epoch in every peer's flag word.  The remote stores of y are plain stores; the block
// barrier below orders them before the system-scope fence of the thread that counts the CTA in, which makes them visible,
// cumulatively, before the flag (the usual barrier + fence + flag pattern: no fence per storing lane).
__device__ __forceinline__ void shard_arrive(const YOut& yo)
{
    if (yo.n_flag == 0) return;
    __syncthreads();
    if (threadIdx.x != 0) return;
    __threadfence_system();
    if (atomicAdd(yo.done, 1u) != gridDim.x - 1u) return;
    atomicExch(yo.done, 0u);
    // one system-scope fence releases everything before it for all the flag words: the stores themselves are relaxed (a
    // release store per word would pay the fence once per peer: measured 2 us each)
    __threadfence_system();
#pragma unroll
    for (int p = 0; p < kMaxShardPeers; ++p)
        if (p < yo.n_flag) asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(yo.flag[p]), "r"(yo.epoch) : "memory");
}

// sum_j w_j x_j over 12 packed bf16 pairs with binary32 accumulation: fma.rn.f32.bf16 takes the bf16 halves as they are
// (products of two bf16 values are exact in binary32, so this is the chain of 24 binary32 FMAs without the unpacking).
__device__ __forceinline__ float dot24_bf16(const uint32_t w[12], const uint32_t x[12])
{
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int j = 0; j < 12; ++j) {
        asm("{\n .reg .b16 wl, wh, xl, xh;\n mov.b32 {wl, wh}, %2;\n mov.b32 {xl, xh}, %3;\n"
            " fma.rn.f32.bf16 %0, wl, xl, %0;\n fma.rn.f32.bf16 %1, wh, xh, %1;\n}"
            : "+f"(s0), "+f"(s1) : "r"(w[j]), "r"(x[j]));
    }
    return s0 + s1;
}

template <bool kBig, bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_fast_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ gain, SgArgs sg,
                 int64_t n_out, int64_t k_in, int64_t bpr, const uint16_t* __restrict__ x, YOut yo,
                 float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    FAST_PROLOGUE(if (kShard) shard_arrive(yo));
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
    const uint32_t kind = !valid ? kKindNull : (T.desc[cls * kFastDescStride] >> 22) & 3u;     // the form is part of the descriptor's flags
    r.p0 = r.p1 = r.p2 = r.neg = r.vals_lo = r.vals_hi = 0u;
    // every form writes r only for its own lanes
    if (__any_sync(kFullMask, kind == kKindOdd)) {
        const bool mine = kind == kKindOdd;
        fast_decode_local<1>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, r);
    }
    if (__any_sync(kFullMask, kind == kKindEven)) {
        const bool mine = kind == kKindEven;
        fast_decode_local<0>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, r);
    }
    if (__any_sync(kFullMask, kind == kKindOther)) {
        const bool mine = kind == kKindOther;
        fast_decode_local<-1>(T, mine ? cls : 0u, mine ? local : 0ull, mine, kFullMask, r);
    }
}

__device__ __forceinline__ uint32_t decode_sorted_entry(const FastArgs& fa, const FastSmem& T, uint64_t I, bool valid, Decoded& r)
{
    uint64_t local = 0;
    const uint32_t cls = valid ? fast_find_class(T, I, local) : 0u;
    decode_known_class(T, cls, local, valid, r);
    return cls;
}

// One matrix of a launch that works through several matrices one after another (llvq_gemv_multi, llvq_gemv_sorted_multi):
// every CTA takes its share of each matrix in turn, so the table image, the launch and the ramp-up are paid once.
constexpr int kMaxMultiMats = 8;
struct GemvMat {
    const void* weights;        // stored stream or sorted entries
    const uint16_t* gain;
    const uint16_t* x;
    void* y;
    int64_t n_out, k_in;
    int64_t slot0;              // first scratch row / pair slot of this matrix (a multiple of 8)
    uint32_t nq_magic;          // floor(2^32 / units per row group)
    int32_t seg_units;          // stored stream only: units per binned segment
};
struct GemvMulti {
    GemvMat m[kMaxMultiMats];
    int n;
};

// Ask for the first chunk of every warp of this CTA in L2 (one request per 128-byte line).
__device__ __forceinline__ void prefetch_first_chunks(const unsigned long long* sorted, int64_t n_out, int64_t bpr)
{
    const int64_t nq0 = (bpr + 3) / 4, U0 = ((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq0;
    const int64_t ub = blockIdx.x * U0 / gridDim.x, ue = (blockIdx.x + 1) * U0 / gridDim.x;
    if ((threadIdx.x & 15u) == 0u && ub + (int64_t)(threadIdx.x >> 5) < ue)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(sorted + ub * 32 + threadIdx.x));
}

// The sorted-layout GEMV of one matrix by this CTA (all threads call it; shared memory behind `staging` is reused by the
// next call, which the caller separates with a block barrier).
template <bool kOutBf16, bool kSg, bool kShard>
__device__ __forceinline__ void gemv_sorted_body(const FastArgs& fa, const FastSmem& T, uint8_t* staging,
                                                 const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, const SgArgs& sg,
                                                 int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, const uint16_t* __restrict__ x,
                                                 const YOut& yo, float* __restrict__ scratch, uint32_t* __restrict__ counters, int64_t slot0)
{
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
            uint16_t gbits = 0;
            if (!kSg && valid) gbits = ldg_u16_here(gain + ((int64_t)rg0 * kGemvGroupRows + rloc) * bpr + cb);
            Decoded r;
            const uint32_t cls = decode_sorted_entry(fa, T, I, valid, r);
            if (!kSg) gn = gain_to_float(gbits);
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
            const float dot = dot24_bf16(w, xv);
            if (valid) atomicAdd(&acc[(warp & (kSortAccCopies - 1)) * (kGemvGroupsPerPass * kGemvGroupRows) + rloc], dot);
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
        finish_pass<kOutBf16, kShard>(yo, rg0, rg1, nq, ub, ue, U, G, n_out, scratch, counters, row_sum, slot0);
        __syncthreads();                                   // the sums are read above: the next pass may clear them only now
    });
}

template <bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_sorted_kernel(FastArgs fa, const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, SgArgs sg,
                   int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, const uint16_t* __restrict__ x, YOut yo,
                   float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    prefetch_first_chunks(sorted, n_out, bpr);          // while the table image is on its way
    FAST_PROLOGUE(if (kShard) shard_arrive(yo));
    gemv_sorted_body<kOutBf16, kSg, kShard>(fa, T, staging, sorted, gain, sg, n_out, k_in, bpr, nq_magic, x, yo, scratch, counters, 0);
    if (kShard) shard_arrive(yo);
}

// Several independent matrices in one launch (no output of one may be an input of another).
template <bool kOutBf16>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_sorted_multi_kernel(FastArgs fa, const __grid_constant__ GemvMulti mm, float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    prefetch_first_chunks(static_cast<const unsigned long long*>(mm.m[0].weights), mm.m[0].n_out, (mm.m[0].k_in + 23) / 24);
    FAST_PROLOGUE();
    for (int i = 0; i < mm.n; ++i) {
        const GemvMat& M = mm.m[i];
        if (i + 1 < mm.n)
            prefetch_first_chunks(static_cast<const unsigned long long*>(mm.m[i + 1].weights), mm.m[i + 1].n_out, (mm.m[i + 1].k_in + 23) / 24);
        YOut yo{};
        yo.y = M.y;
        gemv_sorted_body<kOutBf16, false, false>(fa, T, staging, static_cast<const unsigned long long*>(M.weights), M.gain, SgArgs{}, M.n_out, M.k_in,
                                                 (M.k_in + 23) / 24, M.nq_magic, M.x, yo, scratch, counters, M.slot0);
        __syncthreads();                                   // the next matrix restages x and clears the row sums
    }
}

// The same, without a block barrier between the matrices: a warp that finds no chunk of matrix i left goes on to matrix
// i + 1 while the others finish theirs, so the partly filled last round of chunks, the end of the pass and the staging of
// x of one matrix run under the next matrix's work.  Three sets of (x, row sums, chunk counter) rotate: the warp that
// completes matrix i (the last to run out of its chunks) ends the pass alone and then prepares set i % 3 for matrix
// i + 3.  Taken when every CTA's share of every matrix is one segment and one pass (checked on the host).
constexpr int kOverlapSets = 3;
constexpr uint32_t kOverlapSpins = 1u << 22;         // polls of a shared-memory flag before a warp gives up (never in a correct run)

struct OverlapSet {
    uint32_t next_chunk;
    uint32_t arrived;                                // warps that have run out of chunks of the set's matrix
    uint32_t ready;                                  // index + 1 of the matrix the set is prepared for
    uint32_t pad;
};

template <bool kOutBf16>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_sorted_overlap_kernel(FastArgs fa, const __grid_constant__ GemvMulti mm, int xs_words, int acc_rows, float* __restrict__ scratch,
                           uint32_t* __restrict__ counters)
{
    prefetch_first_chunks(static_cast<const unsigned long long*>(mm.m[0].weights), mm.m[0].n_out, (mm.m[0].k_in + 23) / 24);
    FAST_PROLOGUE();
    // [kOverlapSets] x { x as packed pairs [xs_words] | row sums [kSortAccCopies][acc_rows] } | control words
    const int set_words = xs_words + kSortAccCopies * acc_rows;
    uint32_t* sets = reinterpret_cast<uint32_t*>(staging);
    volatile OverlapSet* ctl = reinterpret_cast<volatile OverlapSet*>(sets + kOverlapSets * set_words);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t kWarps = blockDim.x >> 5;
    const int64_t G = gridDim.x;

    // what this CTA owns of matrix i
    auto share = [&](int i, int64_t& nq, int64_t& U, int64_t& ub, int64_t& ue) {
        const GemvMat& M = mm.m[i];
        nq = ((M.k_in + 23) / 24 + 3) / 4;
        U = ((M.n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
        ub = blockIdx.x * U / G; ue = (blockIdx.x + 1) * U / G;
    };
    // prepare set i % kOverlapSets for matrix i with the calling threads (`nthreads` of them, numbered `tid`)
    auto prepare = [&](int i, int tid, int nthreads) {
        const GemvMat& M = mm.m[i];
        uint32_t* xs = sets + (i % kOverlapSets) * set_words;
        float* acc = reinterpret_cast<float*>(xs + xs_words);
        const int64_t words = (int64_t)(((M.k_in + 23) / 24 + 3) / 4) * 48;
        for (int64_t w = tid; w < words; w += nthreads) {
            const int64_t e = 2 * w;
            const uint32_t lo = e < M.k_in ? __ldg(M.x + e) : 0u, hi = e + 1 < M.k_in ? __ldg(M.x + e + 1) : 0u;
            xs[w] = lo | hi << 16;
        }
        for (int r = tid; r < kSortAccCopies * acc_rows; r += nthreads) acc[r] = 0.f;
    };

    if (threadIdx.x < kOverlapSets) { ctl[threadIdx.x].next_chunk = 0u; ctl[threadIdx.x].arrived = 0u; ctl[threadIdx.x].ready = 0u; }
    for (int i = 0; i < kOverlapSets && i < mm.n; ++i) prepare(i, (int)threadIdx.x, (int)blockDim.x);
    __syncthreads();
    if (threadIdx.x < kOverlapSets && (int)threadIdx.x < mm.n) ctl[threadIdx.x].ready = threadIdx.x + 1u;
    __syncthreads();

    for (int i = 0; i < mm.n; ++i) {
        const GemvMat& M = mm.m[i];
        const int set = i % kOverlapSets;
        int64_t nq, U, ub, ue;
        share(i, nq, U, ub, ue);
        const int64_t bpr = (M.k_in + 23) / 24;
        const int64_t rg0 = ub / nq, rg1 = ub < ue ? (ue - 1) / nq : rg0 - 1;
        // the set is prepared for this matrix long before a warp gets here; a bounded wait all the same
        {
            uint32_t spins = 0;
            while (ctl[set].ready != (uint32_t)i + 1u && ++spins < kOverlapSpins) {}
            if (ctl[set].ready != (uint32_t)i + 1u) { if (lane == 0) atomicOr(fa.flags, 1u); return; }
            __threadfence_block();
        }
        const uint32_t* xs = sets + set * set_words;
        float* acc = reinterpret_cast<float*>(sets + set * set_words + xs_words);
        const uint32_t nchunks = (uint32_t)(ue - ub), nq32 = (uint32_t)nq;
        const uint32_t kq_a = (uint32_t)(ub - rg0 * nq);
        const unsigned long long* seg = static_cast<const unsigned long long*>(M.weights) + ub * 32 + lane;
        if (i + 1 < mm.n && warp == 0) {                    // ask for the next matrix's first chunks in L2
            int64_t nq2, U2, ub2, ue2;
            share(i + 1, nq2, U2, ub2, ue2);
            const unsigned long long* nxt = static_cast<const unsigned long long*>(mm.m[i + 1].weights) + ub2 * 32;
            for (int c = lane; c < 64 && ub2 + c / 2 < ue2; c += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(nxt + c * 16));
        }
        uint32_t ch = 0;
        if (lane == 0) ch = atomicAdd(const_cast<uint32_t*>(&ctl[set].next_chunk), 1u);
        ch = __shfl_sync(kFullMask, ch, 0);
        unsigned long long e = ch < nchunks ? __ldg(seg + (uint64_t)ch * 32) : 0ull;
        while (ch < nchunks) {
            uint32_t nxt = 0;
            if (lane == 0) nxt = atomicAdd(const_cast<uint32_t*>(&ctl[set].next_chunk), 1u);
            nxt = __shfl_sync(kFullMask, nxt, 0);
            const unsigned long long e_next = nxt < nchunks ? __ldg(seg + (uint64_t)nxt * 32) : 0ull;
            const uint64_t I = e & kSortIndexMask;
            const uint32_t pos = (uint32_t)(e >> 48);
            const bool valid = I != kSortIndexMask && I < fa.n_points;
            const uint32_t v = kq_a + (pos >> 5);
            uint32_t q = __umulhi(v, M.nq_magic), kq = v - q * nq32;
            if (kq >= nq32) { kq -= nq32; ++q; }
            const uint32_t rloc = q * kGemvGroupRows + ((pos >> 2) & 7u);                 // row inside the CTA's share
            const uint32_t cb = kq * 4u + (pos & 3u);
            float gn = 0.f;
            uint16_t gbits = 0;
            if (valid) gbits = ldg_u16_here(M.gain + ((int64_t)rg0 * kGemvGroupRows + rloc) * bpr + cb);
            Decoded r;
            decode_sorted_entry(fa, T, I, valid, r);
            gn = gain_to_float(gbits);
            uint32_t w[12];
            expand_bf16(r, gn, w);
            const uint4* xb = reinterpret_cast<const uint4*>(xs + cb * 12u);
            const uint4 x0 = xb[0], x1 = xb[1], x2 = xb[2];
            const uint32_t xv[12] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w};
            const float dot = dot24_bf16(w, xv);
            if (valid) atomicAdd(&acc[(warp & (kSortAccCopies - 1)) * acc_rows + rloc], dot);
            ch = nxt; e = e_next;
        }
        // out of chunks: count this warp in; the last one ends the pass and hands the set on
        __threadfence_block();
        uint32_t last = 0;
        if (lane == 0) last = atomicAdd(const_cast<uint32_t*>(&ctl[set].arrived), 1u) == kWarps - 1u;
        last = __shfl_sync(kFullMask, last, 0);
        if (last) {
            __threadfence_block();
            YOut yo{};
            yo.y = M.y;
            auto row_sum = [&](int64_t rr) {
                float vv = 0.f;
#pragma unroll
                for (int c = 0; c < kSortAccCopies; ++c) vv += acc[c * acc_rows + rr];
                return vv;
            };
            if (ub < ue) finish_pass<kOutBf16, false>(yo, rg0, rg1, nq, ub, ue, U, G, M.n_out, scratch, counters, row_sum, M.slot0, 0, 1);
            __syncwarp();
            if (i + kOverlapSets < mm.n) {
                if (lane == 0) { ctl[set].next_chunk = 0u; ctl[set].arrived = 0u; }
                prepare(i + kOverlapSets, lane, 32);
                __threadfence_block();
                __syncwarp();
                if (lane == 0) ctl[set].ready = (uint32_t)(i + kOverlapSets) + 1u;
            }
        }
    }
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

// The span of the index stream and of the gains that this CTA's row groups cover is contiguous: request it from DRAM ahead
// of time; the binning phases then read it from L2.
template <bool kSg>
__device__ __forceinline__ void prefetch_bin_span(const FastArgs& fa, const uint32_t* stream, const uint16_t* gain, const SgArgs& sg,
                                                  int64_t n_out, int64_t bpr)
{
    const int64_t nq0 = (bpr + 3) / 4, U0 = ((n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq0;
    const int64_t ub = blockIdx.x * U0 / gridDim.x, ue = (blockIdx.x + 1) * U0 / gridDim.x;
    if (ub < ue) {
        const uint64_t b_first = (uint64_t)(ub / nq0) * kGemvGroupRows * (uint64_t)bpr;
        const uint64_t b_last = (uint64_t)min(((ue - 1) / nq0 + 1) * kGemvGroupRows, n_out) * (uint64_t)bpr;
        const uint64_t wf = (uint64_t)fa.L.W + (kSg ? (uint64_t)sg.bits : 0ull);
        prefetch_span_l2(stream, b_first * wf / 8, (b_last * wf + 7) / 8);
        if (!kSg) prefetch_span_l2(gain, b_first * 2, b_last * 2);
    }
}

template <bool kOutBf16, bool kSg, bool kShard>
__device__ __forceinline__ void gemv_bin_body(const FastArgs& fa, const FastSmem& T, uint8_t* staging, const uint32_t* __restrict__ stream,
                                              const uint16_t* __restrict__ sort_rank, const uint16_t* __restrict__ gain, const SgArgs& sg,
                                              int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, int seg_units,
                                              const uint16_t* __restrict__ x, const YOut& yo, float* __restrict__ scratch,
                                              uint32_t* __restrict__ counters, int64_t slot0)
{
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
    const uint32_t nq32 = (uint32_t)nq;
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
            uint16_t gbits = 0;
            if (valid) {
                if (kSg) {
                    const float scale = sg.row_scale ? __ldg(sg.row_scale + (int64_t)rg0 * kGemvGroupRows + rloc) : 1.f;
                    gn = __fmul_rn(__fmul_rn(scale, __ldg(sg.codebook + (cls16 >> 10))), __uint_as_float(T.desc[cls * kFastDescStride + kFastDescRnorm]));
                } else {
                    gbits = ldg_u16_here(gain_pass + (int64_t)rloc * bpr + cb);
                }
            }
            Decoded r;
            decode_known_class(T, cls, e & ((1ull << 48) - 1ull), valid, r);
            if (!kSg) gn = gain_to_float(gbits);
            uint32_t w[12];
            expand_bf16(r, gn, w);
            const uint4* xb = reinterpret_cast<const uint4*>(xs + cb * 12u);
            const uint4 x0 = xb[0], x1 = xb[1], x2 = xb[2];
            const uint32_t xv[12] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w, x2.x, x2.y, x2.z, x2.w};
            const float dot = dot24_bf16(w, xv);
            if (valid) atomicAdd(&acc[(warp & (kSortAccCopies - 1)) * (kGemvGroupsPerPass * kGemvGroupRows) + rloc], dot);
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
        finish_pass<kOutBf16, kShard>(yo, rg0, rg1, nq, ub, ue, U, G, n_out, scratch, counters, row_sum, slot0);
        __syncthreads();
    }, seg_units);
}

template <bool kOutBf16, bool kSg = false, bool kShard = false>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_bin_kernel(FastArgs fa, const uint32_t* __restrict__ stream, const uint16_t* __restrict__ sort_rank, const uint16_t* __restrict__ gain, SgArgs sg,
                int64_t n_out, int64_t k_in, int64_t bpr, uint32_t nq_magic, int seg_units, const uint16_t* __restrict__ x, YOut yo,
                float* __restrict__ scratch, uint32_t* __restrict__ counters)
{
    prefetch_bin_span<kSg>(fa, stream, gain, sg, n_out, bpr);       // while the table image is on its way
    FAST_PROLOGUE(if (kShard) shard_arrive(yo));
    gemv_bin_body<kOutBf16, kSg, kShard>(fa, T, staging, stream, sort_rank, gain, sg, n_out, k_in, bpr, nq_magic, seg_units, x, yo, scratch, counters, 0);
    if (kShard) shard_arrive(yo);
}

// Several independent matrices on their stored streams in one launch.
template <bool kOutBf16>
__global__ void __launch_bounds__(kSortThreads, 1)
gemv_bin_multi_kernel(FastArgs fa, const uint16_t* __restrict__ sort_rank, const __grid_constant__ GemvMulti mm, float* __restrict__ scratch,
                      uint32_t* __restrict__ counters)
{
    prefetch_bin_span<false>(fa, static_cast<const uint32_t*>(mm.m[0].weights), mm.m[0].gain, SgArgs{}, mm.m[0].n_out, (mm.m[0].k_in + 23) / 24);
    FAST_PROLOGUE();
    for (int i = 0; i < mm.n; ++i) {
        const GemvMat& M = mm.m[i];
        if (i + 1 < mm.n)
            prefetch_bin_span<false>(fa, static_cast<const uint32_t*>(mm.m[i + 1].weights), mm.m[i + 1].gain, SgArgs{}, mm.m[i + 1].n_out,
                                     (mm.m[i + 1].k_in + 23) / 24);
        YOut yo{};
        yo.y = M.y;
        gemv_bin_body<kOutBf16, false, false>(fa, T, staging, static_cast<const uint32_t*>(M.weights), sort_rank, M.gain, SgArgs{}, M.n_out, M.k_in,
                                              (M.k_in + 23) / 24, M.nq_magic, M.seg_units, M.x, yo, scratch, counters, M.slot0);
        __syncthreads();
    }
}
