// The fused dequant + small-batch GEMM kernels (tcgen05, accumulator in tensor memory): the kernel with two thread
// groups on alternating stages, the sorted layouts (sort kernels and the consumer with a block barrier), and the
// kernel without a block barrier that both entry points run for the 48-bit codes.  Included by gemm.cu inside its
// unnamed namespace, after kernels_common.cuh and gemv_kernels.cuh (unit_owner, shard_arrive).
#pragma once

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
constexpr int kStageBlocks = 4;                       // column blocks per stage
constexpr int kStageK = kStageBlocks * 24;            // 96
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
    int y_f32;                 // Y holds binary32 instead of bf16 (the batch-1 product behind llvq_gemv_sorted of the 72-bit code)
    const uint16_t* sort_rank; // stored stream ordered inside the kernel (gemm_sorted_kernel<.., kBin>): sort key of every class, else null
    int nbins;                 // ... and the number of bins (a multiple of 32 above the largest key; the last bin is "no block")
    int bin_round;             // ... and how many domains are ordered at a time (a multiple of the domains per iteration, at most 4)
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
    if (!kShard && ga.y_f32) { reinterpret_cast<float*>(ga.y)[at] = v; return; }
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
    const uint32_t img_bytes = fa.image_bytes;
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
    const bool image_ok = fast_load_image(smem, fa.image, fa.image_bytes, bar_img, fa.flags);
    pdl_wait();                                        // also when the image did not arrive: the dependents of this launch rely on it
    if (!image_ok) {
        if (kShard) shard_arrive(*ga.shard);           // the peers must not wait for this rank
        return;
    }
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

// The same layout for codes whose class tables live in global memory (72-bit indices): 96-bit entries (three 32-bit
// words).  An index is stored as its two digits in the mixed radix of the class table (App. A step 2, taken when the
// layout is made): words 0-1 = the class-local index I - offset[class] (class sizes fit 63 bits; bit 63 set marks "no
// block": ragged edge or index out of range), word 2 = class (17 bits) | position in the domain << 17 (10 bits).  The
// kernel then needs neither the bucket table nor the 128-bit offsets, and the class record can be requested as soon as
// the entry is there.  The blocks of a domain are ordered by the shape of their unranking: parity (odd first), number of
// steps (most first), which of the steps take at most three slots, steps of the first group; the lanes of a warp then
// run the same trip counts over similar slot counts and mostly agree on the cheap form of a step.
// Inside the kernels an entry travels as two 64-bit words: x = the class-local index (stored stream: index bits 0..63),
// y = class << 8 | position << 32, bit 63 = no block (stored stream: index bits 64..71 in the low byte).
constexpr unsigned long long kBigNoBlock = 1ull << 63;
constexpr int kBigEntryWords = 3;
constexpr int kBigClassBits = 17;

// Top 16 bits of a W-bit index (hi:lo): the bucket of the class table.
__device__ __forceinline__ uint32_t big_bucket(const DevCode& dc, uint64_t lo, uint64_t hi)
{
    const int sh = dc.W > 16 ? dc.W - 16 : 0;
    return (uint32_t)(sh >= 64 ? hi >> (sh - 64) : (sh ? (lo >> sh) | (hi << (64 - sh)) : lo)) & 0xffffu;
}

// Entry `at` of a sorted stream of 96-bit entries, in the two-word form the kernels use.
__device__ __forceinline__ ulonglong2 load_big_entry(const void* sorted, int64_t at)
{
    const uint32_t* p = static_cast<const uint32_t*>(sorted) + at * kBigEntryWords;
    const uint32_t w0 = __ldg(p), w1 = __ldg(p + 1), w2 = __ldg(p + 2);
    const unsigned long long pos = w2 >> kBigClassBits, cls = w2 & ((1u << kBigClassBits) - 1u);
    return make_ulonglong2((unsigned long long)(w1 & 0x7fffffffu) << 32 | w0,
                           ((unsigned long long)(w1 >> 31) << 63) | cls << 8 | pos << 32);
}

__global__ void __launch_bounds__(kDomEntries, 1)
sort_blocks_gemm_big_kernel(FastArgs fa, const uint32_t* __restrict__ stream, int64_t n_out, int64_t bpr, int64_t ndomains,
                            uint32_t* __restrict__ out)
{
    __shared__ uint32_t keys[kDomEntries];
    __shared__ unsigned long long ex[kDomEntries], ey[kDomEntries];
    const int64_t nd = (bpr + kDomBlocks - 1) / kDomBlocks;
    const int i = threadIdx.x;
    for (int64_t dom = blockIdx.x; dom < ndomains; dom += gridDim.x) {
        const int64_t rt = dom / nd, d = dom - rt * nd;
        const int64_t row = rt * kGemmRows + (i >> 3), cb = d * kDomBlocks + (i & 7);
        unsigned long long x = kBigNoBlock, y = (unsigned long long)i << kBigClassBits;   // words 0-1 and word 2 of an entry
        uint32_t key = 0x7ffffc00u | (uint32_t)i;                   // no block: after everything else
        if (row < n_out && cb < bpr) {
            uint64_t lo, hi;
            load_index(stream, (uint64_t)(row * bpr + cb), fa.dc.W, lo, hi);
            if (hi < fa.dc.n_hi || (hi == fa.dc.n_hi && lo < fa.dc.n_lo)) {
                uint64_t local;
                const uint32_t cls = (uint32_t)big_find_class(fa.dc, lo, hi, local);
                const uint32_t* rec = reinterpret_cast<const uint32_t*>(fa.dc.big + cls);
                const uint32_t h = __ldg(rec), small_k = __ldg(rec + 6) >> 24;
                const uint32_t nlev = h >> 28, nlev1 = (h >> 24) & 7u, parity = (h >> 16) & 1u;
                x = local;
                y = (unsigned long long)cls | (unsigned long long)i << kBigClassBits;
                // odd classes first (their steps choose among up to 24 slots, the even classes' among at most 16), then by steps
                key = (1u - parity) << 24 | (7u - min(nlev, 7u)) << 21 | (small_k & 0x7fu) << 14 | nlev1 << 11 | (uint32_t)i;
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
        uint32_t* o = out + (dom * kDomEntries + i) * kBigEntryWords;
        o[0] = (uint32_t)ex[src]; o[1] = (uint32_t)(ex[src] >> 32); o[2] = (uint32_t)ey[src];
        __syncthreads();
    }
}

// kBin: `sorted` points at the stored stream instead; at the start of an iteration every thread looks up the class of
// one block per domain (S1-S2) and the CTA puts the 1024 fields of a domain into the order of the sorted layout with a
// counting sort in shared memory (one bin per class), so that the unranking below runs on the same entries as with a
// stream sorted at load time.  ga.bin_round domains are ordered at a time (their four block barriers are then paid once per
// round, not once per iteration); the stream words of the next round are requested in L2 a round ahead.
// kRound (with kBin): a round is longer than an iteration; else it is one iteration and the words come through registers.
// kBin with kBig (class tables in global memory; rounds only): the bins are the coarse shape of the unranking (parity,
// number of steps, steps of the first group: 128 bins) instead of the full key of the sorted layout, the entries
// (class-local index, class | position) as in the 96-bit layout; the class look-ups of a round's domains (dependent
// reads from L2) run side by side.
template <bool kBig, bool kSg = false, bool kShard = false, bool kBin = false, bool kRound = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_sorted_kernel(FastArgs fa, const unsigned long long* __restrict__ sorted, const uint16_t* __restrict__ gain, SgArgs sg, GemmArgs ga, int dpi)
{
    static_assert(!(kBin && kBig && (kSg || !kRound)), "in-kernel ordering for the codes with tables in global memory: stored gains, rounds");
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t img_bytes = fa.image_bytes;
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
    // kBin: per domain of the iteration the bins (block counts, then the first slot of every bin), the warp totals of their prefix sum
    // and the ordered entries
    constexpr int kMaxRound = kRound ? 4 : 2;
    const int nround = kBin ? ga.bin_round : 1;
    uint32_t* bin_hist = reinterpret_cast<uint32_t*>(b_buf + (uint32_t)dpi * kDomStages * b_stage);   // [nround][nbins] counts, then first slots
    uint32_t* bin_wt = bin_hist + nround * ga.nbins;                        // [nround][32]
    unsigned long long* bin_ent = reinterpret_cast<unsigned long long*>(bin_wt + nround * 32);          // [nround][1024]
    uint32_t* bin_ent2 = reinterpret_cast<uint32_t*>(bin_ent + nround * kDomEntries);                    // kBig: [nround][1024] class | position << 17

    pdl_launch_dependents();
    const bool image_ok = fast_load_image(smem, fa.image, fa.image_bytes, bar_img, fa.flags);
    pdl_wait();                                        // also when the image did not arrive: the dependents of this launch rely on it
    if (!image_ok) {
        if (kShard) shard_arrive(*ga.shard);           // the peers must not wait for this rank
        return;
    }
    const FastSmem T = fast_view(smem, fa.L);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (kBin)
        for (int i = threadIdx.x; i < nround * ga.nbins; i += kGemmThreads) bin_hist[i] = 0u;
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
            if (kBin) {       // a round is one iteration (no room for more): the stream words that hold the field of this thread's block
                              // (position = thread) are requested an iteration ahead into registers; y bit 63 = no block
                if (kRound) return no_entry;             // longer rounds ask for them in L2 instead, see below
                const int64_t row = rt * kGemmRows + (threadIdx.x >> 3), cb = (int64_t)(d + q) * kDomBlocks + (threadIdx.x & 7u);
                if (row < ga.n_out && cb < ga.bpr)
                    return load_field_words(reinterpret_cast<const uint32_t*>(sorted), (uint64_t)(row * ga.bpr + cb), (int)fa.L.W + (kSg ? sg.bits : 0));
                return no_entry;
            }
            // warp 0 also issues the MMAs of every iteration: it takes the cheapest chunk of each domain (the last), the other
            // warps pair chunk w - 1 of the first domain with chunk 31 - w of the second
            const int chunk = warp == 0 ? 31 : (q == 0 ? warp - 1 : 31 - warp);
            const int64_t at = (rt * nd + d + q) * kDomEntries + chunk * 32 + lane;
            if (kBig) return load_big_entry(sorted, at);
            return make_ulonglong2(__ldg(sorted + at), 0ull);
        };
        ulonglong2 e0 = entry_at(d_begin, 0), e1 = dpi > 1 ? entry_at(d_begin, 1) : no_entry;
        for (int d0 = d_begin; d0 < d_end; d0 += dpi, ++uses) {
            const int nd_now = min(dpi, d_end - d0);
            ulonglong2 cur0 = e0, cur1 = e1;
            e0 = entry_at(d0 + dpi, 0);
            if (dpi > 1) e1 = entry_at(d0 + dpi, 1);
            if (kBin) {
                const int in_round = kRound ? (d0 - d_begin) % nround : 0;  // this iteration's first domain inside the round
                if (in_round == 0) {
                    // ---- order the fields of the round's domains, each by the sort key of its blocks' classes
                    const uint32_t nbins = (uint32_t)ga.nbins;
                    const int wbits = (int)fa.L.W + (kSg ? sg.bits : 0);
                    const int nr = min(nround, d_end - d0);                  // domains in this round
                    const uint32_t* words = reinterpret_cast<const uint32_t*>(sorted);
                    const int64_t row = rt * kGemmRows + (threadIdx.x >> 3);
                    unsigned long long f[kMaxRound];
                    uint32_t f2[kMaxRound];                                  // kBig: class | position << 17
                    uint32_t key[kMaxRound], rank[kMaxRound], cnt[kMaxRound], incl[kMaxRound];
#pragma unroll
                    for (int r = 0; r < kMaxRound; ++r) {
                        f[r] = kBig ? kBigNoBlock : kSortIndexMask; f2[r] = threadIdx.x << kBigClassBits;
                        key[r] = nbins - 1u; rank[r] = cnt[r] = incl[r] = 0u;
                        if (r >= nr) continue;
                        const int64_t cb = (int64_t)(d0 + r) * kDomBlocks + (threadIdx.x & 7u);
                        if (kBig) {
                            if (row < ga.n_out && cb < ga.bpr) {
                                uint64_t lo, hi;
                                load_index(words, (uint64_t)(row * ga.bpr + cb), fa.dc.W, lo, hi);
                                if (hi < fa.dc.n_hi || (hi == fa.dc.n_hi && lo < fa.dc.n_lo)) {
                                    uint64_t local;
                                    const uint32_t cls = (uint32_t)big_find_class(fa.dc, lo, hi, local);
                                    const uint32_t h = __ldg(reinterpret_cast<const uint32_t*>(fa.dc.big + cls));
                                    const uint32_t nlev = h >> 28, nlev1 = (h >> 24) & 7u, parity = (h >> 16) & 1u;
                                    key[r] = (1u - parity) << 6 | (7u - min(nlev, 7u)) << 3 | nlev1;
                                    f[r] = local;
                                    f2[r] |= cls;
                                } else {
                                    atomicAdd(fa.bad_index, 1ull);
                                }
                                const int64_t cbn = cb + (int64_t)nround * kDomBlocks;
                                if (d0 + r + nround < d_end && cbn < ga.bpr)
                                    asm volatile("prefetch.global.L2 [%0];" ::"l"(words + (((uint64_t)(row * ga.bpr + cbn) * (uint64_t)fa.dc.W) >> 5)));
                            }
                        } else if (row < ga.n_out && cb < ga.bpr) {
                            if (!kRound) f[r] = field_of_words(r == 0 ? cur0 : cur1, wbits);            // requested an iteration ago
                            else f[r] = load_field(words, (uint64_t)(row * ga.bpr + cb), wbits);
                            const uint64_t I = kSg ? f[r] & ((1ull << fa.L.W) - 1ull) : f[r];
                            if (I < fa.n_points) {
                                uint64_t local;
                                key[r] = __ldg(ga.sort_rank + fast_find_class(T, I, local));
                            } else {
                                atomicAdd(fa.bad_index, 1ull);
                                f[r] = kSortIndexMask;
                            }
                            // the same block of the next round: ask for its stream words in L2
                            const int64_t cbn = cb + (int64_t)nround * kDomBlocks;
                            if (kRound && d0 + r + nround < d_end && cbn < ga.bpr)
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(words + (((uint64_t)(row * ga.bpr + cbn) * (uint64_t)wbits) >> 5)));
                        }
                        rank[r] = atomicAdd(&bin_hist[r * nbins + key[r]], 1u);   // its place among the blocks of its bin
                    }
                    __syncthreads();
#pragma unroll
                    for (int r = 0; r < kMaxRound; ++r) {
                        if (r >= nr) continue;
                        cnt[r] = threadIdx.x < nbins ? bin_hist[r * nbins + threadIdx.x] : 0u;
                        uint32_t v = cnt[r];
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(kFullMask, v, o); if (lane >= o) v += t; }
                        incl[r] = v;
                        if (lane == 31) bin_wt[r * 32 + warp] = v;
                    }
                    __syncthreads();
#pragma unroll
                    for (int r = 0; r < kMaxRound; ++r) {
                        if (r >= nr) continue;
                        uint32_t v = bin_wt[r * 32 + lane];                  // every warp scans the 32 warp totals
                        const uint32_t own = v;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(kFullMask, v, o); if (lane >= o) v += t; }
                        const uint32_t before = __shfl_sync(kFullMask, v - own, warp);
                        if (threadIdx.x < nbins) bin_hist[r * nbins + threadIdx.x] = before + incl[r] - cnt[r];
                    }
                    __syncthreads();
#pragma unroll
                    for (int r = 0; r < kMaxRound; ++r) {
                        if (r >= nr) continue;
                        const uint32_t slot = bin_hist[r * nbins + key[r]] + rank[r];
                        if (kBig) { bin_ent[r * kDomEntries + slot] = f[r]; bin_ent2[r * kDomEntries + slot] = f2[r]; }
                        else bin_ent[r * kDomEntries + slot] = f[r] | (unsigned long long)threadIdx.x << 48;
                    }
                    __syncthreads();
                    for (int i = threadIdx.x; i < nround * (int)nbins; i += kGemmThreads) bin_hist[i] = 0u;   // for the next round (barriers follow below)
                }
                auto ordered = [&](int at) {                               // entry `at` of the round's ordered domains in the form the unranking takes
                    if (!kBig) return make_ulonglong2(bin_ent[at], 0ull);
                    const unsigned long long x = bin_ent[at];
                    const uint32_t y2 = bin_ent2[at];
                    return make_ulonglong2(x & ~kBigNoBlock, (x & kBigNoBlock) | (unsigned long long)(y2 & ((1u << kBigClassBits) - 1u)) << 8 |
                                                                  (unsigned long long)(y2 >> kBigClassBits) << 32);
                };
                cur0 = ordered(in_round * kDomEntries + (warp == 0 ? 31 : warp - 1) * 32 + lane);
                if (nd_now > 1) cur1 = ordered((in_round + 1) * kDomEntries + (warp == 0 ? 31 : 31 - warp) * 32 + lane);
            }
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
                uint16_t gbits = 0;
                if (!kSg && valid) gbits = ldg_u16_here(gain + row * ga.bpr + cb);
                float gn = 0.f;                                               // the gain is converted once the block is unranked
                uint32_t w[12];
                if (kBig) {
                    const int cls = valid ? (int)((uint32_t)(e.y >> 8) & 0xffffffu) : 0;
                    DecodedBig dec{};
                    big_decode_planes(T, fa.dc, cls, valid ? e.x : 0ull, valid, kFullMask, dec);
                    gn = gain_to_float(gbits);
                    expand_bf16(dec.d, gn, w);
                    patch_id8_bf16(dec, gn, w);
                } else {
                    Decoded dec{};
                    const uint32_t cls = decode_sorted_entry(fa, T, I, valid, dec);
                    if (!kSg) gn = gain_to_float(gbits);
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
    const uint32_t img_bytes = fa.image_bytes;
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
    const bool image_ok = fast_load_image(smem, fa.image, fa.image_bytes, bar_img, fa.flags);
    pdl_wait();                                        // also when the image did not arrive: the dependents of this launch rely on it
    if (!image_ok) {
        if (kShard) shard_arrive(*ga.shard);           // the peers must not wait for this rank
        return;
    }
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
                if (kBig) return load_big_entry(sorted, at);
                return make_ulonglong2(__ldg(sorted + at), 0ull);
            };
            uint32_t tk = (uint32_t)warp - 1u;
            ulonglong2 e = entry_of(tk);
            // sorted 96-bit entries name their class: its record is requested while the previous chunk is still being expanded
            uint4 rec0 = make_uint4(0u, 0u, 0u, 0u), rec1 = rec0;
            if (kBig && !kStored) big_load_record(fa.dc, (int)((uint32_t)(e.y >> 8) & 0xffffffu), !(e.y >> 63), rec0, rec1);
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
                uint16_t gbits = 0;
                if (!kSg && valid) gbits = ldg_u16_here(gain + row * ga.bpr + cb);
                float gn = 0.f;                                               // the gain is converted once the block is unranked
                uint32_t w[12];
                if (kBig) {
                    int cls = 0;
                    uint64_t local = 0;
                    DecodedBig dec{};
                    if (kStored) {
                        if (valid) cls = big_find_class(fa.dc, e.x, e.y & 0xffull, local);
                        big_decode_planes(T, fa.dc, cls, local, valid, kFullMask, dec);
                    } else {
                        big_decode_record(T, rec0, rec1, valid ? e.x : 0ull, valid, kFullMask, dec);
                        // the next chunk's entries were requested a whole chunk ago: they are here, and their records have the
                        // rest of this iteration to arrive
                        big_load_record(fa.dc, (int)((uint32_t)(e_next.y >> 8) & 0xffffffu), !(e_next.y >> 63), rec0, rec1);
                    }
                    gn = gain_to_float(gbits);
                    expand_bf16(dec.d, gn, w);
                    patch_id8_bf16(dec, gn, w);
                } else {
                    Decoded dec{};
                    uint32_t cls;
                    if (kStored) {
                        if (field != kSortIndexMask && !valid) atomicAdd(fa.bad_index, 1ull);
                        uint64_t local = 0;
                        cls = valid ? fast_find_class(T, I, local) : 0u;
                        fast_decode_local<-1>(T, cls, local, valid, kFullMask, dec);
                    } else {
                        cls = decode_sorted_entry(fa, T, I, valid, dec);
                    }
                    if (!kSg) gn = gain_to_float(gbits);
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
