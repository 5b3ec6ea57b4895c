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

// The optional argument is what a kernel still owes its peers when the table image did not arrive (the row-sharded
// kernels count themselves in so that the other ranks do not wait for them).  Also on that path the kernel waits for
// its predecessor before it retires, so that its own programmatic dependent never passes its wait too early.
#define FAST_PROLOGUE(...)                                                                      \
    extern __shared__ __align__(128) uint8_t smem[];                                            \
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + fa.L.total);                              \
    [[maybe_unused]] uint8_t* staging = smem + fa.L.total + 16;                                 \
    pdl_launch_dependents();                                                                    \
    const bool image_ok = fast_load_image(smem, fa.image, fa.L.total, bar, fa.flags);           \
    pdl_wait();                                                                                 \
    if (!image_ok) { __VA_ARGS__; return; }                                                     \
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

#include "gemv_kernels.cuh"
#include "gemm_kernels.cuh"

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
