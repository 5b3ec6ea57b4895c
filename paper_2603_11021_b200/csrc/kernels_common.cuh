// Shared by the translation units of the library (llvq.cu, gemv.cu, gemm.cu): the arguments every table-image kernel
// takes, one block of 24 weights end to end (S1-S7), the kernels' prologue, launch helpers and the argument checks the
// entry points share.  Everything here has internal linkage: each translation unit gets its own copy.
#pragma once
#include "llvq.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
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

constexpr int kGemvGroupRows = 8;        // rows per GEMV work unit
constexpr int kGemvGroupsPerPass = 128;  // row groups whose sums a GEMV CTA keeps in shared memory at a time
constexpr int kGemmRows = 128;           // rows of a GEMM row tile
constexpr int kMaxScratchRows = 65536;
constexpr int kCounterWords = 64 * kMaxScratchRows / 8;      // the word after them counts the CTAs of a row-sharded GEMV that have finished

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


// ===========================================================================
// Fast path (tables in shared memory).  Dynamic shared memory of every fast
// kernel: [table image | mbarrier (16 bytes) | kernel-specific staging].
// Persistent CTAs, one per SM.
// ===========================================================================
constexpr int kFastThreads = 1024;      // decode / dequant kernels
constexpr int kGemvThreads = 1024;     // upper bound; the launch picks the warp count that divides the units per CTA best

struct FastArgs {
    FastLayout L;
    uint32_t image_bytes;           // what the kernel copies into shared memory: L.total, or L.total_ext (with the table of small subsets)
    const uint8_t* image;
    uint32_t* flags;
    unsigned long long* bad_index;
    uint64_t n_points;              // N when it fits 64 bits (fast path)
    DevCode dc;                     // class tables in global memory (big codes)
};

// One block of 24 weights, end to end, in the two forms the consumers use.  kBig selects the decoder for codes
// whose class tables live in global memory; otherwise everything is served from the shared-memory image.
// All 32 lanes of a warp call these together; `in` = the block exists.
// The table-driven decoder of the codes whose class tables stay in global memory, from the stored stream.
__device__ __forceinline__ void block_planes_big(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                                 uint64_t b, bool in, DecodedBig& d)
{
    uint64_t lo = 0, hi = 0;
    if (in) load_index(stream, b, fa.dc.W, lo, hi);
    const bool valid = in && (hi < fa.dc.n_hi || (hi == fa.dc.n_hi && lo < fa.dc.n_lo));
    if (in && !valid) atomicAdd(fa.bad_index, 1ull);
    uint64_t local = 0;
    const int cls = valid ? big_find_class(fa.dc, lo, hi, local) : 0;
    big_decode_planes(T, fa.dc, cls, local, valid, kFullMask, d);
}

template <bool kBig>
__device__ __forceinline__ void block_bytes(const FastArgs& fa, const FastSmem& T, const uint32_t* __restrict__ stream,
                                            uint64_t b, bool in, uint32_t w[6])
{
    if (kBig) {
        DecodedBig d{};
        block_planes_big(fa, T, stream, b, in, d);
        Decoded three = d.d;
        three.neg &= ~d.p3;                               // those positions are written by the patch (a negated zero filler would carry)
        expand_bytes(three, w);
        patch_id8_bytes(d, w);
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
        DecodedBig d{};
        block_planes_big(fa, T, stream, b, in, d);
        expand_bf16(d.d, g, w);
        patch_id8_bf16(d, g, w);
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
    Decoded d{};
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
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + fa.image_bytes);                          \
    [[maybe_unused]] uint8_t* staging = smem + fa.image_bytes + 16;                             \
    pdl_launch_dependents();                                                                    \
    const bool image_ok = fast_load_image(smem, fa.image, fa.image_bytes, bar, fa.flags);       \
    pdl_wait();                                                                                 \
    if (!image_ok) { __VA_ARGS__; return; }                                                     \
    const FastSmem T = fast_view(smem, fa.L, fa.image_bytes == fa.L.total_ext);

// ext: the kernel has room for the table of small subsets behind the image proper (see FastLayout::sub3)
FastArgs fast_args(const llvq_ctx* ctx, bool ext = false)
{
    FastArgs fa;
    fa.L = ctx->fl; fa.image = ctx->d_image;
    fa.image_bytes = ext ? ctx->fl.total_ext : ctx->fl.total; fa.flags = ctx->dev.flags; fa.bad_index = ctx->dev.bad_index;
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

int launch_status()
{
    return cudaGetLastError() == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA;
}


// Checks the destinations of a GEMV: every pointer present and aligned for the output type.
int check_yout(const YOut& yo, int y_dtype)
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

YOut single_y(void* d_y)
{
    YOut yo{};
    yo.y = d_y;
    return yo;
}

// Argument checks of the shape-gain entry points.
int check_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook, const float* d_row_scale)
{
    if (int e = check_common(ctx, d_fields)) return e;
    if (gain_bits < 0 || gain_bits > 8 || !d_codebook) return LLVQ_EINVAL;
    if (!aligned(d_codebook, 4) || !aligned(d_row_scale, 4)) return LLVQ_EALIGN;
    if (!ctx->fast || ctx->host.W + gain_bits > 64 || ctx->host.W > 63) return LLVQ_EUNSUPPORTED;
    return LLVQ_OK;
}

// Row-sharded GEMV: the destinations of one rank's band.  d_y_all[0..n_dest) are the ranks' full-length copies of y
// (own_slot = this rank's own copy), the band starts at row row0; d_flag_words (optional) = for every destination
// the word that receives `epoch` when the band is in place (the own slot's entry is not used).
int shard_yout(const llvq_ctx* ctx, void* const* d_y_all, int n_dest, int own_slot, int64_t row0, int y_dtype,
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
int signal_only(const llvq_ctx* ctx, const YOut& yo, void* stream)
{
    if (yo.n_flag == 0) return LLVQ_OK;
    return llvq_signal_ranks(ctx, yo.flag, yo.n_flag, yo.epoch, stream);
}

}  // namespace
