// The fused dequant + small-batch GEMM entry points of the C ABI (see include/llvq.h): stored stream, sorted layout,
// shape-gain form, the row-sharded variants and the entry point that allocates nothing, with the kernels they launch
// (gemm_kernels.cuh; tcgen05 with the accumulator in tensor memory).
#include "kernels_common.cuh"

namespace {

#include "gemv_kernels.cuh"
#include "gemm_kernels.cuh"

// The codes whose class tables stay in global memory have room for the table of small subsets beside the GEMM's buffers.
size_t gemm_image_bytes(const llvq_ctx* ctx) { return ctx->fast ? ctx->fl.total : ctx->fl.total_ext; }

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
                        const YOut* yo = nullptr, int64_t y_ld = 0, const SgArgs* sg = nullptr, int y_f32 = 0)
{
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    GemmArgs ga;
    ga.y = d_y_bf16; ga.y_ld = n_out; ga.shard = nullptr; ga.y_f32 = y_f32; ga.sort_rank = nullptr; ga.nbins = 0; ga.bin_round = 0;
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
    const size_t head = (gemm_image_bytes(ctx) + 64 + 1023) & ~size_t(1023), a_set = (size_t)kDomStages * kGemmRows * kStageK * 2,
                 x_set = (size_t)kDomStages * ga.npad * kStageK * 2;
    int pipe = 0, b_double = 0;
    size_t smem = head + (size_t)dpi * (a_set + x_set);
    if (head + 2 * a_set + 2 * x_set <= 227 * 1024) { pipe = 1; b_double = 1; smem = head + 2 * a_set + 2 * x_set; }
    else if (head + 2 * a_set + x_set <= 227 * 1024) { pipe = 1; smem = head + 2 * a_set + x_set; }
    if (smem > 227 * 1024) return LLVQ_EUNSUPPORTED;
#define LLVQ_LAUNCH_DOMAINS(BIG, SG, SH)                                                                                      \
    do {                                                                                                                     \
        if (pipe) {                                                                                                          \
            if (!set_smem(gemm_pipe_kernel<BIG, SG, SH>, smem)) return LLVQ_ECUDA;                                            \
            if (launch_pdl(gemm_pipe_kernel<BIG, SG, SH>, grid, (unsigned)kGemmThreads, smem, (cudaStream_t)stream, fast_args(ctx, !ctx->fast), \
                           static_cast<const unsigned long long*>(p), d_gain_f16, sga, ga, b_double) != cudaSuccess) return LLVQ_ECUDA; \
        } else {                                                                                                             \
            if (!set_smem(gemm_sorted_kernel<BIG, SG, SH>, smem)) return LLVQ_ECUDA;                                          \
            if (launch_pdl(gemm_sorted_kernel<BIG, SG, SH>, grid, (unsigned)kGemmThreads, smem, (cudaStream_t)stream, fast_args(ctx, !ctx->fast), \
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
    ga.y = d_y_bf16; ga.y_ld = n_out; ga.shard = nullptr; ga.y_f32 = 0; ga.sort_rank = nullptr; ga.nbins = 0; ga.bin_round = 0;
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
    const size_t img = gemm_image_bytes(ctx);
    const size_t smem = ((img + 64 + 1023) & ~size_t(1023)) + 2 * kGemmRows * kStageK * 2 + 2 * (size_t)ga.npad * kStageK * 2;
    if (smem > 227 * 1024) return LLVQ_EUNSUPPORTED;
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    if (yo && sg) return LLVQ_EUNSUPPORTED;              // row-sharded: stored-gain form only
    // codes with their class tables in shared memory and many classes (a warp of 32 unrelated blocks is what costs there):
    // the kernel that puts every domain of 1024 blocks into the order of the sorted layout before unranking it, as many
    // domains at a time (up to 4) as shared memory has room for beside the operand buffers
    const int ncls = (int)ctx->host.desc.size();
    if (ctx->fast && ctx->d_sort_rank && ncls >= 64 && ncls < 1024 && ctx->host.W + (sg ? sg->bits : 0) <= 48) {
        const size_t head = (img + 64 + 1023) & ~size_t(1023), a_set = (size_t)kDomStages * kGemmRows * kStageK * 2,
                     x_set = (size_t)kDomStages * ga.npad * kStageK * 2;
        GemmArgs gb = ga;
        gb.nstages = (int)((ga.bpr + kDomBlocks - 1) / kDomBlocks);            // domains per row tile
        gb.split = 1;
        gb.sort_rank = ctx->d_sort_rank;
        gb.nbins = (ncls + 1 + 31) / 32 * 32;                                    // one bin per class and one for "no block"
        const size_t bins = (size_t)gb.nbins * 4 + 32 * 4 + (size_t)kDomEntries * 8;   // per ordered domain
        const int dpi = ga.npad <= 32 ? 2 : 1;
        gb.bin_round = 4;
        while (gb.bin_round > dpi && head + (size_t)dpi * (a_set + x_set) + (size_t)gb.bin_round * bins > 227 * 1024) gb.bin_round -= dpi;
        const size_t smem_bin = head + (size_t)dpi * (a_set + x_set) + (size_t)gb.bin_round * bins;
        if (smem_bin <= 227 * 1024) {
            const unsigned grid_bin = (unsigned)std::min<int64_t>(row_tiles * gb.nstages, ctx->sm_count);
            const unsigned long long* words = static_cast<const unsigned long long*>(d_idx);
            const SgArgs sga = sg ? *sg : SgArgs{};
#define LLVQ_LAUNCH_BINNED(SG, SH, RD)                                                                                          \
    do {                                                                                                                        \
        if (!set_smem(gemm_sorted_kernel<false, SG, SH, true, RD>, smem_bin)) return LLVQ_ECUDA;                                 \
        if (launch_pdl(gemm_sorted_kernel<false, SG, SH, true, RD>, grid_bin, (unsigned)kGemmThreads, smem_bin, st, fast_args(ctx, false), words, \
                       d_gain_f16, sga, gb, dpi) != cudaSuccess) return LLVQ_ECUDA;                                             \
    } while (0)
            if (gb.bin_round > dpi) {                    // rounds of several iterations
                if (yo) LLVQ_LAUNCH_BINNED(false, true, true);
                else if (sg) LLVQ_LAUNCH_BINNED(true, false, true);
                else LLVQ_LAUNCH_BINNED(false, false, true);
            } else {
                if (yo) LLVQ_LAUNCH_BINNED(false, true, false);
                else if (sg) LLVQ_LAUNCH_BINNED(true, false, false);
                else LLVQ_LAUNCH_BINNED(false, false, false);
            }
#undef LLVQ_LAUNCH_BINNED
            return launch_status();
        }
    }
    // the 72-bit code at wide batches (one domain per iteration): the same with the coarse shape of the unranking as sort key,
    // four domains ordered per round (at padded batch <= 32 the pipeline kernel on unordered chunks is faster: measured)
    if (!ctx->fast && ctx->host.W > 64 && ctx->host.W <= 72 && ga.npad > 32 && !sg && (int)ctx->host.desc.size() <= (1 << kBigClassBits)) {
        const size_t head = (img + 64 + 1023) & ~size_t(1023), a_set = (size_t)kDomStages * kGemmRows * kStageK * 2,
                     x_set = (size_t)kDomStages * ga.npad * kStageK * 2;
        GemmArgs gb = ga;
        gb.nstages = (int)((ga.bpr + kDomBlocks - 1) / kDomBlocks);            // domains per row tile
        gb.split = 1;
        gb.nbins = 160;                                                         // 128 shapes; the last bin is "no block"
        gb.bin_round = 4;
        const size_t bins = (size_t)gb.nbins * 4 + 32 * 4 + (size_t)kDomEntries * (8 + 4);
        const int dpi = 1;
        const size_t smem_bin = head + (size_t)dpi * (a_set + x_set) + (size_t)gb.bin_round * bins;
        if (smem_bin <= 227 * 1024) {
            const unsigned grid_bin = (unsigned)std::min<int64_t>(row_tiles * gb.nstages, ctx->sm_count);
            const unsigned long long* words = static_cast<const unsigned long long*>(d_idx);
            if (yo) {
                if (!set_smem(gemm_sorted_kernel<true, false, true, true, true>, smem_bin)) return LLVQ_ECUDA;
                if (launch_pdl(gemm_sorted_kernel<true, false, true, true, true>, grid_bin, (unsigned)kGemmThreads, smem_bin, st, fast_args(ctx, true), words,
                               d_gain_f16, SgArgs{}, gb, dpi) != cudaSuccess) return LLVQ_ECUDA;
            } else {
                if (!set_smem(gemm_sorted_kernel<true, false, false, true, true>, smem_bin)) return LLVQ_ECUDA;
                if (launch_pdl(gemm_sorted_kernel<true, false, false, true, true>, grid_bin, (unsigned)kGemmThreads, smem_bin, st, fast_args(ctx, true), words,
                               d_gain_f16, SgArgs{}, gb, dpi) != cudaSuccess) return LLVQ_ECUDA;
            }
            return launch_status();
        }
    }
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
        if (launch_pdl(gemm_pipe_kernel<BIG, SG, SH, true>, grid_pipe, (unsigned)kGemmThreads, smem_pipe, st, fast_args(ctx, !ctx->fast), words, \
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
            if (launch_pdl(gemm_kernel<false, false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx, !ctx->fast), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
        } else {
            if (!set_smem(gemm_kernel<true, false, true>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemm_kernel<true, false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx, !ctx->fast), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
        }
    } else if (sg) {
        if (!set_smem(gemm_kernel<false, true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<false, true>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx, !ctx->fast), idx, d_gain_f16, *sg, ga) != cudaSuccess) return LLVQ_ECUDA;
    } else if (ctx->fast) {
        if (!set_smem(gemm_kernel<false, false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<false, false>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx, !ctx->fast), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(gemm_kernel<true, false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(gemm_kernel<true, false>, grid, (unsigned)kGemmThreads, smem, st, fast_args(ctx, !ctx->fast), idx, d_gain_f16, SgArgs{}, ga) != cudaSuccess) return LLVQ_ECUDA;
    }
    return launch_status();
}

}  // namespace

extern "C" {

// Sorted layout of the small-batch GEMM (see the comment at sort_blocks_gemm_kernel).
static bool gemm_sortable(const llvq_ctx* ctx)
{
    if (!ctx->fast) return (int)ctx->host.desc.size() <= (1 << kBigClassBits);   // 96-bit entries: class-local index (63 bits) + class + position
    return ctx->d_sort_rank && ctx->host.W <= 48 && ctx->host.N < (u128)kSortIndexMask;
}

size_t llvq_sorted_gemm_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in)
{
    if (!ctx || ctx->device < 0 || n_out <= 0 || k_in <= 0 || !gemm_sortable(ctx)) return 0;
    const int64_t bpr = (k_in + 23) / 24;
    return (size_t)(((n_out + kGemmRows - 1) / kGemmRows) * ((bpr + kDomBlocks - 1) / kDomBlocks)) * kDomEntries * (ctx->fast ? 8 : 4 * kBigEntryWords);
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
        sort_blocks_gemm_big_kernel<<<g, kDomEntries, 0, (cudaStream_t)stream>>>(fast_args(ctx, !ctx->fast), static_cast<const uint32_t*>(d_idx), n_out, bpr,
                                                                                 ndomains, static_cast<uint32_t*>(d_sorted));
        return launch_status();
    }
    const size_t smem = ctx->fl.total + 16;
    if (!set_smem(sort_blocks_gemm_kernel, smem)) return LLVQ_ECUDA;
    sort_blocks_gemm_kernel<<<g, kDomEntries, smem, (cudaStream_t)stream>>>(fast_args(ctx, !ctx->fast), static_cast<const uint32_t*>(d_idx), ctx->d_sort_rank,
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

}  // extern "C"

// llvq_gemv_sorted of the codes whose class tables stay in global memory: the batch-1 case of the sorted small-batch
// product (same layout, same kernel), with the output type of the GEMV.  Called from gemv.cu.
__attribute__((visibility("hidden")))
int llvq_internal_gemv_domains(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                               const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (!gemm_sortable(ctx) || n_out > kMaxScratchRows || k_in <= 0) return LLVQ_EUNSUPPORTED;
    if (!aligned(d_x_bf16, 16) || (k_in & 7)) return LLVQ_EALIGN;          // the tensor-core kernel stages x in 16-byte pieces
    return launch_gemm_domains(ctx, d_sorted, d_gain_f16, n_out, k_in, d_x_bf16, 1, static_cast<uint16_t*>(d_y), ctx->d_scratch, ctx->d_counters,
                               stream, nullptr, 0, nullptr, y_dtype == LLVQ_F32 ? 1 : 0);
}
