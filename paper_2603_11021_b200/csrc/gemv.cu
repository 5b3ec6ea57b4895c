// The fused dequant + GEMV entry points of the C ABI (see include/llvq.h): stored stream, sorted layout, shape-gain
// form and the row-sharded variants, with the kernels they launch (gemv_kernels.cuh).
#include "kernels_common.cuh"

int llvq_internal_gemv_domains(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
                               const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream);      // gemm.cu

namespace {

#include "gemv_kernels.cuh"

constexpr size_t kSmemLimit = 227 * 1024;

// Shared memory of gemv_bin_kernel for `su` units per segment, and whether the table of small subsets still fits.
void bin_smem(const llvq_ctx* ctx, int64_t nq, int su, size_t& bytes, bool& ext)
{
    const size_t rest = 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16 + 2 * 1024 * 4 + (size_t)su * 32 * (8 + 2);
    ext = ctx->fl.total_ext + rest <= kSmemLimit;
    bytes = (ext ? ctx->fl.total_ext : ctx->fl.total) + rest;
}

// The same for gemv_sorted_kernel.
void sorted_smem(const llvq_ctx* ctx, int64_t nq, size_t& bytes, bool& ext)
{
    const size_t rest = 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16;
    ext = ctx->fl.total_ext + rest <= kSmemLimit;
    bytes = (ext ? ctx->fl.total_ext : ctx->fl.total) + rest;
}

bool bin_kernel_serves(const llvq_ctx* ctx, int64_t nq, const SgArgs* sg)
{
    size_t bytes; bool ext;
    bin_smem(ctx, nq, kBinSegUnits, bytes, ext);
    return (!sg || sg->bits <= 5) && ctx->fast && ctx->d_sort_rank && ctx->host.desc.size() >= 64 && ctx->host.W <= 48 && bytes <= kSmemLimit &&
           nq < (1ll << 24);
}

// Shared by llvq_gemv, llvq_gemv_sg and llvq_gemv_rowshard: exactly one of d_gain_f16 / sg is used.
int gemv_common(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, const SgArgs* sg, int64_t n_out, int64_t k_in,
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
    const size_t kSmemMax = 227 * 1024;
    const size_t rest = 16 + (size_t)nq * 48 * 4 + kGemvGroupsPerPass * kGemvGroupRows * 4 + 16;
    // room for the table of small subsets (not for the 72-bit code: its warps hold 32 unrelated classes that almost never take it together)
    const bool ext_direct = ctx->fast && ctx->fl.total_ext + rest <= kSmemMax;
    const size_t smem = (ext_direct ? ctx->fl.total_ext : ctx->fl.total) + rest;
    if (smem > kSmemMax || n_out > 64ll * kMaxScratchRows) return LLVQ_EUNSUPPORTED;
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
    const SgArgs sga = sg ? *sg : SgArgs{};
    const bool shard = yo.n_peer > 0 || yo.n_flag > 0;                  // row-sharded launch: stored-gain form only
    if (shard && sg) return LLVQ_EUNSUPPORTED;
    // fast-path codes with many classes (mixed warps are what costs there): the kernel that bins the blocks of a segment by
    // class before unranking them; codes with a handful of classes keep the direct kernel
    int seg_units = kBinSegUnits;
    size_t smem_bin; bool ext_bin;
    bin_smem(ctx, nq, seg_units, smem_bin, ext_bin);
    // (smaller segments sort too few blocks to pay for the sort: the direct kernel takes over when 8192 do not fit)
    if (bin_kernel_serves(ctx, nq, sg)) {
        const uint32_t magic = nq == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)nq);
        const FastArgs fa = fast_args(ctx, ext_bin);
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
    const FastArgs fa = fast_args(ctx, ext_direct);
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

// Sorted layout (see the comment at sort_blocks_kernel).  Available for fast-path codes whose indices fit 48 bits
// with 2^48 - 1 left over as the "no block" marker.
bool sortable(const llvq_ctx* ctx, int64_t k_in)
{
    if (!ctx->fast || !ctx->d_sort_rank || ctx->host.W > 48 || ctx->host.N >= (u128)kSortIndexMask) return false;
    const int64_t nq = ((k_in + 23) / 24 + 3) / 4;
    size_t smem; bool ext;
    sorted_smem(ctx, nq, smem, ext);
    return smem <= kSmemLimit && nq < (1ll << 24);
}

}  // namespace

extern "C" {

int llvq_gemv(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_out, int64_t k_in,
              const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;                     // nothing to do: pointers may be null
    if (int e = check_common(ctx, d_idx)) return e;
    if (!d_gain_f16) return LLVQ_EINVAL;
    if (!aligned(d_gain_f16, 2)) return LLVQ_EALIGN;
    return gemv_common(ctx, d_idx, d_gain_f16, nullptr, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

int llvq_gemv_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32, const float* d_row_scale_f32,
                 int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16, void* d_y, int y_dtype, void* stream)
{
    if (ctx && ctx->device >= 0 && n_out == 0) return LLVQ_OK;                     // nothing to do: pointers may be null
    if (int e = check_sg(ctx, d_fields, gain_bits, d_codebook_f32, d_row_scale_f32)) return e;
    const SgArgs sg{d_codebook_f32, d_row_scale_f32, gain_bits};
    return gemv_common(ctx, d_fields, nullptr, &sg, n_out, k_in, d_x_bf16, single_y(d_y), y_dtype, stream);
}

size_t llvq_sorted_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in)
{
    if (ctx && !ctx->fast) return llvq_sorted_gemm_bytes(ctx, n_out, k_in);      // one sorted layout serves both products of these codes
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
    if (ctx && !ctx->fast) return llvq_sort_blocks_gemm(ctx, d_idx, n_out, k_in, d_sorted, stream);
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
    size_t smem; bool ext;
    sorted_smem(ctx, nq, smem, ext);
    const FastArgs fa = fast_args(ctx, ext);
    const uint32_t magic = nq == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)nq);
    const unsigned long long* sp = static_cast<const unsigned long long*>(d_sorted);
    const SgArgs sga = sg ? *sg : SgArgs{};
#define LLVQ_LAUNCH_SORTED(BF16, SG, SH)                                                                                \
    do {                                                                                                                \
        if (!set_smem(gemv_sorted_kernel<BF16, SG, SH>, smem)) return LLVQ_ECUDA;                                        \
        if (launch_pdl(gemv_sorted_kernel<BF16, SG, SH>, g, (unsigned)kSortThreads, smem, st, fa, sp, d_gain_f16, sga, n_out, k_in, bpr, \
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
    if (!ctx->fast) {
        if (!d_x_bf16 || n_out < 0 || k_in <= 0) return LLVQ_EINVAL;
        if (int e = check_yout(single_y(d_y), y_dtype)) return e;
        return llvq_internal_gemv_domains(ctx, d_sorted, d_gain_f16, n_out, k_in, d_x_bf16, d_y, y_dtype, stream);
    }
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

// llvq_gemv_multi / llvq_gemv_sorted_multi: checks, then one launch that walks the matrices.
static int gemv_multi_common(const llvq_ctx* ctx, const llvq_gemv_desc* descs, int n_mats, int y_dtype, bool sorted, void* stream)
{
    if (!ctx || ctx->device < 0 || !descs || n_mats < 1) return LLVQ_EINVAL;
    if (y_dtype != LLVQ_F32 && y_dtype != LLVQ_BF16) return LLVQ_EINVAL;
    if (n_mats > kMaxMultiMats) return LLVQ_EUNSUPPORTED;
    GemvMulti mm{};
    mm.n = n_mats;
    size_t smem = 0; bool ext = true;
    int64_t slot = 0;
    for (int i = 0; i < n_mats; ++i) {
        const llvq_gemv_desc& d = descs[i];
        if (int e = check_common(ctx, d.d_weights)) return e;
        if (!d.d_gain_f16 || !d.d_x_bf16 || !d.d_y || d.n_out <= 0 || d.k_in <= 0) return LLVQ_EINVAL;
        if (!aligned(d.d_gain_f16, 2) || !aligned(d.d_x_bf16, 2) || !aligned(d.d_y, y_dtype == LLVQ_F32 ? 4 : 2)) return LLVQ_EALIGN;
        const int64_t bpr = (d.k_in + 23) / 24, nq = (bpr + 3) / 4;
        const int64_t units = ((d.n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
        // every matrix must give every CTA work: the sorted layout was made for that many CTAs
        if (units < ctx->sm_count) return LLVQ_EUNSUPPORTED;
        size_t bytes; bool e1;
        if (sorted) {
            if (!sortable(ctx, d.k_in)) return LLVQ_EUNSUPPORTED;
            sorted_smem(ctx, nq, bytes, e1);
        } else {
            if (!bin_kernel_serves(ctx, nq, nullptr)) return LLVQ_EUNSUPPORTED;
            bin_smem(ctx, nq, kBinSegUnits, bytes, e1);
        }
        ext = ext && e1;
        smem = std::max(smem, bytes);
        GemvMat& m = mm.m[i];
        m.weights = d.d_weights; m.gain = d.d_gain_f16; m.x = d.d_x_bf16; m.y = d.d_y;
        m.n_out = d.n_out; m.k_in = d.k_in; m.slot0 = slot;
        m.nq_magic = nq == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)nq);
        m.seg_units = kBinSegUnits;
        slot += (d.n_out + kGemvGroupRows - 1) / kGemvGroupRows * kGemvGroupRows;
    }
    if (slot > 64ll * kMaxScratchRows) return LLVQ_EUNSUPPORTED;
    if (!ext) {                                          // one image size for the whole launch: recompute without the extension
        smem = 0;
        for (int i = 0; i < n_mats; ++i) {
            const int64_t nq = ((descs[i].k_in + 23) / 24 + 3) / 4;
            const size_t rest = 16 + (size_t)nq * 48 * 4 + kSortAccCopies * kGemvGroupsPerPass * kGemvGroupRows * 4 + 16 +
                                (sorted ? 0 : 2 * 1024 * 4 + (size_t)kBinSegUnits * 32 * (8 + 2));
            smem = std::max(smem, ctx->fl.total + rest);
        }
    }
    if (smem > kSmemLimit) return LLVQ_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const FastArgs fa = fast_args(ctx, ext);
    const unsigned g = (unsigned)ctx->sm_count;
    if (sorted && n_mats >= 2) {
        // the kernel without a barrier between the matrices, when every CTA's share of every matrix is one segment and
        // one pass and three sets of (x, row sums) fit beside the tables
        int64_t max_groups = 0, max_nq = 0;
        bool one_pass = true;
        for (int i = 0; i < n_mats && one_pass; ++i) {
            const int64_t nq = ((descs[i].k_in + 23) / 24 + 3) / 4;
            const int64_t U = ((descs[i].n_out + kGemvGroupRows - 1) / kGemvGroupRows) * nq;
            max_nq = std::max(max_nq, nq);
            for (int64_t c = 0; c < g; ++c) {
                const int64_t ub = c * U / g, ue = (c + 1) * U / g;
                if (ue - ub > kSortSegUnits) { one_pass = false; break; }
                max_groups = std::max(max_groups, (ue - 1) / nq - ub / nq + 1);
            }
        }
        const int xs_words = (int)(max_nq * 48), acc_rows = (int)(max_groups * kGemvGroupRows);
        const size_t smem_ov = fa.image_bytes + 16 + (size_t)kOverlapSets * ((size_t)xs_words + (size_t)kSortAccCopies * acc_rows) * 4 + kOverlapSets * sizeof(OverlapSet);
        if (one_pass && max_groups <= kGemvGroupsPerPass && smem_ov <= kSmemLimit) {
            if (y_dtype == LLVQ_BF16) {
                if (!set_smem(gemv_sorted_overlap_kernel<true>, smem_ov)) return LLVQ_ECUDA;
                if (launch_pdl(gemv_sorted_overlap_kernel<true>, g, (unsigned)kSortThreads, smem_ov, st, fa, mm, xs_words, acc_rows, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
            } else {
                if (!set_smem(gemv_sorted_overlap_kernel<false>, smem_ov)) return LLVQ_ECUDA;
                if (launch_pdl(gemv_sorted_overlap_kernel<false>, g, (unsigned)kSortThreads, smem_ov, st, fa, mm, xs_words, acc_rows, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
            }
            return launch_status();
        }
    }
    if (sorted) {
        if (y_dtype == LLVQ_BF16) {
            if (!set_smem(gemv_sorted_multi_kernel<true>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemv_sorted_multi_kernel<true>, g, (unsigned)kSortThreads, smem, st, fa, mm, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
        } else {
            if (!set_smem(gemv_sorted_multi_kernel<false>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemv_sorted_multi_kernel<false>, g, (unsigned)kSortThreads, smem, st, fa, mm, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
        }
    } else {
        if (y_dtype == LLVQ_BF16) {
            if (!set_smem(gemv_bin_multi_kernel<true>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemv_bin_multi_kernel<true>, g, (unsigned)kSortThreads, smem, st, fa, ctx->d_sort_rank, mm, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
        } else {
            if (!set_smem(gemv_bin_multi_kernel<false>, smem)) return LLVQ_ECUDA;
            if (launch_pdl(gemv_bin_multi_kernel<false>, g, (unsigned)kSortThreads, smem, st, fa, ctx->d_sort_rank, mm, ctx->d_scratch, ctx->d_counters) != cudaSuccess) return LLVQ_ECUDA;
        }
    }
    return launch_status();
}

int llvq_gemv_multi(const llvq_ctx* ctx, const llvq_gemv_desc* descs, int n_mats, int y_dtype, void* stream)
{
    return gemv_multi_common(ctx, descs, n_mats, y_dtype, false, stream);
}

int llvq_gemv_sorted_multi(const llvq_ctx* ctx, const llvq_gemv_desc* descs, int n_mats, int y_dtype, void* stream)
{
    return gemv_multi_common(ctx, descs, n_mats, y_dtype, true, stream);
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

}  // extern "C"
