// C ABI and kernels of the LLVQ dequantization library (see include/llvq.h).
#include "kernels_common.cuh"

namespace {


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
    // class records in global memory: the full descriptors where the encoder's indexing kernel reads them (codes with their
    // tables in shared memory), the compact 32-byte records for the codes whose decoders read them from global memory
    std::vector<BigDesc> big;
    if (!ctx->fast) {
        if (h.max_levels > kMaxLevels - 1) { delete ctx; return LLVQ_EUNSUPPORTED; }
        build_big_descs(h, big);
    }
    const bool full_descs = ctx->fast || h.W <= 64;      // the encoder's indexing kernel reads them
    const size_t cls_bytes = (full_descs ? ncls * sizeof(ClassDesc) : 0) + 256 + big.size() * sizeof(BigDesc);
    const size_t big_at = ((full_descs ? ncls * sizeof(ClassDesc) : 0) + 255) & ~size_t(255);

    // encoder tables (point -> index), for codes the encoder supports
    std::vector<uint64_t> hkeys; std::vector<uint32_t> hcls;
    std::vector<uint16_t> pos12(4096, 0xffff);
    ctx->can_encode = m_lo == 2 && m_hi >= 3 && h.W <= 64 && build_class_hash(h, hkeys, hcls);
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
    size_t o_lut = up(o_cls + cls_bytes);
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
    if (full_descs) std::memcpy(blob.data() + o_cls, h.desc.data(), ncls * sizeof(ClassDesc));
    if (!big.empty()) std::memcpy(blob.data() + o_cls + big_at, big.data(), big.size() * sizeof(BigDesc));
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
    ctx->dev.cls = full_descs ? reinterpret_cast<const ClassDesc*>(d + o_cls) : nullptr;
    ctx->dev.big = big.empty() ? nullptr : reinterpret_cast<const BigDesc*>(d + o_cls + big_at);
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
    // a warp of these kernels holds 32 unrelated classes: the table of small subsets (FastLayout::sub3) would almost never be taken
    // by all lanes of a step, and asking whether it can be costs more than it returns (measured), so the image goes without it
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    if (ctx->fast) {
        if (!set_smem(decode_blocks_fast_kernel<false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(decode_blocks_fast_kernel<false>, g, (unsigned)kFastThreads, smem, (cudaStream_t)stream, fast_args(ctx, false), idx, nblocks,
                       reinterpret_cast<uint2*>(d_points)) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(decode_blocks_fast_kernel<true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(decode_blocks_fast_kernel<true>, g, (unsigned)kFastThreads, smem, (cudaStream_t)stream, fast_args(ctx, false), idx, nblocks,
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
    // (image without the table of small subsets, as in llvq_decode_blocks)
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    const uint32_t* idx = static_cast<const uint32_t*>(d_idx);
    __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(d_w_bf16);
    if (ctx->fast) {
        if (!set_smem(dequant_fast_kernel<false>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(dequant_fast_kernel<false, false>, g, (unsigned)kFastThreads, smem, st, fast_args(ctx, false), idx, d_gain_f16, SgArgs{}, (uint64_t)nblocks,
                       rows, cols, bpr, w, ld) != cudaSuccess) return LLVQ_ECUDA;
    } else {
        if (!set_smem(dequant_fast_kernel<true>, smem)) return LLVQ_ECUDA;
        if (launch_pdl(dequant_fast_kernel<true, false>, g, (unsigned)kFastThreads, smem, st, fast_args(ctx, false), idx, d_gain_f16, SgArgs{}, (uint64_t)nblocks,
                       rows, cols, bpr, w, ld) != cudaSuccess) return LLVQ_ECUDA;
    }
    return launch_status();
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
    // (image without the table of small subsets, as in llvq_decode_blocks)
    const size_t smem = ctx->fl.total + 16;
    const uint64_t tiles = (nblocks + kFastThreads - 1) / kFastThreads;
    const unsigned g = (unsigned)std::min<uint64_t>(tiles, (uint64_t)ctx->sm_count);
    if (!set_smem(dequant_fast_kernel<false, true>, smem)) return LLVQ_ECUDA;
    dequant_fast_kernel<false, true><<<g, kFastThreads, smem, (cudaStream_t)stream>>>(
        fast_args(ctx, false), static_cast<const uint32_t*>(d_fields), nullptr, SgArgs{d_codebook_f32, d_row_scale_f32, gain_bits},
        nblocks, rows, cols, bpr, reinterpret_cast<__nv_bfloat16*>(d_w_bf16), ld);
    return launch_status();
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
