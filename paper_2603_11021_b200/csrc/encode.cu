// Encoder side of the library: nearest point of the code to a real vector (Sec. 3.1, Euclidean and angular
// scoring), point -> index (Sec. 3.2, the inverse of the dequantizer's steps) and packing of the stored fields.
// The paper defers the search itself to the literature; the search here is coset decoding of the whole lattice
// (exact for the unbounded lattice) plus a policy that keeps the result inside the shells of the code.
#include "llvq.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "ctx.h"
#include "tables.h"

using namespace llvq;

namespace {

constexpr uint32_t kFull = 0xffffffffu;
constexpr int kEncWarps = 8;               // vectors in flight per CTA, one warp each
constexpr uint32_t kFlagSearchGaveUp = 4u; // LLVQ_FLAG_SEARCH_GAVE_UP

constexpr int kMaxCand = 64;               // cosets re-scored in binary64 per search; more (massive ties) means all 8192 are

// Per-warp scratch of the lattice search.
struct WarpTables {
    float2 grp[2][4][64];   // [parity][group of 6 coordinates][bit pattern]: {sum of squared errors, smallest cost of
                            //  moving one coordinate to its other neighbour; its sign bit = parity of the sum of z}
    float e[24][4];         // squared rounding error of coordinate i for offset b = parity + 2 * codeword bit
    float d[24][4];         // cost of moving it to the other neighbour: 1 - 2 |error|
    uint8_t zp[24][4];      // z & 1
    uint32_t cand[kMaxCand];
    uint32_t ncand;
};

// sum of the values of lanes 0..23, added in lane order, one binary64 rounding per addition (every lane gets the sum)
__device__ __forceinline__ double seq_sum24(double v)
{
    double acc = 0.0;
#pragma unroll
    for (int i = 0; i < 24; ++i) acc = __dadd_rn(acc, __shfl_sync(kFull, v, i));
    return acc;
}

// Cost of coset (pi, codeword j) from the group tables, in units of 16 (binary32).
__device__ __forceinline__ float coset_cost(const WarpTables& W, uint32_t c, uint32_t pi)
{
    const float2 a0 = W.grp[pi][0][c & 63u], a1 = W.grp[pi][1][(c >> 6) & 63u], a2 = W.grp[pi][2][(c >> 12) & 63u], a3 = W.grp[pi][3][c >> 18];
    float cost = (a0.x + a1.x) + (a2.x + a3.x);
    const uint32_t par = (__float_as_uint(a0.y) ^ __float_as_uint(a1.y) ^ __float_as_uint(a2.y) ^ __float_as_uint(a3.y)) >> 31;
    if (par != pi) cost += fminf(fminf(fabsf(a0.y), fabsf(a1.y)), fminf(fabsf(a2.y), fabsf(a3.y)));
    return cost;
}

// Nearest point of the unbounded lattice to u (one coordinate per lane, lanes 0..23; all in units of the integer
// coordinates).  Every lattice point is b + 4 z with b_i = parity + 2 c_i, c a Golay codeword, and sum z = parity
// (mod 2) (the sum rules of Sec. 2.4: all Golay weights are multiples of 4).  For each of the 2 x 4096 cosets the
// best z is the rounded one, with the coordinate of largest rounding error moved to its other neighbour when the
// sum rule fails.
// Two stages.  A binary32 scan of all cosets through tables per group of 6 coordinates (4 reads and about 20
// instructions per coset) finds the smallest cost; every coset whose binary32 cost is within 2^-12 (+ 2^-13 of the
// cost) of it -- far more than the binary32 scan can err, costs are at most 1 -- is then evaluated again in binary64,
// coordinate by coordinate in lane order, one rounding per operation: its point, and the squared distance as the sum
// over the coordinates in order.  The smallest distance wins, the lowest (parity, codeword position) among equal ones;
// inside a coset the first coordinate with the largest error moves.  The result does not depend on the first stage's
// rounding.  Returns the coordinate of this lane (0 for lanes >= 24) and the squared norm of the point.
__device__ int lattice_nearest(WarpTables& W, const uint32_t* __restrict__ golay_s, double u, int lane, int& norm2)
{
    const float uf = (float)u;
    if (lane < 24) {
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const float t = (uf - (float)b) * 0.25f;
            const float z = rintf(t);
            const float err = t - z;
            W.e[lane][b] = err * err;
            W.d[lane][b] = 1.f - 2.f * fabsf(err);
            W.zp[lane][b] = (uint8_t)((int)z & 1);
        }
    }
    if (lane == 0) W.ncand = 0u;
    __syncwarp();
    for (int q = 0; q < 16; ++q) {
        const int id = q * 32 + lane, pi = id >> 8, g = (id >> 6) & 3, pat = id & 63;
        float cost = 0.f, delta = 2.f;
        uint32_t par = 0;
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            const int b = pi + 2 * ((pat >> k) & 1), i = 6 * g + k;
            cost += W.e[i][b];
            delta = fminf(delta, W.d[i][b]);
            par ^= W.zp[i][b];
        }
        W.grp[pi][g][pat] = make_float2(cost, __uint_as_float(__float_as_uint(delta) | par << 31));
    }
    __syncwarp();
    float best = 3.0e38f;
    for (int s = 0; s < 128; ++s) {
        const uint32_t c = golay_s[s * 32 + lane];
        best = fminf(best, fminf(coset_cost(W, c, 0u), coset_cost(W, c, 1u)));
    }
    const float mine_best = best;                       // over this lane's 256 codewords
#pragma unroll
    for (int o = 16; o; o >>= 1) best = fminf(best, __shfl_xor_sync(kFull, best, o));
    const float thr = best + (1.f / 4096.f + best * (1.f / 8192.f));
    // only the lanes whose own minimum is within the margin can hold candidates (usually one lane): the warp goes through
    // the 256 codewords of each such lane together, 8 per lane
    for (uint32_t holders = __ballot_sync(kFull, mine_best <= thr); holders; holders &= holders - 1u) {
        const uint32_t owner = (uint32_t)__ffs(holders) - 1u;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t j = (uint32_t)((q * 32 + lane) * 32) + owner, c = golay_s[j];
#pragma unroll
            for (uint32_t pi = 0; pi < 2; ++pi) {
                if (coset_cost(W, c, pi) <= thr) {
                    const uint32_t slot = atomicAdd(&W.ncand, 1u);
                    if (slot < (uint32_t)kMaxCand) W.cand[slot] = pi << 12 | j;
                }
            }
        }
    }
    __syncwarp();
    const uint32_t listed = W.ncand;
    const uint32_t n = listed > (uint32_t)kMaxCand ? 8192u : listed;          // too many near-ties to list: every coset
    const bool mine = lane < 24;
    double best_d2 = 1.0e300;
    uint32_t best_id = 0xffffffffu;
    int best_x = 0;
    for (uint32_t t = 0; t < n; ++t) {
        const uint32_t id = listed > (uint32_t)kMaxCand ? t : W.cand[t];
        const int pi = (int)(id >> 12);
        const uint32_t c = golay_s[id & 4095u];
        const int b = pi + 2 * (int)((c >> (lane & 31)) & 1u);
        const double tt = __dmul_rn(__dsub_rn(u, (double)b), 0.25);
        const double z = rint(tt);
        const double err = __dsub_rn(tt, z);
        int x = mine ? b + 4 * (int)z : 0;
        const int sum = __reduce_add_sync(kFull, x);
        if ((((sum % 8) + 8) % 8) != (pi ? 4 : 0)) {
            // the first coordinate with the largest |error| moves by 4 (binary64 magnitudes compare like their bit patterns)
            unsigned long long key = mine ? (unsigned long long)__double_as_longlong(fabs(err)) : 0ull;
            int who = lane;
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                const unsigned long long ok = __shfl_xor_sync(kFull, key, o);
                const int ow = __shfl_xor_sync(kFull, who, o);
                if (ok > key || (ok == key && ow < who)) { key = ok; who = ow; }
            }
            if (lane == who) x += err > 0.0 ? 4 : (err < 0.0 ? -4 : 4);
        }
        const double dd = __dsub_rn(u, (double)x);
        const double d2 = seq_sum24(mine ? __dmul_rn(dd, dd) : 0.0);
        if (d2 < best_d2 || (d2 == best_d2 && id < best_id)) { best_d2 = d2; best_id = id; best_x = x; }
    }
    norm2 = __reduce_add_sync(kFull, best_x * best_x);
    __syncwarp();
    return best_x;
}

// One warp per input vector; inputs are binary32 values, all scoring runs in binary64 with one rounding per operation and
// sums over the coordinates in order.  EUCLIDEAN: if the nearest lattice point of the input lies in the code it is the
// answer (it is then also the nearest point of the cut, App. E "Spherical shaping").  Otherwise, and for ANGULAR always,
// the input direction is decoded at every shell radius sqrt(16 m); of the candidates inside the code the one nearest to
// the input (EUCLIDEAN) or with the largest cosine (ANGULAR) wins, the first radius on ties.  A zero input gives the
// point of index 0, (4, 4, 0^22), the first point of the first class of Shell(2) (Sec. 2.3).  Needs m_lo == 2 and
// m_hi >= 3 (checked on the host).
__global__ void __launch_bounds__(kEncWarps * 32)
encode_search_kernel(const uint32_t* __restrict__ golay, const float* __restrict__ v, uint64_t n, int metric, int m_lo, int m_hi,
                     int8_t* __restrict__ points, uint32_t* __restrict__ flags)
{
    extern __shared__ __align__(16) uint8_t enc_smem[];
    uint32_t* golay_s = reinterpret_cast<uint32_t*>(enc_smem);
    WarpTables* tabs = reinterpret_cast<WarpTables*>(enc_smem + 4096 * 4);
    for (int i = threadIdx.x; i < 4096; i += blockDim.x) golay_s[i] = __ldg(golay + i);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WarpTables& W = tabs[warp];
    for (uint64_t vec = (uint64_t)blockIdx.x * kEncWarps + warp; vec < n; vec += (uint64_t)gridDim.x * kEncWarps) {
        const double vi = lane < 24 ? (double)__ldg(v + vec * 24 + lane) : 0.0;
        const double n2 = seq_sum24(__dmul_rn(vi, vi));
        int bestx = lane == 0 || lane == 1 ? 4 : 0;              // the point of index 0
        bool ok = false, direct = false;
        const bool finite = n2 < 1.0e300;                        // false for NaN too
        if (n2 == 0.0) {
            ok = direct = true;
        } else if (finite && metric == LLVQ_EUCLIDEAN) {
            // no lattice point is farther than 4 from any input (covering radius): beyond radius sqrt(16 m_hi) + 4 the nearest
            // point is certainly outside the code and the decode can be skipped
            const double reach = sqrt(16.0 * (double)m_hi) + 4.01;
            if (n2 <= reach * reach) {
                int norm2;
                const int x = lattice_nearest(W, golay_s, vi, lane, norm2);
                const int m = norm2 / 16;
                if (m >= m_lo && m <= m_hi) { ok = direct = true; bestx = x; }
            }
        }
        if (finite && !direct) {
            const double rn = __ddiv_rn(1.0, __dsqrt_rn(n2));
            double best = -1.0e300;
            bool first = true;
            for (int m = m_lo; m <= m_hi; ++m) {
                const double rad = __dsqrt_rn(__dmul_rn(16.0, (double)m));
                int norm2;
                const int x = lattice_nearest(W, golay_s, __dmul_rn(__dmul_rn(vi, rn), rad), lane, norm2);
                const int mx = norm2 / 16;
                if (mx < m_lo || mx > m_hi) continue;
                double score;
                if (metric == LLVQ_EUCLIDEAN) {
                    const double dd = __dsub_rn(vi, (double)x);
                    score = -seq_sum24(lane < 24 ? __dmul_rn(dd, dd) : 0.0);
                } else {
                    const double dot = seq_sum24(lane < 24 ? __dmul_rn(__dmul_rn(vi, rn), (double)x) : 0.0);
                    score = __ddiv_rn(dot, __dsqrt_rn((double)norm2));
                }
                if (first || score > best) { best = score; bestx = x; ok = true; first = false; }
            }
        }
        if (!ok) {
            bestx = lane == 0 || lane == 1 ? 4 : 0;
            if (lane == 0) atomicOr(flags, kFlagSearchGaveUp);
        }
        if (lane < 24) points[vec * 24 + lane] = (int8_t)bestx;
    }
}

// Bits of a at the set positions of mask, packed lowest first.
__device__ __forceinline__ uint32_t extract_bits(uint32_t a, uint32_t mask)
{
    uint32_t r = 0, k = 0;
    while (mask) {
        const uint32_t low = mask & (0u - mask);
        if (a & low) r |= 1u << k;
        ++k;
        mask ^= low;
    }
    return r;
}

// Point -> index (Sec. 3.2; inverse of App. A steps 1-4), one thread per block.  A point that is not in the code
// gets index 0 and is counted in the out-of-range counter.
__global__ void __launch_bounds__(256)
rank_kernel(DevCode dc, EncTables et, const uint32_t* __restrict__ golay, const uint32_t* __restrict__ pascal,
            const int8_t* __restrict__ points, uint64_t n, unsigned long long* __restrict__ index)
{
    const uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= n) return;
    int a[24];
    uint32_t c = 0, neg = 0, nonzero = 0, bit1 = 0;
    uint64_t sig = 0;
    const int parity = points[b * 24] & 1;
    bool good = true;
#pragma unroll
    for (int i = 0; i < 24; ++i) {
        const int xi = points[b * 24 + i];
        a[i] = xi < 0 ? -xi : xi;
        good &= (xi & 1) == parity && a[i] < 64;
        sig += __ldg(et.sig_of_value + (a[i] & 63));
        c |= (uint32_t)(((xi - parity) >> 1) & 1) << i;
        neg |= (uint32_t)(xi < 0) << i;
        nonzero |= (uint32_t)(xi != 0) << i;
        bit1 |= (uint32_t)((a[i] >> 1) & 1) << i;
    }
    // class of the multiset of absolute values
    uint32_t cls = 0;
    bool found = false;
    uint32_t slot = (uint32_t)(sig >> 20) & et.hash_mask;
    for (uint32_t probe = 0; probe <= et.hash_mask; ++probe) {
        const uint64_t key = __ldg(et.hash_key + slot);
        if (key == sig) { cls = __ldg(et.hash_cls + slot); found = true; break; }
        if (key == 0) break;
        slot = (slot + 1) & et.hash_mask;
    }
    good &= found;
    unsigned long long I = 0;
    if (good) {
        const ClassDesc& d = dc.cls[cls];
        const uint32_t pos = __ldg(et.pos_by_low12 + (c & 0xfffu));
        good &= __ldg(golay + pos) == c;                                   // c must be a codeword
        const uint32_t r = pos - d.goff;
        good &= r < d.A;                                                   // ... of the weight the class needs
        const uint32_t F1 = parity ? 0u : c, F0 = ~F1 & 0xffffffu;
        uint32_t freem = parity ? 0xffffffu : F1;
        bool in0 = parity != 0;
        unsigned long long p = 0, mult = 1;
        const int nlev = d.nlev1 + d.nlev0;
        for (int l = 0; l < nlev; ++l) {
            if (!in0 && l >= d.nlev1) {                                    // the rest of group 1 holds its filler
                for (int i = 0; i < 24; ++i) if ((freem >> i) & 1u) good &= a[i] == d.fill1;
                freem = F0; in0 = true;
            }
            const LevelDesc& lv = d.lev[l];
            uint32_t am = 0;
            for (int i = 0; i < 24; ++i) am |= (uint32_t)(a[i] == lv.val) << i;
            am &= freem;
            good &= __popc(am) == lv.k;
            uint32_t rel = extract_bits(am, freem), rho = 0;
            for (int t = 1; rel; ++t) {                                    // combinatorial number system: sum of C(e_t, t)
                const int e = __ffs(rel) - 1;
                rho += __ldg(pascal + e * 25 + min(t, 24));
                rel &= rel - 1;
            }
            p += mult * rho;
            mult *= lv.radix;
            freem ^= am;
        }
        if (!in0) {
            for (int i = 0; i < 24; ++i) if ((freem >> i) & 1u) good &= a[i] == d.fill1;
            freem = F0;
        }
        for (int i = 0; i < 24; ++i) if ((freem >> i) & 1u) good &= a[i] == d.fill0;
        unsigned long long s = 0;
        if (parity) {
            good &= neg == (c ^ bit1);                                     // 1 mod 4 on F0, 3 mod 4 on F1
        } else {
            // s = the signs of the positions that carry one (F1 and the nonzero ones of F0), ascending, without the last F1
            // position, whose sign the others fix (sum = 0 mod 8)
            const uint32_t last_f1 = F1 ? 0x80000000u >> __clz(F1) : 0u;
            if (d.w) good &= ((neg & last_f1) != 0u) == (((__popc(neg & F1 & ~last_f1) + d.signpar) & 1u) != 0u);
            s = extract_bits(neg, (F1 | (F0 & nonzero)) & ~last_f1);
        }
        I = dc.off_lo[cls] + r + (unsigned long long)d.A * (s + (p << d.B));
    }
    if (!good) { I = 0; atomicAdd(dc.bad_index, 1ull); }
    index[b] = I;
}

// One thread per 32-bit word of the stored stream: gathers the fields that overlap it.
__global__ void __launch_bounds__(256)
pack_kernel(const unsigned long long* __restrict__ index, const uint8_t* __restrict__ gain_index, int W, int gain_bits,
            uint64_t n, uint32_t* __restrict__ out, uint64_t nwords)
{
    const uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= nwords) return;
    const uint64_t bit0 = w * 32, wt = (uint64_t)(W + gain_bits);
    const unsigned long long keep = wt < 64 ? (1ull << wt) - 1ull : ~0ull;
    uint32_t acc = 0;
    for (uint64_t f = bit0 / wt; f < n && f * wt < bit0 + 32; ++f) {
        unsigned long long field = index[f];
        if (gain_index) field |= (unsigned long long)gain_index[f] << W;
        field &= keep;
        const uint64_t start = f * wt;
        acc |= start >= bit0 ? (uint32_t)(field << (start - bit0)) : (uint32_t)(field >> (bit0 - start));
    }
    out[w] = acc;
}

int status_of_launch() { return cudaGetLastError() == cudaSuccess ? LLVQ_OK : LLVQ_ECUDA; }

int launch_rank(const llvq_ctx* ctx, const int8_t* d_points, uint64_t nblocks, uint64_t* d_index, cudaStream_t st)
{
    const uint32_t* pascal = reinterpret_cast<const uint32_t*>(ctx->d_image + ctx->fl.pascal);
    const unsigned grid = (unsigned)((nblocks + 255) / 256);
    rank_kernel<<<grid, 256, 0, st>>>(ctx->dev, ctx->enc, ctx->d_golay, pascal, d_points, nblocks,
                                      reinterpret_cast<unsigned long long*>(d_index));
    return status_of_launch();
}

int check_encoder(const llvq_ctx* ctx, uint64_t nblocks)
{
    if (!ctx || ctx->device < 0) return LLVQ_EINVAL;
    if (!ctx->can_encode || nblocks > (1ull << 31) * 256ull) return LLVQ_EUNSUPPORTED;
    return LLVQ_OK;
}

}  // namespace

extern "C" {

int llvq_encode_blocks(const llvq_ctx* ctx, const float* d_v_f32, uint64_t nblocks, int metric,
                       int8_t* d_points, uint64_t* d_index, void* stream)
{
    if (ctx && ctx->device >= 0 && nblocks == 0) return LLVQ_OK;
    if (int e = check_encoder(ctx, nblocks)) return e;
    if (!d_v_f32 || !d_points || !d_index || (metric != LLVQ_EUCLIDEAN && metric != LLVQ_ANGULAR)) return LLVQ_EINVAL;
    if (!aligned(d_v_f32, 4) || !aligned(d_index, 8)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = 4096 * 4 + kEncWarps * sizeof(WarpTables);
    if (cudaFuncSetAttribute(encode_search_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return LLVQ_ECUDA;
    const uint64_t ctas = (nblocks + kEncWarps - 1) / kEncWarps;
    const unsigned grid = (unsigned)std::min<uint64_t>(ctas, (uint64_t)ctx->sm_count * 4);
    encode_search_kernel<<<grid, kEncWarps * 32, smem, st>>>(ctx->d_golay, d_v_f32, nblocks, metric, ctx->host.m_lo, ctx->host.m_hi,
                                                            d_points, ctx->dev.flags);
    if (int e = status_of_launch()) return e;
    return launch_rank(ctx, d_points, nblocks, d_index, st);
}

int llvq_rank_blocks(const llvq_ctx* ctx, const int8_t* d_points, uint64_t nblocks, uint64_t* d_index, void* stream)
{
    if (ctx && ctx->device >= 0 && nblocks == 0) return LLVQ_OK;
    if (int e = check_encoder(ctx, nblocks)) return e;
    if (!d_points || !d_index) return LLVQ_EINVAL;
    if (!aligned(d_index, 8)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    return launch_rank(ctx, d_points, nblocks, d_index, (cudaStream_t)stream);
}

int llvq_pack_fields(const llvq_ctx* ctx, const uint64_t* d_index, const uint8_t* d_gain_index, int gain_bits,
                     uint64_t nblocks, void* d_fields, void* stream)
{
    if (!ctx || ctx->device < 0 || gain_bits < 0 || gain_bits > 8) return LLVQ_EINVAL;
    if (ctx->host.W + gain_bits > 64) return LLVQ_EUNSUPPORTED;
    if (nblocks == 0) return LLVQ_OK;
    if (!d_index || !d_fields || (gain_bits > 0 && !d_gain_index)) return LLVQ_EINVAL;
    if (!aligned(d_index, 8) || !aligned(d_fields, 16)) return LLVQ_EALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return LLVQ_ECUDA;
    const uint64_t nwords = llvq_field_bytes(ctx, nblocks, gain_bits) / 4;
    if (nwords > (1ull << 31) * 256ull) return LLVQ_EUNSUPPORTED;
    pack_kernel<<<(unsigned)((nwords + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const unsigned long long*>(d_index), gain_bits ? d_gain_index : nullptr, ctx->host.W, gain_bits, nblocks,
        static_cast<uint32_t*>(d_fields), nwords);
    return status_of_launch();
}

}  // extern "C"
