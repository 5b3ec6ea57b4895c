// Host-side table generator (see tables.h).
#include "tables.h"

#include <algorithm>
#include <array>
#include <cmath>
#include <cstring>

namespace llvq {
namespace {

inline int popc(uint32_t v) { return __builtin_popcount(v); }

// Extended Golay code (Sec. 2.3).  Basis: the 12 shifts of the generator
// polynomial x^11+x^10+x^6+x^5+x^4+x^2+1 of the cyclic [23,12,7] code, each
// extended by an overall parity bit at coordinate 23; all 4096 sums are walked
// in Gray-code order.
void make_golay(HostTables& t)
{
    uint32_t basis[12];
    for (int i = 0; i < 12; ++i) {
        uint32_t row = 0xC75u << i;
        if (popc(row) & 1) row |= 1u << 23;
        basis[i] = row;
    }
    t.golay.resize(4096);
    uint32_t word = 0;
    t.golay[0] = 0;
    for (uint32_t g = 1; g < 4096; ++g) {
        word ^= basis[__builtin_ctz(g)];     // Gray code: flip one basis vector per step
        t.golay[g] = word;
    }
    std::sort(t.golay.begin(), t.golay.end(), [](uint32_t a, uint32_t b) {
        int wa = popc(a), wb = popc(b);
        return wa != wb ? wa < wb : a < b;
    });
    for (uint32_t c : t.golay) t.wcnt[popc(c)]++;
    int acc = 0;
    for (int w = 0; w <= 24; ++w) { t.woff[w] = acc; acc += t.wcnt[w]; }
}

void make_pascal(HostTables& t)
{
    for (int n = 0; n < 25; ++n) {
        t.pascal[n * 25] = 1;
        for (int k = 1; k <= n; ++k)
            t.pascal[n * 25 + k] = (n ? t.pascal[(n - 1) * 25 + k - 1] : 0) + (k <= n - 1 ? t.pascal[(n - 1) * 25 + k] : 0);
    }
}

struct Multiset {
    int parity;
    std::array<int, 32> cnt;     // cnt[v] = multiplicity of absolute value v
};

// All multisets of 24 values of one parity with squared norm `norm`,
// generated from the smallest value upwards.
void gen_multisets(int parity, int v, int left, int norm, Multiset& cur, std::vector<Multiset>& out)
{
    if (left == 0) { if (norm == 0) out.push_back(cur); return; }
    if (v * v * left > norm && v > 0) return;      // even the smallest remaining value overshoots
    if (v > 31 || v * v > norm) return;
    int maxc = v == 0 ? left : std::min(left, norm / (v * v));
    for (int c = maxc; c >= 0; --c) {
        cur.cnt[v] = c;
        gen_multisets(parity, v + 2, left - c, norm - c * v * v, cur, out);
    }
    cur.cnt[v] = 0;
}

u128 choose(const HostTables& t, int n, int k) { return (k < 0 || k > n) ? 0 : (u128)t.pascal[n * 25 + k]; }

bool admissible(const Multiset& s, int& w)
{
    int n2 = 0, n4 = 0, n35 = 0;
    for (int v = 0; v < 32; ++v) {
        if (v % 4 == 2) n2 += s.cnt[v];
        if (v % 8 == 4) n4 += s.cnt[v];
        if (v % 8 == 3 || v % 8 == 5) n35 += s.cnt[v];
    }
    if (s.parity) { w = 0; return (n35 % 2) == 1; }            // coordinate sum = 4 mod 8
    w = n2;
    if (!(w == 0 || w == 8 || w == 12 || w == 16 || w == 24)) return false;
    return w != 0 || n4 % 2 == 0;                              // coordinate sum = 0 mod 8
}

std::array<int, 24> leader(const ClassInfo& c)
{
    std::array<int, 24> l{};
    int p = 0;
    for (size_t i = 0; i < c.values.size(); ++i)
        for (int j = 0; j < c.mults[i]; ++j) l[p++] = c.values[i];
    return l;
}

// Fixed class order inside a shell (Sec. 3.2 (2)): even classes by ascending
// Golay weight then ascending leader; then odd classes by descending leader.
bool class_before(const ClassInfo& a, const ClassInfo& b)
{
    if (a.parity != b.parity) return a.parity < b.parity;
    auto la = leader(a), lb = leader(b);
    if (a.parity == 0) {
        if (a.w != b.w) return a.w < b.w;
        return la < lb;
    }
    return la > lb;
}

bool fill_descriptor(const HostTables& t, const ClassInfo& c, ClassDesc& d, int& nlev)
{
    std::memset(&d, 0, sizeof d);
    d.parity = (uint8_t)c.parity; d.w = (uint8_t)c.w; d.B = (uint8_t)c.B; d.m = (uint32_t)c.m;
    d.A = (uint16_t)c.A;
    d.goff = (uint16_t)(c.parity ? 0 : t.woff[c.w]);
    d.magicA = ~0ull / c.A;
    int n46 = 0;
    for (size_t i = 0; i < c.values.size(); ++i)
        if (c.values[i] % 8 == 4 || c.values[i] % 8 == 6) n46 += c.mults[i];
    d.signpar = (uint8_t)(n46 & 1);
    nlev = 0;
    for (int group = 1; group >= 0; --group) {
        std::vector<int> gv, gm;
        for (size_t i = 0; i < c.values.size(); ++i) {
            bool in1 = !c.parity && c.values[i] % 4 == 2;
            if ((group == 1) == in1) { gv.push_back(c.values[i]); gm.push_back(c.mults[i]); }
        }
        int n = group == 1 ? c.w : 24 - c.w;
        if (c.parity) n = group == 1 ? 0 : 24;
        int steps = 0;
        for (size_t i = 0; i + 1 < gv.size(); ++i) {
            if (nlev >= kMaxLevels) return false;
            LevelDesc& l = d.lev[nlev++];
            l.radix = t.pascal[n * 25 + gm[i]];
            l.k = (uint8_t)gm[i]; l.val = (uint8_t)gv[i]; l.n = (uint8_t)n; l.pad = 0;
            l.magic = ~0ull / l.radix;
            n -= gm[i];
            ++steps;
        }
        uint8_t fill = gv.empty() ? 0 : (uint8_t)gv.back();
        if (group == 1) { d.nlev1 = (uint8_t)steps; d.fill1 = fill; }
        else            { d.nlev0 = (uint8_t)steps; d.fill0 = fill; }
    }
    return true;
}

}  // namespace

bool build_tables(int m_lo, int m_hi, HostTables& t)
{
    if (m_lo < 2 || m_hi < m_lo || m_hi > 53) return false;
    t = HostTables();
    t.m_lo = m_lo; t.m_hi = m_hi;
    make_golay(t);
    make_pascal(t);
    u128 running = 0;
    for (int m = m_lo; m <= m_hi; ++m) {
        std::vector<ClassInfo> shell;
        for (int parity = 0; parity <= 1; ++parity) {
            std::vector<Multiset> sets;
            Multiset cur; cur.parity = parity; cur.cnt.fill(0);
            gen_multisets(parity, parity, 24, 16 * m, cur, sets);
            for (const Multiset& s : sets) {
                int w;
                if (!admissible(s, w)) continue;
                ClassInfo c;
                c.m = m; c.parity = parity; c.w = w;
                for (int v = 31; v >= 0; --v)
                    if (s.cnt[v]) { c.values.push_back(v); c.mults.push_back(s.cnt[v]); }
                // cardinality A * 2^B * P (Sec. 2.5)
                u128 P = 1;
                if (parity) {
                    c.A = 4096; c.B = 0;
                    int left = 24;
                    for (int k : c.mults) { P *= choose(t, left, k); left -= k; }
                } else {
                    c.A = (uint64_t)t.wcnt[w];
                    int left1 = w, left0 = 24 - w, nz0 = 0;
                    for (size_t i = 0; i < c.values.size(); ++i) {
                        if (c.values[i] % 4 == 2) { P *= choose(t, left1, c.mults[i]); left1 -= c.mults[i]; }
                        else { P *= choose(t, left0, c.mults[i]); left0 -= c.mults[i]; if (c.values[i]) nz0 += c.mults[i]; }
                    }
                    c.B = nz0 + (w > 0 ? w - 1 : 0);
                }
                c.card = (u128)c.A * ((u128)1 << c.B) * P;
                c.offset = 0;
                shell.push_back(c);
            }
        }
        std::sort(shell.begin(), shell.end(), class_before);
        for (ClassInfo& c : shell) { c.offset = running; running += c.card; t.info.push_back(c); }
    }
    t.N = running;
    t.W = 0;
    while (t.W < 100 && ((u128)1 << t.W) < t.N) ++t.W;
    if (t.W > 72) return false;
    t.desc.resize(t.info.size());
    t.offset.resize(t.info.size() + 1);
    for (size_t j = 0; j < t.info.size(); ++j) {
        int nlev;
        if (!fill_descriptor(t, t.info[j], t.desc[j], nlev)) return false;
        if (t.info[j].card >> 63) return false;          // class-local indices must fit 63 bits
        t.max_levels = std::max(t.max_levels, nlev);
        t.offset[j] = t.info[j].offset;
    }
    t.offset[t.info.size()] = t.N;
    return true;
}

}  // namespace llvq

namespace llvq {

bool build_fast_image(const HostTables& t, FastLayout& L, std::vector<uint8_t>& img, bool with_classes)
{
    const size_t ncls = with_classes ? t.desc.size() : 0;
    if (with_classes && (t.W > 64 || t.W < 12 || ncls > 1024 || t.max_levels > kFastMaxLevels)) return false;
    auto up16 = [](size_t v) { return (uint32_t)((v + 15) & ~size_t(15)); };
    // r14: all k-subsets of 14 slots, grouped by k, each group in numeric order
    std::vector<uint16_t> r14;
    uint32_t base14[16] = {0};
    for (int k = 0; k <= kLowBits; ++k) {
        base14[k] = (uint32_t)r14.size();
        for (uint32_t m = 0; m < (1u << kLowBits); ++m)
            if (__builtin_popcount(m) == k) r14.push_back((uint16_t)m);
    }
    L.golay = 0;
    L.lut = up16(L.golay + 4096 * 4);
    L.pascal = up16(L.lut + (with_classes ? 4096 * 2 : 0));
    L.base14 = up16(L.pascal + 625 * 4);
    if (L.base14 - L.pascal != 2512) return false;                      // the kernels address base14 relative to pascal
    L.r14 = up16(L.base14 + 16 * 4);
    L.pd6 = up16(L.r14 + r14.size() * 2);
    L.off = up16(L.pd6 + 4096);
    L.desc = up16(L.off + (with_classes ? (ncls + 1) * 8 : 0));
    L.recip64 = L.recip32 = 0;
    size_t end = L.desc + ncls * kFastDescStride * 4;
    if (!with_classes) {                                   // the class-independent reciprocals the compact class records rely on
        L.recip64 = up16(end);
        L.recip32 = up16(L.recip64 + 625 * 8);
        end = L.recip32 + 625 * 4;
    }
    L.total = up16(end);
    L.sub3 = L.total;
    L.total_ext = up16(L.sub3 + kSmallSubsetWords * 4);
    L.lut_shift = (uint32_t)(t.W >= 12 ? t.W - 12 : 0);
    L.ncls = (uint32_t)ncls;
    L.W = (uint32_t)t.W;
    img.assign(L.total_ext, 0);
    {
        // all k-subsets of 24 slots for k <= 3, each group in numeric order (= the order of their combinatorial-number-system
        // ranks, whatever the number of slots in use), behind a four-word directory
        uint32_t* sub = reinterpret_cast<uint32_t*>(img.data() + L.sub3);
        uint32_t at = 4;
        for (int k = 0; k <= kSmallSubsetMaxK; ++k) {
            sub[k] = at;
            for (uint32_t m = 0; m < (1u << kDim); ++m)
                if (__builtin_popcount(m) == k) sub[at++] = m;
        }
        if (at != (uint32_t)kSmallSubsetWords) return false;
    }
    std::memcpy(img.data() + L.golay, t.golay.data(), 4096 * 4);
    std::memcpy(img.data() + L.pascal, t.pascal, 625 * 4);
    for (int n = 0; n < 25; ++n)                           // column 0 is a sentinel in the image: "no element left to place"
        reinterpret_cast<uint32_t*>(img.data() + L.pascal)[n * 25] = 0xffffffffu;
    std::memcpy(img.data() + L.base14, base14, sizeof base14);
    std::memcpy(img.data() + L.r14, r14.data(), r14.size() * 2);
    // pd6
    for (uint32_t f = 0; f < 64; ++f)
        for (uint32_t s = 0; s < 64; ++s) {
            uint32_t out = 0, src = s;
            for (int b = 0; b < 6; ++b)
                if ((f >> b) & 1u) { if (src & 1u) out |= 1u << b; src >>= 1; }
            img[L.pd6 + (f << 6 | s)] = (uint8_t)out;
        }
    if (!with_classes) {                                   // small tables only: the class tables stay in global memory
        uint64_t* r64 = reinterpret_cast<uint64_t*>(img.data() + L.recip64);
        uint32_t* r32 = reinterpret_cast<uint32_t*>(img.data() + L.recip32);
        for (int i = 0; i < 625; ++i) {
            const uint32_t c = t.pascal[i];
            r64[i] = c ? ~0ull / c : 0ull;
            r32[i] = c > 1 ? (uint32_t)((1ull << 32) / c) : 0xffffffffu;
        }
        return true;
    }
    // class lookup by the top 12 bits of the index
    uint16_t* lut = reinterpret_cast<uint16_t*>(img.data() + L.lut);
    size_t c = 0;
    for (uint32_t b = 0; b < 4096; ++b) {
        u128 first = (u128)b << L.lut_shift;
        while (c + 1 < ncls && t.offset[c + 1] <= first) ++c;
        lut[b] = (uint16_t)c;
    }
    uint64_t* off = reinterpret_cast<uint64_t*>(img.data() + L.off);
    for (size_t j = 0; j <= ncls; ++j) off[j] = (uint64_t)t.offset[j];
    uint32_t* dw = reinterpret_cast<uint32_t*>(img.data() + L.desc);
    for (size_t j = 0; j < ncls; ++j) {
        const ClassDesc& d = t.desc[j];
        uint32_t* w = dw + j * kFastDescStride;
        const int nlev = d.nlev1 + d.nlev0;
        if (nlev > kFastMaxLevels || nlev + 2 > 8) return false;
        uint32_t flags = (d.parity ? 1u : 0u) | (d.signpar ? 2u : 0u) | (d.fill0 ? 4u : 0u) |
                         ((d.fill1 & 2) ? 8u : 0u) | ((d.fill0 & 2) ? 16u : 0u);
        if (!((t.info[j].card / ((u128)d.A << d.B)) >> 32)) flags |= kFastFlagRank32;
        // decoder form of the class (bits 6-7): 0 even with Golay weight 8, 12 or 16, 1 odd, 2 any other
        flags |= (d.parity ? 1u : ((d.w == 8 || d.w == 12 || d.w == 16) ? 0u : 2u)) << 6;
        w[0] = d.w | (uint32_t)d.B << 8 | flags << 16 | (uint32_t)d.nlev1 << 24 | (uint32_t)nlev << 28;
        w[1] = d.goff | (uint32_t)d.A << 16;
        w[2] = (uint32_t)d.magicA; w[3] = (uint32_t)(d.magicA >> 32);
        uint8_t vals[8] = {d.fill0, d.fill1, 0, 0, 0, 0, 0, 0};
        uint32_t nbytes = 0;
        u128 p_after = t.info[j].card / ((u128)d.A << d.B);        // number of arrangements P
        for (int l = 0; l < nlev; ++l) {
            const LevelDesc& lv = d.lev[l];
            if (lv.radix >= (1u << 22)) return false;
            vals[2 + l] = lv.val;
            w[8 + l] = lv.radix | (uint32_t)lv.k << 22 | (uint32_t)(2 + l) << 27 | ((lv.val & 2) ? 1u << 30 : 0u) | (lv.val ? 1u << 31 : 0u);
            nbytes |= (uint32_t)lv.n << (8 * l);
            if (l == 0) {
                w[6] = (uint32_t)lv.magic; w[7] = (uint32_t)(lv.magic >> 32); p_after = (p_after + lv.radix - 1) / lv.radix;
                w[kFastDescMagic0] = lv.radix > 1 ? (uint32_t)((1ull << 32) / lv.radix) : 0xffffffffu;
            }
            else {
                if (p_after >> 32) return false;                     // 32-bit quotient chain after the first step
                w[11 + l] = (uint32_t)((1ull << 32) / lv.radix);
            }
        }
        for (int l = nlev; l < kFastMaxLevels; ++l) {          // steps the class does not have: radix 1 and the matching reciprocals, no slots:
            w[8 + l] = 1u;                                      // the division by multiplication then returns the rank unchanged and
            if (l == 0) { w[6] = w[7] = 0xffffffffu; w[kFastDescMagic0] = 0xffffffffu; }    // remainder 0, so a lane that runs such a
            else w[11 + l] = 0xffffffffu;                       // step beside lanes with more steps needs no special case
        }
        std::memcpy(&w[4], vals, 8);
        // odd classes have no group 1: numbered without the gap at id 1, a class of four distinct values stays within ids 0..3
        // (two bit planes) for the decoder form that handles odd classes alone
        uint8_t vals_odd[8] = {d.fill0, 0, 0, 0, 0, 0, 0, 0};
        if (d.parity)
            for (int l = 0; l < nlev; ++l) vals_odd[1 + l] = d.lev[l].val;
        std::memcpy(&w[kFastDescValsOdd], vals_odd, 8);
        w[15] = nbytes;
        const float rnorm = (float)(1.0 / std::sqrt(16.0 * (double)d.m));
        std::memcpy(&w[kFastDescRnorm], &rnorm, 4);
    }
    return true;
}

void build_big_descs(const HostTables& t, std::vector<BigDesc>& out)
{
    out.assign(t.desc.size(), BigDesc{});
    for (size_t j = 0; j < t.desc.size(); ++j) {
        const ClassDesc& d = t.desc[j];
        BigDesc& b = out[j];
        const int nlev = d.nlev1 + d.nlev0;
        b.w = d.w; b.B = d.B;
        b.flags = (uint8_t)((d.parity ? 1u : 0u) | (d.signpar ? 2u : 0u) | (d.fill0 ? 4u : 0u) | ((d.fill1 & 2) ? 8u : 0u) | ((d.fill0 & 2) ? 16u : 0u));
        b.nlev = (uint8_t)(d.nlev1 | nlev << 4);
        b.goff = d.goff; b.A = d.A;
        b.val[0] = d.fill0; b.val[1] = d.fill1;
        for (int l = 0; l < nlev && l < kMaxLevels - 1; ++l) {
            const LevelDesc& lv = d.lev[l];
            if (l < 6) b.val[2 + l] = lv.val; else b.val8 = lv.val;
            b.k[l] = lv.k;
            if (lv.val & 2) b.lvl_bit1 |= (uint8_t)(1u << l);
            if (lv.val) b.lvl_nz |= (uint8_t)(1u << l);
            if (lv.k <= kSmallSubsetMaxK) b.small_k |= (uint8_t)(1u << l);
        }
    }
}

// Class of the first index of every bucket (I >> (W - 16)), plus a final entry = last class: the class of an
// index lies between the entries of its bucket and of the next one.
void build_bucket_table(const HostTables& t, std::vector<uint32_t>& lut)
{
    const size_t ncls = t.desc.size();
    const int shift = t.W > 16 ? t.W - 16 : 0;
    lut.assign(65537, (uint32_t)(ncls - 1));
    size_t c = 0;
    for (uint32_t b = 0; b < 65536; ++b) {
        u128 first = (u128)b << shift;
        if (first >= t.N) break;
        while (c + 1 < ncls && t.offset[c + 1] <= first) ++c;
        lut[b] = (uint32_t)c;
    }
}

}  // namespace llvq

namespace llvq {

// splitmix64 of (a + 1): fixed, well-mixed 64-bit numbers
uint64_t sig_of_value(int a)
{
    uint64_t z = (uint64_t)(a + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Open-addressing table (linear probing) from class signature to class number, at most 25 % full.
bool build_class_hash(const HostTables& t, std::vector<uint64_t>& keys, std::vector<uint32_t>& cls)
{
    size_t size = 64;
    while (size < 4 * t.info.size()) size *= 2;
    keys.assign(size, 0);
    cls.assign(size, 0);
    for (size_t j = 0; j < t.info.size(); ++j) {
        const ClassInfo& c = t.info[j];
        uint64_t sig = 0;
        for (size_t i = 0; i < c.values.size(); ++i) sig += (uint64_t)c.mults[i] * sig_of_value(c.values[i]);
        if (sig == 0) return false;
        size_t slot = (size_t)(sig >> 20) & (size - 1);
        while (keys[slot]) {
            if (keys[slot] == sig) return false;             // two classes with one signature
            slot = (slot + 1) & (size - 1);
        }
        keys[slot] = sig; cls[slot] = (uint32_t)j;
    }
    return true;
}

}  // namespace llvq
