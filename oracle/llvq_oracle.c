/*
 * LLVQ CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-purpose C implementation of the Leech-lattice indexing
 * and dequantization of "Leech Lattice Vector Quantization for Efficient LLM
 * Compression".  It exists so that the CUDA library can be checked against
 * something written independently from the paper.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.  It shares no
 * code, table or constant generator with the CUDA path.
 *
 * Every function names the passage of the paper it follows.  Where the paper
 * leaves a convention open (orderings, bit assignment), the convention chosen
 * is stated at the function that implements it.
 *
 * Parity pins (see tests, "-m not gpu"): Golay weight distribution; shell
 * sizes of Table 1; the 15 class rows of Table 2; class cardinalities summing
 * to the theta-series shell sizes; lattice membership of every decoded point;
 * exhaustive rank(unrank(I)) == I on Shell(2) and Shell(3); set equality of
 * the decoded Shell(2) with the textbook description of the 196560 minimal
 * vectors; bf16 rounding against a library conversion; GEMV against exact
 * integer special cases.  No function here is "parity unpinned".
 *
 * Integer coordinates throughout: x in Z^24 with sum x_i^2 = 16 m for
 * Shell(m); the lattice itself is x / sqrt(8) (Sec. 2.3, "Integer-coordinate
 * formulation").
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

typedef unsigned __int128 u128;

#define OC_DIM 24
#define OC_MAX_M 64          /* shells 2..64 supported by the shell-size table */
#define OC_MAX_VALS 24

/* ------------------------------------------------------------------------- */
/* Extended binary Golay code (Sec. 2.3: 4096 words, weights 0/8/12/16/24).   */
/* Convention (paper silent): cyclic [23,12,7] code with generator polynomial */
/* g(x) = x^11+x^10+x^6+x^5+x^4+x^2+1, message u -> u(x) g(x), bit i of the    */
/* word <-> coordinate i, plus an overall parity bit at coordinate 23.        */
/* The table T lists the words sorted by (weight, numeric value).             */
/* ------------------------------------------------------------------------- */
static uint32_t g_T[4096];
static int g_woff[25];        /* first position in T of the words of weight w */
static int g_wcnt[25];
static int g_golay_ready = 0;
static int16_t* g_pos_of_word = NULL;   /* word -> position in T, -1 if not a codeword */

static int popcount32(uint32_t v) { int c = 0; while (v) { c += (int)(v & 1u); v >>= 1; } return c; }

static uint32_t poly_mul_gf2(uint32_t u, uint32_t g)
{
    uint32_t r = 0;
    for (int i = 0; i < 12; ++i)
        if ((u >> i) & 1u) r ^= g << i;
    return r;
}

static int cmp_weight_then_value(const void* a, const void* b)
{
    uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
    int wx = popcount32(x), wy = popcount32(y);
    if (wx != wy) return wx < wy ? -1 : 1;
    return x < y ? -1 : (x > y ? 1 : 0);
}

void oc_golay_init(void)
{
    if (g_golay_ready) return;
    const uint32_t g = 0xC75u;
    for (uint32_t u = 0; u < 4096; ++u) {
        uint32_t c = poly_mul_gf2(u, g);                 /* 23-bit cyclic codeword */
        c |= (uint32_t)(popcount32(c) & 1) << 23;          /* overall parity bit     */
        g_T[u] = c;
    }
    qsort(g_T, 4096, sizeof(uint32_t), cmp_weight_then_value);
    memset(g_wcnt, 0, sizeof g_wcnt);
    for (int i = 0; i < 4096; ++i) g_wcnt[popcount32(g_T[i])]++;
    int off = 0;
    for (int w = 0; w <= 24; ++w) { g_woff[w] = off; off += g_wcnt[w]; }
    g_pos_of_word = (int16_t*)malloc(sizeof(int16_t) << 24);
    for (uint32_t v = 0; v < (1u << 24); ++v) g_pos_of_word[v] = -1;
    for (int i = 0; i < 4096; ++i) g_pos_of_word[g_T[i]] = (int16_t)i;
    g_golay_ready = 1;
}

/* Copy of the sorted codeword table, for tests. */
void oc_golay_table(uint32_t out[4096]) { oc_golay_init(); memcpy(out, g_T, sizeof g_T); }

/* Position of word c inside the sorted table, or -1 if c is not a codeword
 * (direct lookup over all 2^24 words, filled on first use). */
static int golay_find(uint32_t c)
{
    if (c >> 24) return -1;
    return g_pos_of_word[c];
}

/* ------------------------------------------------------------------------- */
/* Lattice membership, Sec. 2.3 conditions (i)-(iii) of L^even and L^odd.      */
/* Returns 0 = even coset, 1 = odd coset, -1 = not a lattice point.           */
/* Floor semantics for negative coordinates: bit = ((x - parity) >> 1) & 1.   */
/* ------------------------------------------------------------------------- */
int oc_is_member(const int8_t x[OC_DIM])
{
    oc_golay_init();
    int parity = x[0] & 1;
    long sum = 0;
    uint32_t word = 0;
    for (int i = 0; i < OC_DIM; ++i) {
        if ((x[i] & 1) != parity) return -1;                       /* (i)   */
        int h = ((int)x[i] - parity) >> 1;                          /* floor */
        word |= (uint32_t)(h & 1) << i;
        sum += x[i];
    }
    if (golay_find(word) < 0) return -1;                            /* (ii)  */
    long r = ((sum % 8) + 8) % 8;
    if (r != (parity ? 4 : 0)) return -1;                           /* (iii) */
    return parity;
}

/* ------------------------------------------------------------------------- */
/* Shell sizes n(m): coefficients of the Leech theta series (Sec. 2.2 cites    */
/* them as such).  Closed form: n(m) = 65520/691 * (sigma_11(m) - tau(m)),    */
/* tau = Ramanujan's function, the coefficients of q * prod (1-q^n)^24.       */
/* ------------------------------------------------------------------------- */
static u128 g_shell[OC_MAX_M + 1];
static int g_shell_ready = 0;

static void shell_init(void)
{
    if (g_shell_ready) return;
    /* tau(1..OC_MAX_M): expand prod_{n>=1} (1 - q^n)^24 up to q^(OC_MAX_M-1). */
    __int128 poly[OC_MAX_M + 1];
    memset(poly, 0, sizeof poly);
    poly[0] = 1;
    for (int n = 1; n <= OC_MAX_M; ++n)
        for (int rep = 0; rep < 24; ++rep)
            for (int d = OC_MAX_M; d >= n; --d) poly[d] -= poly[d - n];
    /* tau(m) = coefficient of q^(m-1) in the product */
    for (int m = 1; m <= OC_MAX_M; ++m) {
        u128 sigma = 0;
        for (int d = 1; d <= m; ++d) {
            if (m % d) continue;
            u128 p = 1;
            for (int e = 0; e < 11; ++e) p *= (u128)d;
            sigma += p;
        }
        __int128 diff = (__int128)sigma - poly[m - 1];
        g_shell[m] = (u128)(diff * 65520 / 691);
    }
    g_shell[0] = 0;
    g_shell_ready = 1;
}

/* n(m) as two 64-bit halves (lo, hi). */
void oc_shell_size(int m, uint64_t out[2])
{
    shell_init();
    u128 v = (m >= 1 && m <= OC_MAX_M) ? g_shell[m] : 0;
    out[0] = (uint64_t)v; out[1] = (uint64_t)(v >> 64);
}

/* ------------------------------------------------------------------------- */
/* Classes (Sec. 2.4-2.5, Table 2).  A class is a multiset of 24 absolute      */
/* values plus a parity.  Admissibility, derived from the placement and sign  */
/* rules of Sec. 2.4:                                                         */
/*   even: all values even; w = #{a = 2 mod 4} is a Golay weight; if w = 0     */
/*         the number of values = 4 mod 8 must be even (sum = 0 mod 8).       */
/*   odd:  all values odd; #{a = 3 or 5 mod 8} is odd (sum = 4 mod 8).        */
/* Cardinality (Sec. 2.5): A * 2^B * P with                                    */
/*   odd:  A = 4096, B = 0, P = 24!/prod p_i!                                  */
/*   even: A = #codewords of weight w, B = #{a = 0 mod 4, a > 0} + max(w-1,0), */
/*         P = P1*P0, P1 = w!/prod(mult of values = 2 mod 4)!,                */
/*         P0 = (24-w)!/prod(mult of values = 0 mod 4, zero included)!.       */
/* (The formula as typeset in Sec. 2.5 does not reproduce Table 2; this one   */
/* reproduces all 15 rows.)                                                   */
/* ------------------------------------------------------------------------- */
typedef struct {
    int m;                         /* shell                                    */
    int parity;                    /* 0 even, 1 odd                            */
    int w;                         /* even: number of coordinates = 2 mod 4    */
    int nvals;                     /* number of distinct absolute values       */
    int val[OC_MAX_VALS];          /* distinct absolute values, descending     */
    int mult[OC_MAX_VALS];         /* their multiplicities                     */
    uint64_t A;                    /* Golay refinements                        */
    int B;                         /* free sign bits                           */
    u128 P1, P0, P;                /* arrangement counts                       */
    u128 card;                     /* A * 2^B * P                              */
    u128 offset;                   /* first global index of the class          */
} oc_class;

typedef struct {
    int m_lo, m_hi;
    int nclasses;
    oc_class* cls;
    u128 N;                        /* number of points of the code             */
    int W;                         /* ceil(log2 N) index bits                  */
    int first_class_of_shell[OC_MAX_M + 2];
} oc_code;

static u128 binom(int n, int k)
{
    if (k < 0 || k > n) return 0;
    u128 r = 1;
    for (int i = 1; i <= k; ++i) r = r * (u128)(n - k + i) / (u128)i;
    return r;
}

/* multinomial n!/prod mult[i]! over the entries flagged by sel[] */
static u128 multinomial(int n, const int* mult, const int* sel, int nvals)
{
    u128 r = 1; int left = n;
    for (int i = 0; i < nvals; ++i) {
        if (!sel[i]) continue;
        r *= binom(left, mult[i]);
        left -= mult[i];
    }
    return left == 0 ? r : 0;
}

static int class_admissible(oc_class* c)
{
    if (c->parity == 0) {
        int w = 0, n4 = 0;
        for (int i = 0; i < c->nvals; ++i) {
            if (c->val[i] % 4 == 2) w += c->mult[i];
            if (c->val[i] % 8 == 4) n4 += c->mult[i];
        }
        if (!(w == 0 || w == 8 || w == 12 || w == 16 || w == 24)) return 0;
        if (w == 0 && (n4 & 1)) return 0;
        c->w = w;
        return 1;
    } else {
        int n35 = 0;
        for (int i = 0; i < c->nvals; ++i)
            if (c->val[i] % 8 == 3 || c->val[i] % 8 == 5) n35 += c->mult[i];
        c->w = 0;
        return n35 & 1;
    }
}

static void class_counts(oc_class* c)
{
    oc_golay_init();
    int sel1[OC_MAX_VALS], sel0[OC_MAX_VALS], all[OC_MAX_VALS];
    for (int i = 0; i < c->nvals; ++i) {
        sel1[i] = (c->val[i] % 4 == 2);
        sel0[i] = (c->val[i] % 4 == 0);
        all[i] = 1;
    }
    if (c->parity) {
        c->A = 4096; c->B = 0;
        c->P1 = 1; c->P0 = 1;
        c->P = multinomial(24, c->mult, all, c->nvals);
    } else {
        c->A = (uint64_t)g_wcnt[c->w];
        int b = 0;
        for (int i = 0; i < c->nvals; ++i)
            if (c->val[i] % 4 == 0 && c->val[i] > 0) b += c->mult[i];
        c->B = b + (c->w > 0 ? c->w - 1 : 0);
        c->P1 = multinomial(c->w, c->mult, sel1, c->nvals);
        c->P0 = multinomial(24 - c->w, c->mult, sel0, c->nvals);
        c->P = c->P1 * c->P0;
    }
    c->card = (u128)c->A * ((u128)1 << c->B) * c->P;
}

typedef struct { oc_class* v; int n, cap; } class_vec;

static void push_class(class_vec* out, const oc_class* c)
{
    if (out->n == out->cap) {
        out->cap = out->cap ? out->cap * 2 : 64;
        out->v = (oc_class*)realloc(out->v, (size_t)out->cap * sizeof(oc_class));
    }
    out->v[out->n++] = *c;
}

/* Enumerate multisets: values v, v-2, ... of one parity, multiplicities summing
 * to 24, squares summing to 16 m.  cur holds the partial multiset. */
static void enum_rec(int v, int left, long norm, oc_class* cur, class_vec* out)
{
    if (v < 0) return;
    if (v <= 1) {                       /* last value: 0 (even) or 1 (odd) takes the rest */
        if ((long)left * v * v != norm) return;
        oc_class c = *cur;
        if (left > 0) { c.val[c.nvals] = v; c.mult[c.nvals] = left; c.nvals++; }
        if (class_admissible(&c)) { class_counts(&c); push_class(out, &c); }
        return;
    }
    for (int k = 0; k <= left && (long)k * v * v <= norm; ++k) {
        int saved = cur->nvals;
        if (k > 0) { cur->val[cur->nvals] = v; cur->mult[cur->nvals] = k; cur->nvals++; }
        enum_rec(v - 2, left - k, norm - (long)k * v * v, cur, out);
        cur->nvals = saved;
    }
}

/* Leader = the 24 absolute values in descending order. */
static void leader_of(const oc_class* c, int out[OC_DIM])
{
    int p = 0;
    for (int i = 0; i < c->nvals; ++i)
        for (int j = 0; j < c->mult[i]; ++j) out[p++] = c->val[i];
}

/* Class order inside a shell (paper: "a deterministic total order"; Table 2
 * prints even classes before odd ones).  Convention: even classes first, by
 * ascending w, then by leader ascending lexicographically; then odd classes
 * by leader descending lexicographically.  This is the row order of Table 2
 * for m = 2, 3, 4 and puts (4^2, 0^22) first in Shell(2) (Sec. 2.3). */
static int cmp_class(const void* pa, const void* pb)
{
    const oc_class* a = (const oc_class*)pa; const oc_class* b = (const oc_class*)pb;
    if (a->parity != b->parity) return a->parity < b->parity ? -1 : 1;
    int la[OC_DIM], lb[OC_DIM];
    leader_of(a, la); leader_of(b, lb);
    int lex = 0;
    for (int i = 0; i < OC_DIM && !lex; ++i) lex = (la[i] > lb[i]) - (la[i] < lb[i]);
    if (a->parity == 0) {
        if (a->w != b->w) return a->w < b->w ? -1 : 1;
        return lex;
    }
    return -lex;
}

static void shell_classes(int m, class_vec* out)
{
    long norm = 16L * m;
    int vmax = (int)floor(sqrt((double)norm) + 1e-9);
    int first = out->n;
    for (int parity = 0; parity <= 1; ++parity) {
        int v0 = vmax;
        if ((v0 & 1) != parity) v0--;
        oc_class cur; memset(&cur, 0, sizeof cur);
        cur.m = m; cur.parity = parity;
        enum_rec(v0, 24, norm, &cur, out);
    }
    qsort(out->v + first, (size_t)(out->n - first), sizeof(oc_class), cmp_class);
}

/* Code = union of Shell(m), m_lo <= m <= m_hi (Sec. 2.2 ball cut when m_lo = 2).
 * Global offsets: shells in increasing m, classes in the order above
 * (Sec. 3.2 (1)-(2)).  Indices are 0-based, ranges half-open. */
oc_code* oc_code_create(int m_lo, int m_hi)
{
    if (m_lo < 2 || m_hi < m_lo || m_hi > OC_MAX_M) return NULL;
    oc_golay_init(); shell_init();
    oc_code* code = (oc_code*)calloc(1, sizeof(oc_code));
    code->m_lo = m_lo; code->m_hi = m_hi;
    class_vec v = {0, 0, 0};
    for (int m = m_lo; m <= m_hi; ++m) {
        code->first_class_of_shell[m] = v.n;
        shell_classes(m, &v);
    }
    code->first_class_of_shell[m_hi + 1] = v.n;
    u128 off = 0;
    for (int i = 0; i < v.n; ++i) { v.v[i].offset = off; off += v.v[i].card; }
    code->cls = v.v; code->nclasses = v.n; code->N = off;
    int W = 0;
    while (W < 128 && ((u128)1 << W) < off) ++W;
    code->W = W;
    return code;
}

void oc_code_destroy(oc_code* c) { if (c) { free(c->cls); free(c); } }
int  oc_code_num_classes(const oc_code* c) { return c->nclasses; }
int  oc_code_index_bits(const oc_code* c) { return c->W; }
void oc_code_num_points(const oc_code* c, uint64_t out[2]) { out[0] = (uint64_t)c->N; out[1] = (uint64_t)(c->N >> 64); }

/* Class description for tests: info = {m, parity, w, nvals, B}, A, card, offset, values, mults. */
void oc_class_info(const oc_code* c, int j, int info[5], uint64_t* A, uint64_t card[2], uint64_t offset[2],
                   int vals[OC_MAX_VALS], int mults[OC_MAX_VALS])
{
    const oc_class* k = &c->cls[j];
    info[0] = k->m; info[1] = k->parity; info[2] = k->w; info[3] = k->nvals; info[4] = k->B;
    *A = k->A;
    card[0] = (uint64_t)k->card; card[1] = (uint64_t)(k->card >> 64);
    offset[0] = (uint64_t)k->offset; offset[1] = (uint64_t)(k->offset >> 64);
    for (int i = 0; i < k->nvals; ++i) { vals[i] = k->val[i]; mults[i] = k->mult[i]; }
}

/* ------------------------------------------------------------------------- */
/* Arrangement of a multiset on n slots from a rank (App. A step 4: "the       */
/* absolute-value pattern is rearranged by applying the permutation encoded   */
/* by I''").  Convention (paper: "a rank in its orbit"): the distinct values  */
/* are taken in descending order; each value except the last chooses its k    */
/* slots among the slots still free, by the combinatorial-number-system rank  */
/* rho_j = sum_t C(e_t, t) of the chosen slot numbers e_1 < ... < e_k         */
/* (numbered inside the list of free slots); rho = rho_0 + C_0*(rho_1 + ...). */
/* The last value fills what is left.                                         */
/* ------------------------------------------------------------------------- */
static void arrange(u128 rho, const int* vals, const int* mults, int nv, int n, int* out /* n slots */)
{
    int free_slot[OC_DIM]; int nfree = n;
    for (int i = 0; i < n; ++i) free_slot[i] = i;
    for (int j = 0; j < nv; ++j) {
        int k = mults[j];
        if (j == nv - 1) {                           /* last value fills the rest */
            for (int i = 0; i < nfree; ++i) out[free_slot[i]] = vals[j];
            break;
        }
        u128 C = binom(nfree, k);
        u128 rj = rho % C; rho /= C;
        int chosen[OC_DIM]; memset(chosen, 0, sizeof chosen);
        int hi = nfree;                              /* candidates e < hi */
        for (int t = k; t >= 1; --t) {
            int e = hi - 1;
            while (binom(e, t) > rj) --e;            /* largest e with C(e,t) <= rj */
            rj -= binom(e, t);
            chosen[e] = 1; hi = e;
        }
        int keep = 0;
        for (int i = 0; i < nfree; ++i) {
            if (chosen[i]) out[free_slot[i]] = vals[j];
            else free_slot[keep++] = free_slot[i];
        }
        nfree = keep;
    }
}

/* Inverse of arrange(): rank of the arrangement a[0..n) of the given multiset. */
static u128 arrange_rank(const int* a, const int* vals, const int* mults, int nv, int n)
{
    int free_slot[OC_DIM]; int nfree = n;
    for (int i = 0; i < n; ++i) free_slot[i] = i;
    u128 rho = 0, radix = 1;
    for (int j = 0; j + 1 < nv; ++j) {
        int k = mults[j];
        u128 rj = 0; int t = 0, keep = 0;
        for (int i = 0; i < nfree; ++i) {
            if (a[free_slot[i]] == vals[j]) { ++t; rj += binom(i, t); }
            else free_slot[keep++] = free_slot[i];
        }
        rho += radix * rj;
        radix *= binom(nfree, k);
        nfree = keep;
    }
    return rho;
}

static const oc_class* find_class(const oc_code* code, u128 I)
{
    /* App. A steps 1-2: the class whose half-open range [offset, offset+card)
     * contains I; the classes are sorted by offset, so bisect. */
    int lo = 0, hi = code->nclasses - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) / 2;
        if (code->cls[mid].offset <= I) lo = mid; else hi = mid - 1;
    }
    return &code->cls[lo];
}

/* ------------------------------------------------------------------------- */
/* Dequantizer, App. A steps 1-4: index -> integer lattice point.              */
/* Returns 0, or 1 when I >= N (then x is all zero).                          */
/* Sign conventions (paper silent on which bit signs which coordinate):       */
/*   odd:  x_i = -a_i iff c_i xor ((a_i >> 1) & 1), i.e. x_i = 1 mod 4 on F0  */
/*         and 3 mod 4 on F1 (Sec. 2.4).                                      */
/*   even: the positions that carry a sign -- all of F1 and the nonzero ones  */
/*         of F0 -- take the bits of s in ascending order of position (1 =    */
/*         negative), except the last F1 position, which takes the sign that  */
/*         makes the coordinate sum 0 mod 8.                                  */
/* ------------------------------------------------------------------------- */
static int unrank_point(const oc_code* code, u128 I, int8_t x[OC_DIM])
{
    memset(x, 0, OC_DIM);
    if (I >= code->N) return 1;
    const oc_class* k = find_class(code, I);
    u128 Ic = I - k->offset;
    /* step 3: r fastest, then s, then the permutation rank */
    uint64_t r = (uint64_t)(Ic % k->A);
    u128 I1 = Ic / k->A;
    uint64_t s = (uint64_t)(I1 % ((u128)1 << k->B));
    u128 p = I1 >> k->B;

    int a[OC_DIM];
    if (k->parity) {
        uint32_t c = g_T[r];
        arrange(p, k->val, k->mult, k->nvals, OC_DIM, a);
        for (int i = 0; i < OC_DIM; ++i) {
            int neg = (int)((c >> i) & 1u) ^ ((a[i] >> 1) & 1);
            x[i] = (int8_t)(neg ? -a[i] : a[i]);
        }
        return 0;
    }
    uint32_t c = g_T[g_woff[k->w] + (int)r];
    int F1[OC_DIM], F0[OC_DIM], n1 = 0, n0 = 0;
    for (int i = 0; i < OC_DIM; ++i) { if ((c >> i) & 1u) F1[n1++] = i; else F0[n0++] = i; }
    /* split the multiset by residue mod 4, keeping descending order */
    int v1[OC_MAX_VALS], m1[OC_MAX_VALS], nv1 = 0, v0[OC_MAX_VALS], m0[OC_MAX_VALS], nv0 = 0;
    int n4 = 0, n6 = 0;
    for (int i = 0; i < k->nvals; ++i) {
        if (k->val[i] % 4 == 2) { v1[nv1] = k->val[i]; m1[nv1++] = k->mult[i]; }
        else                    { v0[nv0] = k->val[i]; m0[nv0++] = k->mult[i]; }
        if (k->val[i] % 8 == 4) n4 += k->mult[i];
        if (k->val[i] % 8 == 6) n6 += k->mult[i];
    }
    u128 p1 = p % k->P1, p0 = p / k->P1;
    int a1[OC_DIM], a0[OC_DIM];
    if (n1) arrange(p1, v1, m1, nv1, n1, a1);
    if (n0) arrange(p0, v0, m0, nv0, n0, a0);
    /* absolute values by position, then the signs in one pass over the positions */
    int abs_at[OC_DIM];
    for (int t = 0; t < n1; ++t) abs_at[F1[t]] = a1[t];
    for (int t = 0; t < n0; ++t) abs_at[F0[t]] = a0[t];
    const int last_f1 = n1 ? F1[n1 - 1] : -1;
    int bit = 0, negs = 0;
    for (int i = 0; i < OC_DIM; ++i) {
        const int in_f1 = (int)((c >> i) & 1u);
        int neg = 0;
        if (in_f1 && i == last_f1) neg = (negs + n4 + n6) & 1;          /* every other F1 sign is known by now */
        else if (in_f1 || abs_at[i] != 0) { neg = (int)((s >> bit) & 1u); ++bit; negs += in_f1 ? neg : 0; }
        x[i] = (int8_t)(neg ? -abs_at[i] : abs_at[i]);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Indexing (Sec. 3.2): lattice point -> index, the inverse of the above.      */
/* Returns 0, or 1 if x is not a point of the code (then *I = 0).             */
/* ------------------------------------------------------------------------- */
static int rank_point(const oc_code* code, const int8_t x[OC_DIM], u128* I)
{
    *I = 0;
    int parity = oc_is_member(x);
    if (parity < 0) return 1;
    long norm = 0; int a[OC_DIM];
    for (int i = 0; i < OC_DIM; ++i) { a[i] = abs((int)x[i]); norm += (long)a[i] * a[i]; }
    if (norm % 16) return 1;
    int m = (int)(norm / 16);
    if (m < code->m_lo || m > code->m_hi) return 1;
    /* class = same shell, parity and multiset of absolute values */
    int cnt[64]; memset(cnt, 0, sizeof cnt);
    for (int i = 0; i < OC_DIM; ++i) cnt[a[i]]++;
    const oc_class* k = NULL;
    for (int j = code->first_class_of_shell[m]; j < code->first_class_of_shell[m + 1] && !k; ++j) {
        const oc_class* q = &code->cls[j];
        if (q->parity != parity) continue;
        int same = 1, total = 0;
        for (int i = 0; i < q->nvals; ++i) { same &= (cnt[q->val[i]] == q->mult[i]); total += q->mult[i]; }
        if (same && total == OC_DIM) k = q;
    }
    if (!k) return 1;
    uint32_t c = 0;
    for (int i = 0; i < OC_DIM; ++i) c |= (uint32_t)((((int)x[i] - parity) >> 1) & 1) << i;
    int pos = golay_find(c);
    u128 r, s = 0, p;
    if (parity) {
        r = (u128)pos;
        p = arrange_rank(a, k->val, k->mult, k->nvals, OC_DIM);
    } else {
        r = (u128)(pos - g_woff[k->w]);
        int F1[OC_DIM], F0[OC_DIM], n1 = 0, n0 = 0;
        for (int i = 0; i < OC_DIM; ++i) { if ((c >> i) & 1u) F1[n1++] = i; else F0[n0++] = i; }
        int v1[OC_MAX_VALS], m1[OC_MAX_VALS], nv1 = 0, v0[OC_MAX_VALS], m0[OC_MAX_VALS], nv0 = 0;
        for (int i = 0; i < k->nvals; ++i) {
            if (k->val[i] % 4 == 2) { v1[nv1] = k->val[i]; m1[nv1++] = k->mult[i]; }
            else                    { v0[nv0] = k->val[i]; m0[nv0++] = k->mult[i]; }
        }
        int a1[OC_DIM], a0[OC_DIM];
        for (int t = 0; t < n1; ++t) a1[t] = a[F1[t]];
        for (int t = 0; t < n0; ++t) a0[t] = a[F0[t]];
        u128 p1 = n1 ? arrange_rank(a1, v1, m1, nv1, n1) : 0;
        u128 p0 = n0 ? arrange_rank(a0, v0, m0, nv0, n0) : 0;
        p = p1 + k->P1 * p0;
        const int last_f1 = n1 ? F1[n1 - 1] : -1;
        int bit = 0;
        for (int i = 0; i < OC_DIM; ++i) {
            const int in_f1 = (int)((c >> i) & 1u);
            if (in_f1 && i == last_f1) continue;                           /* fixed by the others */
            if (in_f1 || a[i] != 0) { s |= (u128)(x[i] < 0) << bit; ++bit; }
        }
    }
    *I = k->offset + r + (u128)k->A * (s + ((u128)1 << k->B) * p);
    return 0;
}

/* Array front ends.  Indices travel as (lo, hi) 64-bit halves. */
int oc_unrank(const oc_code* code, const uint64_t* lo, const uint64_t* hi, int64_t n, int8_t* points)
{
    int bad = 0;
    for (int64_t b = 0; b < n; ++b)
        bad += unrank_point(code, ((u128)hi[b] << 64) | lo[b], points + b * OC_DIM);
    return bad;
}

int oc_rank(const oc_code* code, const int8_t* points, int64_t n, uint64_t* lo, uint64_t* hi)
{
    int bad = 0;
    for (int64_t b = 0; b < n; ++b) {
        u128 I; bad += rank_point(code, points + b * OC_DIM, &I);
        lo[b] = (uint64_t)I; hi[b] = (uint64_t)(I >> 64);
    }
    return bad;
}

/* For every I in [first, first+count): decode, check lattice membership, the
 * shell norm, and rank(unrank(I)) == I.  Returns the number of failures. */
int64_t oc_check_range(const oc_code* code, uint64_t first_lo, uint64_t first_hi, int64_t count)
{
    int64_t fails = 0;
    u128 first = ((u128)first_hi << 64) | first_lo;
    for (int64_t d = 0; d < count; ++d) {
        u128 I = first + (u128)d, J;
        int8_t x[OC_DIM];
        if (unrank_point(code, I, x)) { ++fails; continue; }
        const oc_class* k = find_class(code, I);
        long norm = 0;
        for (int i = 0; i < OC_DIM; ++i) norm += (long)x[i] * x[i];
        int ok = (oc_is_member(x) == k->parity) && (norm == 16L * k->m);
        ok = ok && (rank_point(code, x, &J) == 0) && (J == I);
        fails += !ok;
    }
    return fails;
}

/* ------------------------------------------------------------------------- */
/* Stored format.  Index stream: field b occupies bits [b*W, (b+1)*W) of a      */
/* little-endian bit stream (stream bit t = bit t%8 of byte t/8).  The paper   */
/* only says "bitstring"; this is the convention.                             */
/* ------------------------------------------------------------------------- */
static u128 stream_index(const uint8_t* stream, int W, int64_t b)
{
    u128 I = 0;
    for (int t = 0; t < W; ++t) {
        int64_t bitpos = b * (int64_t)W + t;
        I |= (u128)((stream[bitpos >> 3] >> (bitpos & 7)) & 1u) << t;
    }
    return I;
}

void oc_unpack_stream(const uint8_t* stream, int W, int64_t nblocks, uint64_t* lo, uint64_t* hi)
{
    for (int64_t b = 0; b < nblocks; ++b) {
        u128 I = stream_index(stream, W, b);
        lo[b] = (uint64_t)I; hi[b] = (uint64_t)(I >> 64);
    }
}

int64_t oc_decode_stream(const oc_code* code, const uint8_t* stream, int64_t nblocks, int8_t* points)
{
    int64_t bad = 0;
    for (int64_t b = 0; b < nblocks; ++b)
        bad += unrank_point(code, stream_index(stream, code->W, b), points + b * OC_DIM);
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Shape-gain reconstruction w = g * s (App. E "Shape-gain"), as stored here:  */
/* the gain is an IEEE binary16 number per block that multiplies the integer  */
/* coordinates; the product is formed in binary32 (it is exact: 11-bit by     */
/* 5-bit significands) and rounded once, to nearest even, to bfloat16.        */
/* ------------------------------------------------------------------------- */
static float half_bits_to_float(uint16_t h)
{
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)f, -24);
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp((double)(1024 + f), e - 25);
    return (float)(sign ? -v : v);
}

static uint16_t float_to_bf16_rne(float v)
{
    uint32_t u; memcpy(&u, &v, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fff;              /* NaN */
    uint32_t keep = u >> 16, rest = u & 0xffffu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1;
    return (uint16_t)keep;
}

static double bf16_bits_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16; float f; memcpy(&f, &u, 4);
    return (double)f;
}

uint16_t oc_dequant_scalar(uint16_t gain_f16, int x)
{
    return float_to_bf16_rne(half_bits_to_float(gain_f16) * (float)x);
}

/* layout 0 (FLAT): block b covers elements 24b..24b+23 of the row-major
 * flattened rows x cols matrix; the tail of the last block is dropped.
 * layout 1 (ROWWISE): each row has ceil(cols/24) blocks of its own; the tail
 * of a row's last block is dropped.  out is rows x cols, dense. */
int64_t oc_dequant_matrix(const oc_code* code, const uint8_t* stream, const uint16_t* gain_f16,
                          int64_t rows, int64_t cols, int layout, uint16_t* out)
{
    int64_t bad = 0;
    int8_t x[OC_DIM];
    if (layout == 0) {
        int64_t total = rows * cols, nblocks = (total + OC_DIM - 1) / OC_DIM;
        for (int64_t b = 0; b < nblocks; ++b) {
            bad += unrank_point(code, stream_index(stream, code->W, b), x);
            for (int j = 0; j < OC_DIM; ++j) {
                int64_t e = b * OC_DIM + j;
                if (e < total) out[e] = oc_dequant_scalar(gain_f16[b], x[j]);
            }
        }
    } else {
        int64_t bpr = (cols + OC_DIM - 1) / OC_DIM;
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t cb = 0; cb < bpr; ++cb) {
                int64_t b = r * bpr + cb;
                bad += unrank_point(code, stream_index(stream, code->W, b), x);
                for (int j = 0; j < OC_DIM; ++j) {
                    int64_t col = cb * OC_DIM + j;
                    if (col < cols) out[r * cols + col] = oc_dequant_scalar(gain_f16[b], x[j]);
                }
            }
    }
    return bad;
}

/* Fused product of App. C, Y[b][i] = sum_k X[b][k] * w[i][k], ROWWISE blocks,
 * over the bf16-rounded weights and the bf16 inputs, accumulated in binary64.
 * Rows [row_first, row_first + row_count) only (so callers can time a sample
 * or split rows over threads); y is batch x n_out, only those columns are
 * written. */
int64_t oc_gemm_rows(const oc_code* code, const uint8_t* stream, const uint16_t* gain_f16,
                     int64_t n_out, int64_t k_in, const uint16_t* x_bf16, int batch,
                     int64_t row_first, int64_t row_count, double* y)
{
    int64_t bad = 0, bpr = (k_in + OC_DIM - 1) / OC_DIM;
    int8_t pt[OC_DIM];
    for (int64_t r = row_first; r < row_first + row_count && r < n_out; ++r) {
        for (int bb = 0; bb < batch; ++bb) y[(int64_t)bb * n_out + r] = 0.0;
        for (int64_t cb = 0; cb < bpr; ++cb) {
            int64_t b = r * bpr + cb;
            bad += unrank_point(code, stream_index(stream, code->W, b), pt);
            for (int j = 0; j < OC_DIM; ++j) {
                int64_t col = cb * OC_DIM + j;
                if (col >= k_in) break;
                double w = bf16_bits_to_double(oc_dequant_scalar(gain_f16[b], pt[j]));
                for (int bb = 0; bb < batch; ++bb)
                    y[(int64_t)bb * n_out + r] += w * bf16_bits_to_double(x_bf16[(int64_t)bb * k_in + col]);
            }
        }
    }
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Shape-gain with a projected spherical code and a scalar gain code (App. E   */
/* "Shape-gain"; App. "spherical shaping or shape-gain": C_shape = {x/|x|},    */
/* C_gain a small codebook, reconstruction = gain * shape), optionally times a */
/* high-precision scale per output row ("0 bit gain": the scale alone).       */
/* Stored field of W + gain_bits bits: shape index I in the low W bits, gain   */
/* index k above it (the paper only says the pair is one integer; this is the */
/* convention).  Arithmetic, all in binary32, each operation rounded once:    */
/*   rn = (float)(1 / sqrt(sum x_i^2))      (formed in binary64, then rounded) */
/*   g  = (row_scale * codebook[k]) * rn                                        */
/*   w_j = bf16_rne(g * (float)x_j)                                            */
/* row_scale == NULL means 1.  An index I >= N decodes to zeros (rn = 0).     */
/* ------------------------------------------------------------------------- */
static u128 stream_field(const uint8_t* stream, int width, int64_t b) { return stream_index(stream, width, b); }

static float sg_block_gain(const int8_t x[OC_DIM], float row_scale, float cb)
{
    long norm = 0;
    for (int i = 0; i < OC_DIM; ++i) norm += (long)x[i] * x[i];
    volatile float rn = norm ? (float)(1.0 / sqrt((double)norm)) : 0.0f;
    volatile float sc = row_scale * cb;
    volatile float g = sc * rn;
    return g;
}

static uint16_t sg_weight(float g, int x)
{
    volatile float prod = g * (float)x;
    return float_to_bf16_rne(prod);
}

/* ROWWISE blocks only (a row scale has no meaning for a block that spans rows). */
int64_t oc_dequant_matrix_sg(const oc_code* code, const uint8_t* stream, int gain_bits, const float* codebook,
                             const float* row_scale, int64_t rows, int64_t cols, uint16_t* out)
{
    int64_t bad = 0, bpr = (cols + OC_DIM - 1) / OC_DIM;
    int8_t x[OC_DIM];
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t cb = 0; cb < bpr; ++cb) {
            u128 field = stream_field(stream, code->W + gain_bits, r * bpr + cb);
            u128 I = field & (((u128)1 << code->W) - 1);
            int k = (int)(field >> code->W);
            bad += unrank_point(code, I, x);
            float g = sg_block_gain(x, row_scale ? row_scale[r] : 1.0f, codebook[k]);
            for (int j = 0; j < OC_DIM; ++j) {
                int64_t col = cb * OC_DIM + j;
                if (col < cols) out[r * cols + col] = sg_weight(g, x[j]);
            }
        }
    return bad;
}

int64_t oc_gemm_rows_sg(const oc_code* code, const uint8_t* stream, int gain_bits, const float* codebook,
                        const float* row_scale, int64_t n_out, int64_t k_in, const uint16_t* x_bf16, int batch,
                        int64_t row_first, int64_t row_count, double* y)
{
    int64_t bad = 0, bpr = (k_in + OC_DIM - 1) / OC_DIM;
    int8_t pt[OC_DIM];
    for (int64_t r = row_first; r < row_first + row_count && r < n_out; ++r) {
        for (int bb = 0; bb < batch; ++bb) y[(int64_t)bb * n_out + r] = 0.0;
        for (int64_t cb = 0; cb < bpr; ++cb) {
            u128 field = stream_field(stream, code->W + gain_bits, r * bpr + cb);
            u128 I = field & (((u128)1 << code->W) - 1);
            int k = (int)(field >> code->W);
            bad += unrank_point(code, I, pt);
            float g = sg_block_gain(pt, row_scale ? row_scale[r] : 1.0f, codebook[k]);
            for (int j = 0; j < OC_DIM; ++j) {
                int64_t col = cb * OC_DIM + j;
                if (col >= k_in) break;
                double w = bf16_bits_to_double(sg_weight(g, pt[j]));
                for (int bb = 0; bb < batch; ++bb)
                    y[(int64_t)bb * n_out + r] += w * bf16_bits_to_double(x_bf16[(int64_t)bb * k_in + col]);
            }
        }
    }
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Encoder: nearest point of the code to a real vector (Sec. 3.1, "Extending to */
/* spherical search": Euclidean scoring for spherical shaping, angular scoring */
/* for shape-gain).  The paper defers the search itself to the literature; the */
/* search used here is coset decoding of the whole lattice, which is exact for */
/* the unbounded lattice: every lattice point is pi + 2c + 4z with pi the      */
/* parity, c a Golay codeword and z integer, subject to the sum rule of        */
/* Sec. 2.4; for fixed (pi, c) the nearest z is found by rounding each          */
/* coordinate and, if the sum rule fails, moving the coordinate with the       */
/* largest rounding error to its other neighbour.  The best of the 2 x 4096     */
/* cosets is the nearest lattice point.  Ties: lowest parity, then lowest      */
/* codeword position in T; inside a coset the first coordinate with the        */
/* largest error.  Inputs are in integer-coordinate units (|x|^2 = 16 m).      */
/*                                                                           */
/* Restriction to the shells m_lo..m_hi of the code (m_lo must be 2, m_hi >= 3).  */
/* Inputs are binary32 values widened exactly; every operation below is one     */
/* binary64 operation (no contraction), sums run over the coordinates in order. */
/* EUCLIDEAN (metric 0): if the nearest lattice point of the input lies in the   */
/*   code it is the answer (it is then the nearest point of the cut as well).   */
/*   Otherwise -- the input lies outside the ball of App. E "Spherical shaping", */
/*   or so close to the origin that the origin is nearest -- the input direction */
/*   is decoded at every shell radius sqrt(16 m), and of the candidates that lie  */
/*   in the code the one nearest to the input wins (first radius on ties).       */
/* ANGULAR (metric 1): for every shell radius sqrt(16 m) the input direction    */
/*   scaled to that radius is decoded; of the candidates that lie in the code   */
/*   the one with the largest cosine wins (first radius on ties).              */
/* A zero input encodes to index 0.  The search is exact for the unbounded      */
/* lattice, hence on the cut whenever the unconstrained answer lies in it; for  */
/* the other inputs it is a candidate search, pinned by what it reaches.        */
/* ------------------------------------------------------------------------- */
static double nearest_in_lattice(const double v[OC_DIM], int best_x[OC_DIM])
{
    oc_golay_init();
    double best = INFINITY;
    for (int pi = 0; pi < 2; ++pi)
        for (int j = 0; j < 4096; ++j) {
            uint32_t c = g_T[j];
            int x[OC_DIM]; double err[OC_DIM]; long sum = 0; double d2 = 0;
            for (int i = 0; i < OC_DIM; ++i) {
                int base = pi + 2 * (int)((c >> i) & 1u);
                double t = (v[i] - base) / 4.0;
                double z = rint(t);                       /* ties to even */
                err[i] = t - z;
                x[i] = base + 4 * (int)z;
                sum += x[i];
            }
            long want = pi ? 4 : 0;
            if (((sum % 8) + 8) % 8 != want) {            /* sum rule violated: one coordinate moves by 4 */
                int k = 0;
                for (int i = 1; i < OC_DIM; ++i) if (fabs(err[i]) > fabs(err[k])) k = i;
                x[k] += err[k] > 0 ? 4 : (err[k] < 0 ? -4 : 4);
            }
            for (int i = 0; i < OC_DIM; ++i) { double d = v[i] - x[i]; d2 += d * d; }
            if (d2 < best) { best = d2; memcpy(best_x, x, sizeof x); }
        }
    return best;
}

static int shell_of(const int x[OC_DIM])
{
    long n = 0;
    for (int i = 0; i < OC_DIM; ++i) n += (long)x[i] * x[i];
    return (int)(n / 16);
}

/* Returns 0 and the point, or 1 if the code is not one the encoder supports / the search gave up (point = index 0). */
static int encode_point(const oc_code* code, const double v[OC_DIM], int metric, int8_t out[OC_DIM])
{
    int x[OC_DIM], bestx[OC_DIM];
    double n2 = 0;
    for (int i = 0; i < OC_DIM; ++i) n2 += v[i] * v[i];
    int ok = 0;
    if (code->m_lo != 2 || code->m_hi < 3) { unrank_point(code, 0, out); return 1; }
    if (n2 == 0) { unrank_point(code, 0, out); return 0; }
    int direct = 0;
    if (metric == 0) {
        nearest_in_lattice(v, x);
        int m = shell_of(x);
        if (m >= code->m_lo && m <= code->m_hi) { ok = direct = 1; memcpy(bestx, x, sizeof x); }
    }
    if (!direct) {
        /* the input direction at every shell radius; metric 0 keeps the candidate nearest to the input, metric 1 the one
           with the largest cosine */
        double best = -INFINITY, rn = 1.0 / sqrt(n2);
        for (int m = code->m_lo; m <= code->m_hi; ++m) {
            double u[OC_DIM], rad = sqrt(16.0 * m);
            for (int i = 0; i < OC_DIM; ++i) u[i] = (v[i] * rn) * rad;
            nearest_in_lattice(u, x);
            int mx = shell_of(x);
            if (mx < code->m_lo || mx > code->m_hi) continue;
            double score;
            if (metric == 0) {
                double d2 = 0;
                for (int i = 0; i < OC_DIM; ++i) { double d = v[i] - x[i]; d2 += d * d; }
                score = -d2;
            } else {
                double dot = 0, xx = 0;
                for (int i = 0; i < OC_DIM; ++i) { dot += (v[i] * rn) * x[i]; xx += (double)x[i] * x[i]; }
                score = dot / sqrt(xx);
            }
            if (score > best) { best = score; ok = 1; memcpy(bestx, x, sizeof x); }
        }
    }
    if (!ok) { unrank_point(code, 0, out); return 1; }
    for (int i = 0; i < OC_DIM; ++i) out[i] = (int8_t)bestx[i];
    return 0;
}

/* v: n x 24 doubles.  points: n x 24 int8; lo/hi: the indices.  Returns the number of vectors the search gave up on. */
int64_t oc_encode(const oc_code* code, const double* v, int64_t n, int metric, int8_t* points, uint64_t* lo, uint64_t* hi)
{
    int64_t bad = 0;
    for (int64_t b = 0; b < n; ++b) {
        bad += encode_point(code, v + b * OC_DIM, metric, points + b * OC_DIM);
        u128 I = 0;
        rank_point(code, points + b * OC_DIM, &I);
        lo[b] = (uint64_t)I; hi[b] = (uint64_t)(I >> 64);
    }
    return bad;
}

/* The exact part alone: nearest point of the unbounded lattice (points may have any norm, the origin included). */
void oc_nearest_lattice_point(const double* v, int64_t n, int32_t* points, double* dist2)
{
    for (int64_t b = 0; b < n; ++b) {
        int x[OC_DIM];
        dist2[b] = nearest_in_lattice(v + b * OC_DIM, x);
        for (int i = 0; i < OC_DIM; ++i) points[b * OC_DIM + i] = x[i];
    }
}

/* ------------------------------------------------------------------------- */
/* Angular nearest point (Sec. 3.1): argmax over all points v of the code of   */
/* <x, v> / |v|, by brute force.  Lowest index wins ties.  Tiny codes only.   */
/* ------------------------------------------------------------------------- */
void oc_nearest_angular(const oc_code* code, const double* x, uint64_t out_index[2])
{
    u128 best = 0; double best_score = -INFINITY;
    for (u128 I = 0; I < code->N; ++I) {
        int8_t v[OC_DIM];
        unrank_point(code, I, v);
        double dot = 0, nn = 0;
        for (int i = 0; i < OC_DIM; ++i) { dot += x[i] * v[i]; nn += (double)v[i] * v[i]; }
        double score = dot / sqrt(nn);
        if (score > best_score) { best_score = score; best = I; }
    }
    out_index[0] = (uint64_t)best; out_index[1] = (uint64_t)(best >> 64);
}
