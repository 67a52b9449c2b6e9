/*
 * CO3 reference oracle — TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded C restatement of what the CO3 uplink pipeline and its
 * parameter-server inverse compute (arXiv 2204.08211): error correction with memory decay
 * (Sec. IV-A (iii)), conversion to the [sgn, exp, mant] floating-point format (Sec. IV-A (i),
 * level form in Sec. V-B), element-wise Huffman coding (Sec. IV-A (ii)), the memory update
 * (Algorithm 1) and decode + average at the parameter server (Sec. II-B (iv)).
 *
 * It exists so that tests can compare the CUDA library against it and so that a benchmark
 * can time it as a CPU baseline.  It shares no code, header, table or constant with the CUDA
 * library; nothing in the product may call it.  Every function is written for checking by
 * eye against the paper, not for speed: levels are enumerated and searched, Huffman merges
 * pick minima from a pool, bits are written and read one at a time.
 *
 * Where the paper is silent the reading taken is stated next to the code (zero and gradual
 * underflow, tie-breaks, length limit, container layout).
 *
 * Pins (tests/test_oracle_*.py): library casts to the standard 8/16-bit layouts, the closed forms
 * of Sec. V-B, exact-rational brute force over the printed level form, the printed bias
 * polynomials of Sec. IV-B, Kraft equality / entropy bounds / brute-force optimality for the
 * code, a hand-worked container example; for the dithered converter the published test vectors of
 * its generator and, with all 2^24 draws enumerated, the exact mean of the result.  Parity unpinned (the paper prints nothing to check
 * them against; only this oracle and the CUDA library agreeing): the order among equal Huffman
 * weights and the 16-bit length limit, the container layout, the NaN/Inf reading, and the tie
 * between zero and the smallest normal level when sub-normal levels are flushed.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CO3O_OK 0
#define CO3O_ERR_ARG 1
#define CO3O_ERR_CAPACITY 2
#define CO3O_ERR_NO_CODEWORD 3
#define CO3O_ERR_CORRUPT 5

#define CO3O_MAX_CODE_LEN 16 /* longest codeword either side accepts */
#define CO3O_MAX_CODES 65536 /* oracle accepts formats up to 16 bits so that binary16 can pin it */

typedef struct {
    int32_t exp_bits;          /* "exp" of [sgn, exp, mant] */
    int32_t mant_bits;         /* "mant" */
    int32_t flush_subnormals;  /* 0: exponent code 0 holds zero and gradual underflow; 1: only zero */
    float scale;               /* multiplier applied before rounding (1 / c_scale) */
    float inv_scale;           /* stored multiplier applied after rounding (c_scale) */
} co3o_fmt;

typedef struct {
    uint8_t len[256];   /* codeword length in bits, 0 = symbol has no codeword */
    uint32_t bits[256]; /* codeword, right-aligned, most significant bit is sent first */
} co3o_code;

/* ------------------------------------------------------------------------------------------
 * Level set (Sec. V-B): values c_sgn * c_scale * c_mant * 2^c_exp with
 *   c_mant in {1 + a_1/2 + ... + a_mant/2^mant},  c_exp in {-(2^(exp-1)-2), ..., 2^(exp-1)-1}.
 * That set uses 2^exp - 2 of the 2^exp exponent codes.  Reading taken for the other two
 * (the section cites the IEEE representation): exponent code 0 holds zero and, unless
 * flush_subnormals is set, the evenly spaced values k * 2^-mant * 2^emin below the smallest
 * normal level; the all-ones exponent code is never produced (out-of-range inputs saturate
 * to the boundary +-B of Sec. V-B instead).  c_scale is applied outside: levels here are for
 * the scaled input.
 *
 * A magnitude code c packs (exponent code << mant) | mantissa code; the symbol adds the sign
 * bit above it.  Zero is always sent with sign 0.
 * ------------------------------------------------------------------------------------------ */
static int co3o_emin(const co3o_fmt *f) { return -((1 << (f->exp_bits - 1)) - 2); }

int co3o_fmt_ok(const co3o_fmt *f)
{
    if (f->exp_bits < 2 || f->exp_bits > 8 || f->mant_bits < 0) return 0;
    if (1 + f->exp_bits + f->mant_bits > 16) return 0;
    if (!(f->scale > 0.0f) || !(f->inv_scale > 0.0f)) return 0;
    if (isinf(f->scale) || isinf(f->inv_scale)) return 0;
    return 1;
}

/* Magnitude of code c, or -1.0 if the code is never produced. */
double co3o_level(const co3o_fmt *f, uint32_t c)
{
    const int E = f->exp_bits, M = f->mant_bits;
    const uint32_t efield = c >> M, mfield = c & ((1u << M) - 1u);
    if (efield >= (1u << E) - 1u) return -1.0; /* reserved exponent code (and out of range) */
    if (efield == 0) {
        if (f->flush_subnormals && mfield != 0) return -1.0;
        return ldexp((double)mfield, co3o_emin(f) - M);
    }
    const double c_mant = 1.0 + ldexp((double)mfield, -M);
    const int c_exp = co3o_emin(f) + (int)efield - 1;
    return ldexp(c_mant, c_exp);
}

uint32_t co3o_max_code(const co3o_fmt *f)
{
    return (((1u << f->exp_bits) - 2u) << f->mant_bits) | ((1u << f->mant_bits) - 1u);
}

/* 1 if the symbol (sign bit above the magnitude code) can be produced by the converter. */
int co3o_symbol_valid(const co3o_fmt *f, uint32_t sym)
{
    const int nb = f->exp_bits + f->mant_bits;
    if (sym >= (2u << nb)) return 0;
    const uint32_t sign = sym >> nb, c = sym & ((1u << nb) - 1u);
    if (co3o_level(f, c) < 0.0) return 0;
    if (sign && c == 0) return 0; /* zero has one symbol */
    return 1;
}

/* Value the parameter server reconstructs for a symbol: level * stored inv_scale, in fp32. */
float co3o_symbol_value(const co3o_fmt *f, uint32_t sym)
{
    const int nb = f->exp_bits + f->mant_bits;
    const uint32_t sign = sym >> nb, c = sym & ((1u << nb) - 1u);
    const double lv = co3o_level(f, c);
    float q = (float)lv; /* exact: every level fits fp32 for exp_bits <= 8 */
    if (sign) q = -q;
    return q * f->inv_scale;
}

/* ------------------------------------------------------------------------------------------
 * Converter Q_fp for one scaled value t: rounds to the nearest level of the set in Sec. V-B.
 * The valid magnitude codes are enumerated in increasing order (their levels increase with
 * the code) and the two levels around |t| are compared against their midpoint.  Ties go to
 * the even code (IEEE default rounding, which the format section cites); when both codes are
 * even — only zero against the smallest normal level with flush_subnormals — to the smaller.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int n;
    uint32_t *code;
    double *level;
} co3o_levels;

static int co3o_levels_init(co3o_levels *L, const co3o_fmt *f)
{
    const uint32_t ncodes = 1u << (f->exp_bits + f->mant_bits);
    L->code = (uint32_t *)malloc(sizeof(uint32_t) * ncodes);
    L->level = (double *)malloc(sizeof(double) * ncodes);
    L->n = 0;
    if (!L->code || !L->level) return 0;
    for (uint32_t c = 0; c < ncodes; ++c) {
        const double lv = co3o_level(f, c);
        if (lv < 0.0) continue;
        L->code[L->n] = c;
        L->level[L->n] = lv;
        L->n++;
    }
    return 1;
}

static void co3o_levels_free(co3o_levels *L)
{
    free(L->code);
    free(L->level);
}

/* Nearest valid magnitude code to a >= 0 (a may be +inf). *saturated = 1 if a lies above the top level. */
static uint32_t co3o_nearest(const co3o_levels *L, double a, int *saturated)
{
    int lo = 0, hi = L->n - 1;
    *saturated = 0;
    if (a > L->level[hi]) {
        *saturated = 1;
        return L->code[hi];
    }
    /* largest index with level <= a */
    while (lo < hi) {
        const int mid = (lo + hi + 1) / 2;
        if (L->level[mid] <= a) lo = mid; else hi = mid - 1;
    }
    if (lo == L->n - 1) return L->code[lo];
    const double twice = 2.0 * a, mid2 = L->level[lo] + L->level[lo + 1]; /* both exact in fp64 */
    if (twice < mid2) return L->code[lo];
    if (twice > mid2) return L->code[lo + 1];
    if ((L->code[lo] & 1u) == 0) return L->code[lo]; /* even code, or the smaller of two even ones */
    return L->code[lo + 1];
}

/*
 * One client, one layer, one round (Algorithm 1, the three per-user updates):
 *   v    = g + gamma * m          (Sec. IV-A (iii)); one fused multiply-add in fp32
 *   ghat = Q_fp(v)                 = level(nearest(v * scale)) * inv_scale, each product in fp32
 *   m    = v - ghat                (= gamma * m + g - ghat, the memory recursion)
 * Readings where the paper is silent: NaN is sent as zero, +-Inf as the boundary level, both
 * counted in *n_nonfinite, and the memory of such an element restarts at 0; a finite value
 * beyond the boundary is counted in *n_saturated.
 * sym, ghat, v_out may be NULL.
 */
int co3o_convert(const float *g, float *m, float decay, const co3o_fmt *f, uint64_t n,
                 uint8_t *sym8, uint16_t *sym16, float *ghat, float *v_out,
                 uint64_t *n_saturated, uint64_t *n_nonfinite)
{
    if (!co3o_fmt_ok(f)) return CO3O_ERR_ARG;
    co3o_levels L;
    if (!co3o_levels_init(&L, f)) return CO3O_ERR_ARG;
    const int nb = f->exp_bits + f->mant_bits;
    uint64_t nsat = 0, nnf = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const float v = fmaf(decay, m[i], g[i]);
        uint32_t c, sign;
        int sat = 0;
        float gh, mnew;
        if (isnan(v)) {
            c = 0; sign = 0; nnf++;
            gh = 0.0f; mnew = 0.0f;
        } else {
            const float t = v * f->scale;
            c = co3o_nearest(&L, fabs((double)t), &sat);
            sign = (t < 0.0f && c != 0) ? 1u : 0u;
            float q = (float)co3o_level(f, c);
            if (sign) q = -q;
            gh = q * f->inv_scale;
            if (isinf(v)) { nnf++; mnew = 0.0f; }
            else { nsat += (uint64_t)sat; mnew = v - gh; }
        }
        const uint32_t s = (sign << nb) | c;
        if (sym8) sym8[i] = (uint8_t)s;
        if (sym16) sym16[i] = (uint16_t)s;
        if (ghat) ghat[i] = gh;
        if (v_out) v_out[i] = v;
        m[i] = mnew;
    }
    co3o_levels_free(&L);
    if (n_saturated) *n_saturated = nsat;
    if (n_nonfinite) *n_nonfinite = nnf;
    return CO3O_OK;
}

/* ------------------------------------------------------------------------------------------
 * Dithered conversion (Sec. II-B (ii): the quantizer may be a stochastic mapping, so that
 * non-subtractive dither quantization can be implemented).  Reading taken: the dither is uniform
 * over the step between the two levels around the scaled value, which is the same as choosing the
 * upper level with probability (|t| - lower) / (upper - lower): with R a uniform 24-bit integer,
 * the upper level is taken iff R < (|t| - lower) / (upper - lower) * 2^24.  Every step of the level
 * set is a power of two, so the right-hand side is exact in fp64; a value that is a level stays
 * where it is for every R, and averaged over all 2^24 values of R the result is the value itself
 * whenever that right-hand side is an integer (every fp32 value from the smallest normal level up).
 * Beyond the largest level the value saturates as before; NaN and infinities are treated as before.
 * The parameter server does not need the draws (the dither is not subtracted).
 *
 * The draws are inputs here.  co3o_dither_draws produces the ones the library uses: Philox-4x32
 * with 10 rounds (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC 2011),
 * key (seed, 0), counter (p / 4 low word, p / 4 high word, client, layer) for the element at place
 * p of its layer, output word p % 4, top 24 bits.
 * ------------------------------------------------------------------------------------------ */
void co3o_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; } /* key schedule: add the Weyl constants */
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void co3o_dither_draws(uint32_t seed, uint32_t client, uint32_t layer, uint64_t first_place, uint64_t n,
                       uint32_t *draws)
{
    const uint32_t key[2] = {seed, 0u};
    for (uint64_t i = 0; i < n; ++i) {
        const uint64_t p = first_place + i;
        const uint32_t ctr[4] = {(uint32_t)(p >> 2), (uint32_t)(p >> 34), client, layer};
        uint32_t out[4];
        co3o_philox4x32_10(ctr, key, out);
        draws[i] = out[p & 3u] >> 8;
    }
}

/* Magnitude code for a >= 0 under the draw R (0 <= R < 2^24). */
static uint32_t co3o_dithered(const co3o_levels *L, double a, uint32_t R, int *saturated)
{
    int lo = 0, hi = L->n - 1;
    *saturated = 0;
    if (a > L->level[hi]) {
        *saturated = 1;
        return L->code[hi];
    }
    while (lo < hi) { /* largest index with level <= a */
        const int mid = (lo + hi + 1) / 2;
        if (L->level[mid] <= a) lo = mid; else hi = mid - 1;
    }
    if (lo == L->n - 1 || a == L->level[lo]) return L->code[lo];
    const double where = (a - L->level[lo]) / (L->level[lo + 1] - L->level[lo]); /* in (0, 1), exact */
    return (double)R < where * 16777216.0 ? L->code[lo + 1] : L->code[lo];
}

/* co3o_convert with the nearest-level rule replaced by the dithered one; draws[i] in [0, 2^24). */
int co3o_convert_dithered(const float *g, float *m, float decay, const co3o_fmt *f, uint64_t n,
                          const uint32_t *draws, uint8_t *sym8, uint16_t *sym16, float *ghat,
                          uint64_t *n_saturated, uint64_t *n_nonfinite)
{
    if (!co3o_fmt_ok(f) || !draws) return CO3O_ERR_ARG;
    co3o_levels L;
    if (!co3o_levels_init(&L, f)) return CO3O_ERR_ARG;
    const int nb = f->exp_bits + f->mant_bits;
    uint64_t nsat = 0, nnf = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (draws[i] >> 24) { co3o_levels_free(&L); return CO3O_ERR_ARG; }
        const float v = fmaf(decay, m[i], g[i]);
        uint32_t c, sign;
        int sat = 0;
        float gh, mnew;
        if (isnan(v)) {
            c = 0; sign = 0; nnf++;
            gh = 0.0f; mnew = 0.0f;
        } else {
            const float t = v * f->scale;
            c = co3o_dithered(&L, fabs((double)t), draws[i], &sat);
            sign = (t < 0.0f && c != 0) ? 1u : 0u;
            float q = (float)co3o_level(f, c);
            if (sign) q = -q;
            gh = q * f->inv_scale;
            if (isinf(v)) { nnf++; mnew = 0.0f; }
            else { nsat += (uint64_t)sat; mnew = v - gh; }
        }
        const uint32_t s = (sign << nb) | c;
        if (sym8) sym8[i] = (uint8_t)s;
        if (sym16) sym16[i] = (uint16_t)s;
        if (ghat) ghat[i] = gh;
        m[i] = mnew;
    }
    co3o_levels_free(&L);
    if (n_saturated) *n_saturated = nsat;
    if (n_nonfinite) *n_nonfinite = nnf;
    return CO3O_OK;
}

/* Symbol statistics the code is fitted to (Sec. IV-A (ii): Huffman coding needs the source distribution). */
void co3o_histogram(const uint8_t *sym, uint64_t n, uint64_t hist[256])
{
    for (uint64_t i = 0; i < n; ++i) hist[sym[i]]++;
}

/* ------------------------------------------------------------------------------------------
 * Huffman code from integer weights (Sec. IV-A (ii); optimal prefix code for a known pmf).
 * Textbook construction: keep a pool of nodes, repeatedly remove the two of least weight and
 * put back their parent.  Order among equal weights (the paper fixes none): a leaf before a
 * merged node, leaves by symbol, merged nodes by age.  Every symbol the converter can emit
 * takes part with weight max(w, 1), so it always has a codeword.  If the deepest leaf exceeds
 * CO3O_MAX_CODE_LEN all weights are halved (never below 1) and the construction repeats: an
 * implementation limit, not in the paper; the result is still a complete prefix code.
 * Codewords are assigned canonically: symbols sorted by (length, symbol) get consecutive
 * values, shifted left whenever the length grows.
 * ------------------------------------------------------------------------------------------ */
int co3o_code_build(const uint64_t weights[256], const co3o_fmt *f, co3o_code *out)
{
    if (!co3o_fmt_ok(f) || 1 + f->exp_bits + f->mant_bits > 8) return CO3O_ERR_ARG;
    uint64_t w[256];
    int valid[256], nvalid = 0;
    uint64_t total = 0;
    for (int s = 0; s < 256; ++s) {
        valid[s] = co3o_symbol_valid(f, (uint32_t)s);
        w[s] = 0;
        if (valid[s]) {
            w[s] = weights[s] > 0 ? weights[s] : 1;
            if (w[s] > (UINT64_MAX >> 1) - total) return CO3O_ERR_ARG; /* sum must stay below 2^63 */
            total += w[s];
            nvalid++;
        }
    }
    memset(out, 0, sizeof(*out));
    if (nvalid < 2) return CO3O_ERR_ARG;

    int len[256];
    for (;;) {
        /* nodes 0..255 are leaves (by symbol), 256.. are merged nodes in order of creation */
        uint64_t nw[512];
        int parent[512], alive[512], nnodes = 256;
        for (int s = 0; s < 256; ++s) { nw[s] = w[s]; alive[s] = valid[s]; parent[s] = -1; }
        for (int k = 0; k < nvalid - 1; ++k) {
            int pick[2];
            for (int j = 0; j < 2; ++j) {
                int best = -1;
                for (int i = 0; i < nnodes; ++i) { /* index order = leaf-before-merged, symbol, age */
                    if (!alive[i]) continue;
                    if (best < 0 || nw[i] < nw[best]) best = i;
                }
                alive[best] = 0;
                pick[j] = best;
            }
            nw[nnodes] = nw[pick[0]] + nw[pick[1]];
            alive[nnodes] = 1;
            parent[nnodes] = -1;
            parent[pick[0]] = nnodes;
            parent[pick[1]] = nnodes;
            nnodes++;
        }
        int maxlen = 0;
        for (int s = 0; s < 256; ++s) {
            len[s] = 0;
            if (!valid[s]) continue;
            for (int p = parent[s]; p >= 0; p = parent[p]) len[s]++;
            if (len[s] > maxlen) maxlen = len[s];
        }
        if (maxlen <= CO3O_MAX_CODE_LEN) break;
        for (int s = 0; s < 256; ++s)
            if (valid[s]) w[s] = (w[s] >> 1) > 0 ? (w[s] >> 1) : 1;
    }

    /* canonical assignment */
    uint32_t next = 0;
    int prev_len = 0;
    for (int l = 1; l <= CO3O_MAX_CODE_LEN; ++l) {
        for (int s = 0; s < 256; ++s) {
            if (!valid[s] || len[s] != l) continue;
            if (prev_len) next = (next + 1u) << (l - prev_len);
            out->len[s] = (uint8_t)l;
            out->bits[s] = next;
            prev_len = l;
        }
    }
    return CO3O_OK;
}

/* ------------------------------------------------------------------------------------------
 * Container (the paper only says the codewords form a binary string b of length r; the layout
 * below is this implementation's, chosen so that a decoder can start at many places at once).
 * All fields little-endian.
 *   header, 64 bytes: u32 magic 'CO3S', u32 version 1, u32 n_seg, u32 chunk_syms C,
 *       u32 sub_syms S, u32 0, u64 n_elem, u64 n_chunks, u64 payload_words, u64 payload_bits,
 *       u64 total_bytes
 *   segment table, n_seg x { u64 n_elem, u64 first_chunk, u64 payload_bits }
 *   chunk table,   u64 word_off[n_chunks + 1]      (offset of each chunk in payload words)
 *   sub table,     u16 bit_off[n_chunks][C / S]    (bit offset of each run of S symbols in its chunk)
 *   payload,       u32 words[payload_words]
 * Each section starts on a 16-byte boundary and total_bytes is a multiple of 16.
 * A chunk is C consecutive symbols of one segment (the last chunk of a segment may be
 * shorter) and starts on a word boundary; its codewords are concatenated in element order,
 * h(ghat) "element-wise"; stream bit j of a chunk is bit 31 - (j mod 32) of word j / 32, the
 * first bit of a codeword being its most significant; unused bits of the last word are 0.
 * payload_bits is r, the sum of the codeword lengths; tables and padding are not part of it.
 * ------------------------------------------------------------------------------------------ */
#define CO3O_MAGIC 0x53334F43u
#define CO3O_HEADER_BYTES 64u

static uint64_t co3o_align16(uint64_t x) { return (x + 15u) & ~(uint64_t)15u; }

static void co3o_put32(uint8_t *p, uint32_t v) { for (int i = 0; i < 4; ++i) p[i] = (uint8_t)(v >> (8 * i)); }
static void co3o_put64(uint8_t *p, uint64_t v) { for (int i = 0; i < 8; ++i) p[i] = (uint8_t)(v >> (8 * i)); }
static void co3o_put16(uint8_t *p, uint32_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); }
static uint32_t co3o_get32(const uint8_t *p) { uint32_t v = 0; for (int i = 0; i < 4; ++i) v |= (uint32_t)p[i] << (8 * i); return v; }
static uint64_t co3o_get64(const uint8_t *p) { uint64_t v = 0; for (int i = 0; i < 8; ++i) v |= (uint64_t)p[i] << (8 * i); return v; }
static uint32_t co3o_get16(const uint8_t *p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8); }

typedef struct {
    uint64_t n_elem, n_chunks;
    uint64_t seg_off, chunk_off, sub_off, payload_off;
} co3o_layout;

static int co3o_layout_init(co3o_layout *lay, const uint64_t *seg_n_elem, uint32_t n_seg,
                            uint32_t C, uint32_t S)
{
    if (C == 0 || S == 0 || C % S != 0 || C % 32 != 0) return 0;
    if ((uint64_t)(C - S) * CO3O_MAX_CODE_LEN > 65535u) return 0; /* sub offsets are 16-bit */
    lay->n_elem = 0;
    lay->n_chunks = 0;
    for (uint32_t k = 0; k < n_seg; ++k) {
        lay->n_elem += seg_n_elem[k];
        lay->n_chunks += (seg_n_elem[k] + C - 1) / C;
    }
    lay->seg_off = CO3O_HEADER_BYTES;
    lay->chunk_off = co3o_align16(lay->seg_off + 24u * (uint64_t)n_seg);
    lay->sub_off = co3o_align16(lay->chunk_off + 8u * (lay->n_chunks + 1));
    lay->payload_off = co3o_align16(lay->sub_off + 2u * lay->n_chunks * (C / S));
    return 1;
}

/* Bytes a stream needs when every codeword has the maximum length. */
int co3o_stream_capacity_bytes(const uint64_t *seg_n_elem, uint32_t n_seg, uint32_t C, uint32_t S,
                               uint64_t *out)
{
    co3o_layout lay;
    if (!co3o_layout_init(&lay, seg_n_elem, n_seg, C, S)) return CO3O_ERR_ARG;
    uint64_t words = 0;
    for (uint32_t k = 0; k < n_seg; ++k) {
        const uint64_t n = seg_n_elem[k];
        for (uint64_t start = 0; start < n; start += C) {
            const uint64_t cnt = n - start < C ? n - start : C;
            words += (cnt * CO3O_MAX_CODE_LEN + 31) / 32;
        }
    }
    *out = co3o_align16(lay.payload_off + 4u * words);
    return CO3O_OK;
}

/*
 * b = h_Hf(ghat): encode the symbols of one client (all segments, one code per segment) into
 * a container.  Nothing is written beyond `capacity`.  *used receives total_bytes.
 */
int co3o_encode(const uint8_t *sym, const uint64_t *seg_n_elem, const co3o_code *codes, uint32_t n_seg,
                uint32_t C, uint32_t S, uint8_t *stream, uint64_t capacity, uint64_t *used)
{
    co3o_layout lay;
    if (!co3o_layout_init(&lay, seg_n_elem, n_seg, C, S)) return CO3O_ERR_ARG;
    if (lay.payload_off > capacity) return CO3O_ERR_CAPACITY;
    memset(stream, 0, lay.payload_off);

    const uint32_t subs = C / S;
    uint64_t word_pos = 0, chunk = 0, elem = 0, total_bits = 0;
    for (uint32_t k = 0; k < n_seg; ++k) {
        const co3o_code *code = &codes[k];
        uint64_t seg_bits = 0;
        co3o_put64(stream + lay.seg_off + 24u * k, seg_n_elem[k]);
        co3o_put64(stream + lay.seg_off + 24u * k + 8, chunk);
        for (uint64_t start = 0; start < seg_n_elem[k]; start += C, ++chunk) {
            const uint64_t cnt = seg_n_elem[k] - start < C ? seg_n_elem[k] - start : C;
            uint8_t *words = stream + lay.payload_off + 4u * word_pos;
            uint64_t bit = 0; /* bit position inside this chunk */
            co3o_put64(stream + lay.chunk_off + 8u * chunk, word_pos);
            for (uint64_t i = 0; i < cnt; ++i) {
                if (i % S == 0) co3o_put16(stream + lay.sub_off + 2u * (chunk * subs + i / S), (uint32_t)bit);
                const uint8_t s = sym[elem + start + i];
                const int l = code->len[s];
                if (l == 0) return CO3O_ERR_NO_CODEWORD;
                for (int b = l - 1; b >= 0; --b, ++bit) { /* most significant codeword bit first */
                    const uint64_t byte_off = lay.payload_off + 4u * (word_pos + bit / 32);
                    if (bit % 32 == 0) {
                        if (byte_off + 4 > capacity) return CO3O_ERR_CAPACITY;
                        co3o_put32(stream + byte_off, 0);
                    }
                    if ((code->bits[s] >> b) & 1u) {
                        uint8_t *wp = words + 4u * (bit / 32);
                        co3o_put32(wp, co3o_get32(wp) | (1u << (31 - bit % 32)));
                    }
                }
            }
            /* runs of S symbols that start at or beyond the end of a short chunk point at its end */
            for (uint64_t j = (cnt + S - 1) / S; j < subs; ++j)
                co3o_put16(stream + lay.sub_off + 2u * (chunk * subs + j), (uint32_t)bit);
            seg_bits += bit;
            word_pos += (bit + 31) / 32;
        }
        co3o_put64(stream + lay.seg_off + 24u * k + 16, seg_bits);
        total_bits += seg_bits;
        elem += seg_n_elem[k];
    }
    co3o_put64(stream + lay.chunk_off + 8u * chunk, word_pos);
    const uint64_t total_bytes = co3o_align16(lay.payload_off + 4u * word_pos);
    if (total_bytes > capacity) return CO3O_ERR_CAPACITY;
    memset(stream + lay.payload_off + 4u * word_pos, 0, total_bytes - (lay.payload_off + 4u * word_pos));
    co3o_put32(stream + 0, CO3O_MAGIC);
    co3o_put32(stream + 4, 1);
    co3o_put32(stream + 8, n_seg);
    co3o_put32(stream + 12, C);
    co3o_put32(stream + 16, S);
    co3o_put32(stream + 20, 0);
    co3o_put64(stream + 24, lay.n_elem);
    co3o_put64(stream + 32, lay.n_chunks);
    co3o_put64(stream + 40, word_pos);
    co3o_put64(stream + 48, total_bits);
    co3o_put64(stream + 56, total_bytes);
    if (used) *used = total_bytes;
    return CO3O_OK;
}

/* Prefix-code tree for decoding one bit at a time: child[node][bit], leaves hold ~symbol. */
typedef struct { int child[1024][2]; int n; } co3o_tree;

static int co3o_tree_init(co3o_tree *t, const co3o_code *code)
{
    t->n = 1;
    t->child[0][0] = t->child[0][1] = 0; /* 0 = absent (the root is never a child) */
    for (int s = 0; s < 256; ++s) {
        const int l = code->len[s];
        if (l == 0) continue;
        if (l > CO3O_MAX_CODE_LEN) return 0;
        int node = 0;
        for (int b = l - 1; b >= 0; --b) {
            const int bit = (int)((code->bits[s] >> b) & 1u);
            if (b == 0) {
                if (t->child[node][bit] != 0) return 0; /* not prefix-free */
                t->child[node][bit] = -(s + 1);
            } else {
                if (t->child[node][bit] < 0) return 0;
                if (t->child[node][bit] == 0) {
                    if (t->n >= 1024) return 0;
                    t->child[t->n][0] = t->child[t->n][1] = 0;
                    t->child[node][bit] = t->n++;
                }
                node = t->child[node][bit];
            }
        }
    }
    return 1;
}

/*
 * The inverse of co3o_encode for one client: recover every symbol (and, if ghat is not NULL,
 * the value the parameter server reconstructs).  The stream must describe exactly the given
 * segments; any inconsistency (bad header, offsets that do not match the decoded lengths,
 * a bit pattern that is no codeword, reading past the chunk) returns CO3O_ERR_CORRUPT.
 */
int co3o_decode(const uint8_t *stream, uint64_t stream_bytes, const uint64_t *seg_n_elem,
                const co3o_fmt *fmts, const co3o_code *codes, uint32_t n_seg, uint32_t C, uint32_t S,
                uint8_t *sym_out, float *ghat)
{
    co3o_layout lay;
    if (!co3o_layout_init(&lay, seg_n_elem, n_seg, C, S)) return CO3O_ERR_ARG;
    if (stream_bytes < lay.payload_off) return CO3O_ERR_CORRUPT;
    if (co3o_get32(stream) != CO3O_MAGIC || co3o_get32(stream + 4) != 1 || co3o_get32(stream + 8) != n_seg ||
        co3o_get32(stream + 12) != C || co3o_get32(stream + 16) != S || co3o_get64(stream + 24) != lay.n_elem ||
        co3o_get64(stream + 32) != lay.n_chunks)
        return CO3O_ERR_CORRUPT;
    const uint64_t payload_words = co3o_get64(stream + 40);
    if (co3o_get64(stream + 56) > stream_bytes) return CO3O_ERR_CORRUPT;
    if (payload_words > (stream_bytes - lay.payload_off) / 4) return CO3O_ERR_CORRUPT;
    if (co3o_get64(stream + lay.chunk_off + 8u * lay.n_chunks) != payload_words) return CO3O_ERR_CORRUPT;

    const uint32_t subs = C / S;
    uint64_t chunk = 0, elem = 0, total_bits = 0;
    co3o_tree *tree = (co3o_tree *)malloc(sizeof(co3o_tree));
    if (!tree) return CO3O_ERR_ARG;
    int status = CO3O_OK;
    for (uint32_t k = 0; k < n_seg && status == CO3O_OK; ++k) {
        if (!co3o_tree_init(tree, &codes[k])) { status = CO3O_ERR_ARG; break; }
        if (co3o_get64(stream + lay.seg_off + 24u * k) != seg_n_elem[k] ||
            co3o_get64(stream + lay.seg_off + 24u * k + 8) != chunk) { status = CO3O_ERR_CORRUPT; break; }
        uint64_t seg_bits = 0;
        for (uint64_t start = 0; start < seg_n_elem[k] && status == CO3O_OK; start += C, ++chunk) {
            const uint64_t cnt = seg_n_elem[k] - start < C ? seg_n_elem[k] - start : C;
            const uint64_t w0 = co3o_get64(stream + lay.chunk_off + 8u * chunk);
            const uint64_t w1 = co3o_get64(stream + lay.chunk_off + 8u * (chunk + 1));
            if (w0 > w1 || w1 > payload_words) { status = CO3O_ERR_CORRUPT; break; }
            const uint64_t avail = (w1 - w0) * 32;
            uint64_t bit = 0;
            for (uint64_t i = 0; i < cnt; ++i) {
                if (i % S == 0 && co3o_get16(stream + lay.sub_off + 2u * (chunk * subs + i / S)) != bit) {
                    status = CO3O_ERR_CORRUPT; break;
                }
                int node = 0;
                for (;;) {
                    if (bit >= avail) { status = CO3O_ERR_CORRUPT; break; }
                    const uint32_t word = co3o_get32(stream + lay.payload_off + 4u * (w0 + bit / 32));
                    const int b = (int)((word >> (31 - bit % 32)) & 1u);
                    ++bit;
                    node = tree->child[node][b];
                    if (node == 0) { status = CO3O_ERR_CORRUPT; break; }
                    if (node < 0) break;
                }
                if (status != CO3O_OK) break;
                const uint32_t s = (uint32_t)(-node - 1);
                if (sym_out) sym_out[elem + start + i] = (uint8_t)s;
                if (ghat) ghat[elem + start + i] = co3o_symbol_value(&fmts[k], s);
            }
            if (status != CO3O_OK) break;
            if ((bit + 31) / 32 != w1 - w0) { status = CO3O_ERR_CORRUPT; break; }
            seg_bits += bit;
        }
        if (status == CO3O_OK && co3o_get64(stream + lay.seg_off + 24u * k + 16) != seg_bits) status = CO3O_ERR_CORRUPT;
        total_bits += seg_bits;
        elem += seg_n_elem[k];
    }
    free(tree);
    if (status == CO3O_OK && co3o_get64(stream + 48) != total_bits) status = CO3O_ERR_CORRUPT;
    return status;
}

/*
 * Parameter-server side (Sec. II-B (iv)): decode every client's stream and form
 * (1/U) * sum_u ghat^(u) per element: fp32 additions in client order starting from 0, then one
 * fp32 division by U.  (The learning-rate step of Algorithm 1 is the caller's.)
 * scratch must hold n_elem floats.
 */
int co3o_decode_aggregate(const uint8_t *const *streams, const uint64_t *stream_bytes, uint32_t n_clients,
                          const uint64_t *seg_n_elem, const co3o_fmt *fmts, const co3o_code *codes,
                          uint32_t n_seg, uint32_t C, uint32_t S, float *avg, float *scratch)
{
    uint64_t n = 0;
    for (uint32_t k = 0; k < n_seg; ++k) n += seg_n_elem[k];
    if (n_clients == 0) return CO3O_ERR_ARG;
    for (uint64_t i = 0; i < n; ++i) avg[i] = 0.0f;
    for (uint32_t u = 0; u < n_clients; ++u) {
        const int st = co3o_decode(streams[u], stream_bytes[u], seg_n_elem, fmts, codes, n_seg, C, S, NULL, scratch);
        if (st != CO3O_OK) return st;
        for (uint64_t i = 0; i < n; ++i) avg[i] = avg[i] + scratch[i];
    }
    const float U = (float)n_clients;
    for (uint64_t i = 0; i < n; ++i) avg[i] = avg[i] / U;
    return CO3O_OK;
}

/*
 * Model update at the parameter server (Algorithm 1, last step; Sec. II-B (iv)):
 * w <- w - eta * avg with avg = (1/U) * sum_u ghat^(u) as co3o_decode_aggregate forms it.
 * Per element one fp32 multiplication and one fp32 subtraction, each rounded on its own.
 */
void co3o_ps_update(float *w, const float *avg, float eta, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i) {
        const float step = eta * avg[i];
        w[i] = w[i] - step;
    }
}

/*
 * Fitting the converter's multiplier to a layer (Sec. III: the gradients of a layer are modelled as
 * zero-mean generalized normal, GenNorm(0, alpha, beta); Sec. IV-A (i) and Eq. (exp bias): the multiplier
 * minimises the expected squared conversion error under that model).
 *
 * Kurtosis of GenNorm as a function of the shape: Gamma(5/b) Gamma(1/b) / Gamma(3/b)^2 (Sec. III).
 */
double co3o_gennorm_kurtosis(double beta)
{
    return exp(lgamma(5.0 / beta) + lgamma(1.0 / beta) - 2.0 * lgamma(3.0 / beta));
}

/* Shape whose kurtosis is `kurt`, searched in [lo, hi] (the kurtosis falls as the shape grows); values
 * outside the range of the interval's ends give the nearer end. */
double co3o_gennorm_shape_from_kurtosis(double kurt, double lo, double hi)
{
    if (!(kurt < co3o_gennorm_kurtosis(lo))) return lo;
    if (!(kurt > co3o_gennorm_kurtosis(hi))) return hi;
    for (int it = 0; it < 200 && hi - lo > 1e-15 * hi; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (co3o_gennorm_kurtosis(mid) > kurt) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

/*
 * One layer: moments of v = g + decay * m (m may be NULL: v = g) over the n_clients vectors of n elements
 * each (client u at g + u * stride), all of which share the layer's format; from them
 *   sigma^2 = sum v^2 / N,  kurtosis = N * sum v^4 / (sum v^2)^2  (zero mean: the model's location is 0),
 *   beta  = shape with that kurtosis, kept inside the table's range,
 *   alpha = sigma * sqrt(Gamma(1/beta) / Gamma(3/beta))        (variance of GenNorm, Sec. III),
 *   scale = exp(interp(beta; log_tab)) / alpha, inv_scale = 1 / scale (fp32),
 * where log_tab[i] is the natural logarithm of the best multiplier for unit alpha at shape
 * beta0 + i * dbeta (the numerical minimiser of the conversion error, tabulated by the caller) and the
 * interpolation is linear in the logarithm.  stats (nullable) receives sigma, kurtosis, beta, alpha.
 * Returns 0, or CO3O_ERR_ARG when the layer is empty, all zero or holds a non-finite value (nothing is
 * written then).
 */
int co3o_fit_scale(const float *g, const float *m, float decay, uint64_t n, uint32_t n_clients, uint64_t stride,
                   const float *log_tab, uint32_t n_beta, float beta0, float dbeta,
                   float *scale, float *inv_scale, double *stats)
{
    double s2 = 0.0, s4 = 0.0;
    for (uint32_t u = 0; u < n_clients; ++u) {
        for (uint64_t i = 0; i < n; ++i) {
            const float gv = g[u * stride + i];
            const float v = m ? fmaf(decay, m[u * stride + i], gv) : gv;
            const double x2 = (double)v * (double)v;
            s2 += x2;
            s4 += x2 * x2;
        }
    }
    const double N = (double)n * (double)n_clients;
    if (n_beta < 2 || !(N > 0.0) || !(s2 > 0.0) || !isfinite(s2) || !isfinite(s4)) return CO3O_ERR_ARG;
    const double sigma = sqrt(s2 / N), kurt = N * s4 / (s2 * s2);
    const double blo = (double)beta0, bhi = (double)beta0 + (double)dbeta * (double)(n_beta - 1);
    const double beta = co3o_gennorm_shape_from_kurtosis(kurt, blo, bhi);
    const double alpha = sigma * sqrt(exp(lgamma(1.0 / beta) - lgamma(3.0 / beta)));
    double x = (beta - blo) / (double)dbeta;
    if (x < 0.0) x = 0.0;
    uint32_t i = (uint32_t)x;
    if (i > n_beta - 2) i = n_beta - 2;
    const double f = x - (double)i;
    const double log_s = (double)log_tab[i] + f * ((double)log_tab[i + 1] - (double)log_tab[i]);
    const float sc = (float)(exp(log_s) / alpha);
    if (!(sc > 0.0f) || isinf(sc)) return CO3O_ERR_ARG;
    *scale = sc;
    *inv_scale = 1.0f / sc;
    if (stats) { stats[0] = sigma; stats[1] = kurt; stats[2] = beta; stats[3] = alpha; }
    return CO3O_OK;
}

/*
 * Error magnitude (Sec. VI, "Error magnitude"): the size of the memory term against the size of the gradient
 * term, both as l1 norms, the quantity by which the memory decay gamma is chosen.  One layer of one client:
 * norms[0] = sum |g_i|, norms[1] = sum |m_i|, added in fp64 in element order.  A NaN anywhere gives NaN.
 */
void co3o_error_magnitude(const float *g, const float *m, uint64_t n, double *norms)
{
    double sg = 0.0, sm = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        sg += fabs((double)g[i]);
        sm += fabs((double)m[i]);
    }
    norms[0] = sg;
    norms[1] = sm;
}
