/*
 * nuq_oracle.c -- plain, slow CPU oracle for the NUQSGD codec hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the reference the CUDA kernels are
 * checked against.  It shares no code, header, table or constant generator
 * with the CUDA path and must never be linked into, imported by or called from
 * the product library; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may use it.
 *
 * What it computes (paper = NUQSGD, arXiv 1908.06077):
 *   - level set                L = (0, 2^-s, ..., 1/2, 1)        Sec. 3.1
 *   - stochastic quantizer     Q_s, Definition 1, with the explicit
 *                              probabilities p_1, p_2 of App. B (Eq. h_case1/2)
 *   - Elias recursive coding   Algorithm 2 (App. A)
 *   - ENCODE / DECODE          App. A, applied per bucket (Sec. 5)
 *   - aggregate  sum_i g^_i    Algorithm 1, aggregation line (without alpha/K)
 *   - the aggregation step     w <- w - (alpha/K) sum_i g^_i  (Algorithm 1, aggregation line, Omega = R^d)
 *                              and its momentum form (Sec. 4, "NUQSGD with momentum", the rule y, y^l, w)
 *   - closed-form variance     Lemma 7 / Eq. (genvar)
 *   - uniform level set k/2^s  (QSGD / QSGDinf comparison, Sec. 1 and 3)
 *   - arbitrary level sequences L = (0, l_1, ..., l_s, 1), e.g. L_p = (0, p^s, ..., p, 1)
 *                              (Sec. 3.3, "general level sequences"), given as a table
 *   - coded level indices      the level index of a token written with a Huffman code fitted on
 *                              a histogram of level indices and then kept (Sec. 5, "efficient
 *                              encoding": the variant the paper calls encoded NUQSGD)
 *
 * Everything the paper leaves open (bucket tail, fp32 arithmetic order, random
 * generator, container layout) is fixed here in the most literal form; the
 * repository's design notes list each such reading.
 *
 * Arithmetic: norms are accumulated in fp64 in index order and rounded once to
 * fp32; the quantizer works in IEEE fp32 without contraction (build with
 * -ffp-contract=off); the bit stream is written and read one bit at a time.
 *
 * Parity pins (tests marked "not gpu"): level closed form, Algorithm 2 code
 * words executed by hand, exact rounding probabilities by enumerating every
 * 24-bit draw, unbiasedness by full enumeration on tiny vectors and by Monte
 * Carlo, Lemma 7 closed form against the Theorem 4 / Theorem 12 worked
 * examples, Theorem 1 and Lemma 10 bounds, round trip, Philox against the
 * cuRAND host generator; for level tables: the levels of L_p from exact
 * fractions, rounding probabilities by enumeration against exact rational
 * arithmetic, unbiasedness by enumeration, Lemma 7 on hand-worked vectors;
 * for coded level indices: code lengths of hand-worked trees, least cost among
 * all prefix codes by brute force, the Kraft sum, canonical code words listed
 * by hand, a hand-assembled container, the same symbols as the ERC mode;
 * for the aggregation step: steps worked by hand, heavy-ball and Nesterov
 * iterations written in their velocity forms, a fixed point.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_CAPACITY (-2)
#define ORC_ERR_STREAM (-3)

#define ORC_MAGIC 0x3151554Eu /* bytes 'N','U','Q','1' */
#define ORC_VERSION 1u
#define ORC_SB 256u                /* elements per coding sub-block            */
#define ORC_BLK (32u * ORC_SB)     /* elements per coding block (32 sub-blocks) */
#define ORC_HEADER_WORDS 16u

enum { NORM_L2 = 0, NORM_LINF = 1 };
enum { LEVELS_EXP = 0, LEVELS_UNIFORM = 1, LEVELS_TABLE = 2 };
#define ORC_MAX_S 14u
enum { MODE_ERC = 0, MODE_FIXED = 1, MODE_CODED = 2 };
#define ORC_MAX_CODED_S 7u         /* coded level indices: at most 8 symbols, code words of at most 7 bits */

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw 2011).                    */
/* ------------------------------------------------------------------ */
void nuq_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(prod1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)prod1;
        uint32_t n2 = (uint32_t)(prod0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)prod0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit word that element i of a call draws: one Philox block serves four
 * consecutive elements; key = seed, counter = (i/4, offset).                  */
uint32_t nuq_oracle_draw_word(uint64_t seed, uint64_t offset, uint64_t i) {
    uint64_t q = i >> 2;
    uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), (uint32_t)offset, (uint32_t)(offset >> 32)};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    nuq_oracle_philox4x32_10(ctr, key, out);
    return out[i & 3];
}

/* u in [0,1): the top 24 bits of the word, exactly representable in fp32. */
float nuq_oracle_draw_uniform(uint64_t seed, uint64_t offset, uint64_t i) {
    return (float)(nuq_oracle_draw_word(seed, offset, i) >> 8) * (1.0f / 16777216.0f);
}

/* ------------------------------------------------------------------ */
/* Level sets.                                                          */
/* ------------------------------------------------------------------ */
/* The level table of LEVELS_TABLE (Sec. 3.3): l_0 = 0 < l_1 < ... < l_s < l_{s+1} = 1 in fp32, and
 * 1 / (l_{j+1} - l_j) in fp32 (one IEEE division each), which the quantizer multiplies by.            */
typedef struct { uint32_t s; float level[ORC_MAX_S + 2]; float inv_width[ORC_MAX_S + 2]; } level_table;
static level_table g_table;

static int make_table(const float* interior, uint32_t s, level_table* t) {
    if (s < 1 || s > ORC_MAX_S) return ORC_ERR_ARG;
    t->s = s;
    t->level[0] = 0.0f;
    for (uint32_t j = 1; j <= s; ++j) t->level[j] = interior[j - 1];
    t->level[s + 1] = 1.0f;
    for (uint32_t j = 0; j <= s; ++j) {
        if (!(t->level[j] < t->level[j + 1])) return ORC_ERR_ARG;          /* strictly increasing, no NaN */
        t->inv_width[j] = 1.0f / (t->level[j + 1] - t->level[j]);
        if (isinf(t->inv_width[j])) return ORC_ERR_ARG;
    }
    t->inv_width[s + 1] = 0.0f;
    return ORC_OK;
}

/* the interior levels l_1 .. l_s that LEVELS_TABLE calls use from now on */
int nuq_oracle_set_levels(const float* interior, uint32_t s) { return make_table(interior, s, &g_table); }

/* ------------------------------------------------------------------ */
/* Coded level indices (Sec. 5, "efficient encoding").  The paper says only that a Huffman code
 * is fitted on an initial sample and then kept.  Fixed here: the symbols are the level indices
 * 1..s+1 of the nonzero coordinates; the tree is built by joining, n - 1 times, the two nodes
 * of least weight, where among nodes of equal weight a leaf goes before a joined node, leaves
 * go by index and joined nodes by age; only the code lengths are taken from the tree, and the
 * code words are the canonical ones for those lengths (symbols ordered by length, then index;
 * the first word is all zeros, each next word is the previous plus one, extended with zeros). */
typedef struct { uint32_t n; uint8_t len[ORC_MAX_CODED_S + 1]; uint32_t word[ORC_MAX_CODED_S + 1]; } level_code;
static level_code g_code;

int nuq_oracle_huffman_lengths(const uint64_t* weight, uint32_t n, uint8_t* len) {
    if (n < 2 || n > ORC_MAX_CODED_S + 1) return ORC_ERR_ARG;
    uint64_t w[2 * (ORC_MAX_CODED_S + 1)];
    int parent[2 * (ORC_MAX_CODED_S + 1)], open[2 * (ORC_MAX_CODED_S + 1)];
    uint32_t nodes = n;
    for (uint32_t i = 0; i < n; ++i) { w[i] = weight[i]; parent[i] = -1; open[i] = 1; }
    for (uint32_t join = 0; join + 1 < n; ++join) {
        int pick[2];
        for (int k = 0; k < 2; ++k) {                        /* least weight; the lowest node number among equals */
            int best = -1;
            for (uint32_t i = 0; i < nodes; ++i)
                if (open[i] && (best < 0 || w[i] < w[best])) best = (int)i;
            open[best] = 0;
            pick[k] = best;
        }
        w[nodes] = w[pick[0]] + w[pick[1]];
        parent[nodes] = -1; open[nodes] = 1;
        parent[pick[0]] = parent[pick[1]] = (int)nodes;
        ++nodes;
    }
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t depth = 0;
        for (int at = (int)i; parent[at] >= 0; at = parent[at]) ++depth;
        len[i] = (uint8_t)depth;
    }
    return ORC_OK;
}

static int make_code(const uint8_t* len, uint32_t n, level_code* c) {
    if (n < 2 || n > ORC_MAX_CODED_S + 1) return ORC_ERR_ARG;
    uint32_t kraft = 0;                                      /* in units of 2^-7 */
    for (uint32_t i = 0; i < n; ++i) {
        if (len[i] < 1 || len[i] > ORC_MAX_CODED_S) return ORC_ERR_ARG;
        kraft += 1u << (ORC_MAX_CODED_S - len[i]);
    }
    if (kraft > (1u << ORC_MAX_CODED_S)) return ORC_ERR_ARG; /* no prefix code has these lengths */
    c->n = n;
    uint32_t next = 0, prev_len = 0;
    for (uint32_t l = 1; l <= ORC_MAX_CODED_S; ++l)
        for (uint32_t i = 0; i < n; ++i) {
            if (len[i] != l) continue;
            next <<= (l - prev_len);
            prev_len = l;
            c->len[i] = (uint8_t)l;
            c->word[i] = next++;
        }
    return ORC_OK;
}

/* lengths[j-1] = code length of level index j, j = 1..s+1 */
int nuq_oracle_set_level_code(const uint8_t* lengths, uint32_t s) {
    if (s < 1 || s > ORC_MAX_CODED_S) return ORC_ERR_ARG;
    return make_code(lengths, s + 1, &g_code);
}

/* the code word of level index j under the code last set, one bit per byte; returns its length */
uint32_t nuq_oracle_level_code(uint32_t j, uint8_t* bits) {
    if (j < 1 || j > g_code.n) return 0;
    uint32_t l = g_code.len[j - 1];
    for (uint32_t k = 0; k < l; ++k) bits[k] = (uint8_t)((g_code.word[j - 1] >> (l - 1 - k)) & 1u);
    return l;
}

/* number of levels including 0 and 1 */
uint32_t nuq_oracle_num_levels(uint32_t levelset, uint32_t s) {
    return levelset == LEVELS_UNIFORM ? (1u << s) + 1u : s + 2u;
}

/* value of level `sym` as an fp64 number (exact) */
double nuq_oracle_level_value(uint32_t levelset, uint32_t s, uint32_t sym) {
    if (sym == 0) return 0.0;
    if (levelset == LEVELS_TABLE) return sym <= g_table.s + 1 ? (double)g_table.level[sym] : 1.0;
    if (levelset == LEVELS_EXP) return ldexp(1.0, (int)sym - 1 - (int)s); /* l_j = 2^(j-1-s) */
    return ldexp((double)sym, -(int)s);                                    /* l_k = k / 2^s   */
}

/* bits per element in the fixed-width mode: one sign bit plus the index */
uint32_t nuq_oracle_fixed_width(uint32_t levelset, uint32_t s) {
    uint32_t nlev = nuq_oracle_num_levels(levelset, s), b = 0;
    while ((1u << b) < nlev) ++b;
    return b + 1u;
}

static uint32_t float_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_float(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* ------------------------------------------------------------------ */
/* Bucket norm (Euclidean norm of Sec. 2; max-abs for the QSGDinf case).*/
/* ------------------------------------------------------------------ */
float nuq_oracle_norm(const float* v, uint64_t n, uint32_t norm_kind) {
    if (norm_kind == NORM_LINF) {
        float m = 0.0f;
        for (uint64_t i = 0; i < n; ++i) {
            float a = fabsf(v[i]);
            if (a != a) return bits_float(0x7FC00000u);   /* NaN poisons the bucket */
            if (a > m) m = a;
        }
        return m;
    }
    double acc = 0.0;
    for (uint64_t i = 0; i < n; ++i) acc += (double)v[i] * (double)v[i];
    if (acc != acc) return bits_float(0x7FC00000u);       /* one NaN pattern, whatever the payloads were */
    return (float)sqrt(acc);
}

void nuq_oracle_bucket_norms(const float* g, uint64_t d, uint32_t bucket, uint32_t norm_kind, float* norms) {
    uint64_t nb = (d + bucket - 1) / bucket;
    for (uint64_t b = 0; b < nb; ++b) {
        uint64_t lo = b * (uint64_t)bucket, hi = lo + bucket < d ? lo + bucket : d;
        norms[b] = nuq_oracle_norm(g + lo, hi - lo, norm_kind);
    }
}

/* A bucket is quantized only when 2^s / norm (for a level table: 1 / norm) is a finite positive number. */
static int bucket_is_live(float norm, uint32_t s, uint32_t levelset, float* inv_out) {
    if (!(norm > 0.0f) || isinf(norm)) return 0;
    float inv = (levelset == LEVELS_TABLE ? 1.0f : ldexpf(1.0f, (int)s)) / norm;   /* one IEEE division per bucket */
    if (isinf(inv) || inv != inv) return 0;
    *inv_out = inv;
    return 1;
}

/* ------------------------------------------------------------------ */
/* Definition 1 for one coordinate.  y = 2^s * r in fp32.               */
/*   exponential levels: r in [0, 2^-s]      -> p_1 = 2^s r             */
/*                       r in [2^(j-s), 2^(j+1-s)] -> p_2 = 2^(s-j) r - 1*/
/*   uniform levels:     p = y - floor(y)                                */
/* The coordinate moves to the upper level iff u < p.                    */
/* ------------------------------------------------------------------ */
static void split_coordinate(float v, float inv, uint32_t s, uint32_t levelset, uint32_t* low, float* p) {
    if (levelset == LEVELS_TABLE) {
        /* general level sequence (Sec. 3.3): r = |v| / norm, l_j <= r < l_{j+1},
         * p = (r - l_j) / (l_{j+1} - l_j), all in fp32 */
        float r = fabsf(v) * inv;
        if (!(r < 1.0f)) r = 1.0f;    /* r > 1 can only come from norm rounding */
        uint32_t j = 0;
        while (j <= s && g_table.level[j + 1] <= r) ++j;
        *low = j;
        *p = (r - g_table.level[j]) * g_table.inv_width[j];   /* 0 at the top level */
        return;
    }
    float top = ldexpf(1.0f, (int)s);
    float y = fabsf(v) * inv;
    if (!(y < top)) y = top;          /* r > 1 can only come from norm rounding */
    if (levelset == LEVELS_EXP) {
        if (y < 1.0f) {
            *low = 0; *p = y;
        } else {
            int ex;
            (void)frexpf(y, &ex);      /* y = m * 2^ex, m in [0.5,1) */
            int e = ex - 1;             /* floor(log2 y) */
            if (e > (int)s - 1) e = (int)s - 1;
            *low = (uint32_t)e + 1u;
            *p = ldexpf(y, -e) - 1.0f;  /* exact */
        }
    } else {
        float fl = floorf(y);
        if (fl > top - 1.0f) fl = top - 1.0f;
        *low = (uint32_t)fl;
        *p = y - fl;                    /* exact */
    }
}

static uint32_t quantize_coordinate(float v, float inv, uint32_t s, uint32_t levelset, float u) {
    uint32_t low;
    float p;
    split_coordinate(v, inv, s, levelset, &low, &p);
    return low + (u < p ? 1u : 0u);
}

/* lower level index and probability of moving up, for the pins */
void nuq_oracle_round_probability(float v, float norm, uint32_t s, uint32_t levelset, uint32_t* low, float* p) {
    float inv;
    if (!bucket_is_live(norm, s, levelset, &inv)) { *low = 0; *p = 0.0f; return; }
    split_coordinate(v, inv, s, levelset, low, p);
}

/* Quantize `n` coordinates of one bucket whose first element has index i0 in
 * the call.  sign[i] = 1 for a negative coordinate that quantizes to a nonzero
 * level (0 otherwise); sym[i] = level index.                                  */
void nuq_oracle_quantize_bucket(const float* v, uint64_t n, float norm, uint32_t s, uint32_t levelset,
                                uint64_t seed, uint64_t offset, uint64_t i0, uint8_t* sign, uint16_t* sym) {
    float inv;
    if (!bucket_is_live(norm, s, levelset, &inv)) {
        for (uint64_t i = 0; i < n; ++i) { sign[i] = 0; sym[i] = 0; }
        return;
    }
    for (uint64_t i = 0; i < n; ++i) {
        float u = nuq_oracle_draw_uniform(seed, offset, i0 + i);
        uint32_t q = quantize_coordinate(v[i], inv, s, levelset, u);
        sym[i] = (uint16_t)q;
        sign[i] = (uint8_t)((q != 0 && signbit(v[i])) ? 1 : 0);
    }
}

/* Same, but the uniform draws are supplied (for exhaustive / Monte-Carlo pins) */
void nuq_oracle_quantize_with_draws(const float* v, uint64_t n, float norm, uint32_t s, uint32_t levelset,
                                    const float* u, uint8_t* sign, uint16_t* sym) {
    float inv;
    int live = bucket_is_live(norm, s, levelset, &inv);
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t q = live ? quantize_coordinate(v[i], inv, s, levelset, u[i]) : 0u;
        sym[i] = (uint16_t)q;
        sign[i] = (uint8_t)((q != 0 && signbit(v[i])) ? 1 : 0);
    }
}

/* Q_s(v_i) = ||v|| * sign(v_i) * h_i  in fp32 */
float nuq_oracle_dequantize(float norm, uint32_t s, uint32_t levelset, uint32_t sign, uint32_t sym) {
    if (sym == 0) return 0.0f;
    float level = (float)nuq_oracle_level_value(levelset, s, sym); /* exact in fp32 */
    float q = norm * level;
    return sign ? -q : q;
}

/* whole vector: quantize then dequantize (no coding) */
void nuq_oracle_quantize_dequantize(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind,
                                    uint32_t levelset, uint64_t seed, uint64_t offset, float* out) {
    uint8_t* sg = (uint8_t*)malloc(bucket);
    uint16_t* sy = (uint16_t*)malloc(2u * (size_t)bucket);
    for (uint64_t lo = 0; lo < d; lo += bucket) {
        uint64_t n = lo + bucket < d ? bucket : d - lo;
        float norm = nuq_oracle_norm(g + lo, n, norm_kind);
        nuq_oracle_quantize_bucket(g + lo, n, norm, s, levelset, seed, offset, lo, sg, sy);
        for (uint64_t i = 0; i < n; ++i) out[lo + i] = nuq_oracle_dequantize(norm, s, levelset, sg[i], sy[i]);
    }
    free(sg); free(sy);
}

/* Lemma 7:  E||Q(v)-v||^2 = ||v||^2 sum_i (l_{j+1} - r_i)(r_i - l_j), fp64, for
 * one bucket with the given norm.                                            */
double nuq_oracle_variance_closed_form(const float* v, uint64_t n, float norm, uint32_t s, uint32_t levelset) {
    if (!(norm > 0.0f) || isinf(norm)) return 0.0;
    uint32_t nlev = nuq_oracle_num_levels(levelset, s);
    double total = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double r = fabs((double)v[i]) / (double)norm;
        if (r > 1.0) r = 1.0;
        uint32_t j = 0;
        while (j + 2 < nlev && nuq_oracle_level_value(levelset, s, j + 1) <= r) ++j;
        double lo = nuq_oracle_level_value(levelset, s, j), hi = nuq_oracle_level_value(levelset, s, j + 1);
        total += (hi - r) * (r - lo);
    }
    return total * (double)norm * (double)norm;
}

/* ------------------------------------------------------------------ */
/* Elias recursive coding, Algorithm 2.  Bits are held one per byte.    */
/* ------------------------------------------------------------------ */
static uint32_t bit_length(uint64_t n) { uint32_t b = 0; while (n) { ++b; n >>= 1; } return b; }

/* returns the number of bits written to `bits` (capacity must be >= 128) */
uint32_t nuq_oracle_erc_encode(uint64_t N, uint8_t* bits) {
    uint8_t tmp[160];
    int pos = 160;
    tmp[--pos] = 0;                          /* place a 0 at the end of the string */
    while (N > 1) {
        uint32_t nb = bit_length(N);
        for (uint32_t i = 0; i < nb; ++i) tmp[--pos] = (uint8_t)((N >> i) & 1u);  /* prepend binary(N) */
        N = nb - 1;                          /* N' = bits prepended minus 1 */
    }
    uint32_t len = (uint32_t)(160 - pos);
    memcpy(bits, tmp + pos, len);
    return len;
}

/* decodes one integer starting at bits[*pos]; returns 0 on overrun */
uint64_t nuq_oracle_erc_decode(const uint8_t* bits, uint64_t nbits, uint64_t* pos) {
    uint64_t N = 1;
    for (;;) {
        if (*pos >= nbits) return 0;
        if (bits[*pos] == 0) { ++*pos; return N; }
        if (N + 1 > 64 || *pos + N + 1 > nbits) return 0;
        uint64_t v = 0;
        for (uint64_t i = 0; i <= N; ++i) v = (v << 1) | bits[*pos + i];   /* that bit plus N following */
        *pos += N + 1;
        N = v;
    }
}

/* ------------------------------------------------------------------ */
/* Container.                                                           */
/*   u32 words, little endian.  Bit p of a bit string sits in word p>>5 */
/*   at bit 31-(p&31): words read like the paper's strings.             */
/*   [16-word header]                                                   */
/*   ERC mode:   [(nblk+1) u64 block bit offsets from payload start]    */
/*               per block (<= 8192 elements of one bucket):            */
/*                 norm word | u16 token-bit length per 256-element     */
/*                 sub-block, padded to a word | token strings of the   */
/*                 sub-blocks back to back | zero padding to a word     */
/*   fixed mode: per bucket: norm word | fields of w bits, MSB first,   */
/*               zero padded to a word; no table                        */
/* ------------------------------------------------------------------ */
static void put_bit(uint32_t* words, uint64_t p, uint32_t b) {
    if (b) words[p >> 5] |= 1u << (31u - (uint32_t)(p & 31u));
}
static uint32_t get_bit(const uint32_t* words, uint64_t p) {
    return (words[p >> 5] >> (31u - (uint32_t)(p & 31u))) & 1u;
}

static uint64_t count_blocks(uint64_t d, uint32_t bucket) {
    uint64_t nb = (d + bucket - 1) / bucket;
    uint64_t per = ((uint64_t)bucket + ORC_BLK - 1) / ORC_BLK;
    uint64_t last = d - (nb - 1) * (uint64_t)bucket;
    return (nb - 1) * per + (last + ORC_BLK - 1) / ORC_BLK;
}

/* longest ERC code of a level index, for the capacity bound */
static uint32_t max_level_code_bits(uint32_t levelset, uint32_t s, uint32_t mode) {
    uint8_t tmp[160];
    if (mode == MODE_CODED) return ORC_MAX_CODED_S;
    uint32_t nlev = nuq_oracle_num_levels(levelset, s), best = 0;
    for (uint32_t j = 1; j < nlev; ++j) { uint32_t l = nuq_oracle_erc_encode(j, tmp); if (l > best) best = l; }
    return best;
}

static int check_args(uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, uint32_t levelset, uint32_t mode) {
    if (d == 0 || bucket == 0 || s < 1 || s > ORC_MAX_S) return ORC_ERR_ARG;
    if (norm_kind > 1 || levelset > 2 || mode > 2) return ORC_ERR_ARG;
    if (levelset == LEVELS_UNIFORM && s > 8) return ORC_ERR_ARG;
    if (mode == MODE_CODED && (levelset == LEVELS_UNIFORM || s > ORC_MAX_CODED_S)) return ORC_ERR_ARG;
    return ORC_OK;
}

/* A container with a level table carries the s interior levels (fp32 words) behind the 16 header
 * words, padded with a zero word to an even count so that the offset table stays 8-byte aligned.  */
/* A container with coded level indices carries, behind that, the s + 1 code lengths as the bytes of
 * two words (byte j - 1 in memory = length of index j, the rest zero).                               */
static uint32_t header_words(uint32_t levelset, uint32_t s, uint32_t mode) {
    return ORC_HEADER_WORDS + (levelset == LEVELS_TABLE ? ((s + 1u) & ~1u) : 0u) + (mode == MODE_CODED ? 2u : 0u);
}

/* bytes that always suffice for the container */
uint64_t nuq_oracle_encode_bound(uint64_t d, uint32_t bucket, uint32_t s, uint32_t flags) {
    uint32_t levelset = (flags >> 8) & 0xff, mode = (flags >> 16) & 0xff;
    if (check_args(d, bucket, s, flags & 0xff, levelset, mode) != ORC_OK) return 0;
    uint64_t nb = (d + bucket - 1) / bucket;
    uint64_t hw = header_words(levelset, s, mode);
    if (mode == MODE_FIXED) {
        uint64_t w = nuq_oracle_fixed_width(levelset, s);
        return 4 * (hw + nb * (1 + ((uint64_t)bucket * w + 31) / 32));
    }
    uint64_t nblk = count_blocks(d, bucket);
    uint64_t token_bits = d * (2 + (uint64_t)max_level_code_bits(levelset, s, mode));
    return 4 * hw + 8 * (nblk + 1) + nblk * (4 + 64 + 4) + (token_bits + 7) / 8;
}

/* ENCODE (App. A) of a whole vector, bucket by bucket.
 * flags: bits 0-7 norm kind, 8-15 level set, 16-23 mode.
 * norms_in: NULL, or nb precomputed bucket norms to use instead.             */
int nuq_oracle_encode(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t flags, uint64_t seed,
                      uint64_t offset, const float* norms_in, void* out, uint64_t capacity_bytes,
                      uint64_t* out_bits) {
    uint32_t norm_kind = flags & 0xff, levelset = (flags >> 8) & 0xff, mode = (flags >> 16) & 0xff;
    int rc = check_args(d, bucket, s, norm_kind, levelset, mode);
    if (rc != ORC_OK) return rc;
    if (levelset == LEVELS_TABLE && g_table.s != s) return ORC_ERR_ARG;   /* the table set by nuq_oracle_set_levels */
    if (mode == MODE_CODED && g_code.n != s + 1) return ORC_ERR_ARG;      /* the code set by nuq_oracle_set_level_code */
    if (capacity_bytes < nuq_oracle_encode_bound(d, bucket, s, flags)) return ORC_ERR_CAPACITY;
    memset(out, 0, (size_t)nuq_oracle_encode_bound(d, bucket, s, flags));

    uint32_t* words = (uint32_t*)out;
    uint64_t nb = (d + bucket - 1) / bucket;
    uint64_t nblk = mode != MODE_FIXED ? count_blocks(d, bucket) : nb;
    uint32_t hw = header_words(levelset, s, mode);
    if (levelset == LEVELS_TABLE)
        for (uint32_t j = 1; j <= s; ++j) words[ORC_HEADER_WORDS + j - 1] = float_bits(g_table.level[j]);
    if (mode == MODE_CODED)
        for (uint32_t j = 1; j <= s + 1; ++j) ((uint8_t*)(words + hw - 2))[j - 1] = g_code.len[j - 1];
    uint64_t* table = (uint64_t*)(words + hw);
    uint32_t* payload = mode != MODE_FIXED ? words + hw + 2 * (nblk + 1) : words + hw;
    uint32_t w = nuq_oracle_fixed_width(levelset, s);

    uint8_t* sign = (uint8_t*)malloc(bucket);
    uint16_t* sym = (uint16_t*)malloc(2u * (size_t)bucket);
    uint8_t code[160];
    uint64_t pbits = 0;       /* payload bit cursor */
    uint64_t code_bits = 0, nnz = 0, blk = 0;

    for (uint64_t b = 0; b < nb; ++b) {
        uint64_t lo = b * (uint64_t)bucket;
        uint64_t n = lo + bucket < d ? bucket : d - lo;
        float norm = norms_in ? norms_in[b] : nuq_oracle_norm(g + lo, n, norm_kind);
        nuq_oracle_quantize_bucket(g + lo, n, norm, s, levelset, seed, offset, lo, sign, sym);

        if (mode == MODE_FIXED) {
            pbits = b * 32u * (1 + ((uint64_t)bucket * w + 31) / 32);
            payload[pbits >> 5] = float_bits(norm);
            pbits += 32;
            for (uint64_t i = 0; i < n; ++i) {
                uint32_t field = ((uint32_t)sign[i] << (w - 1)) | sym[i];
                for (uint32_t k = 0; k < w; ++k) put_bit(payload, pbits++, (field >> (w - 1 - k)) & 1u);
                if (sym[i]) ++nnz;
            }
            code_bits += n * w;
            pbits = (pbits + 31) & ~(uint64_t)31;
            continue;
        }

        for (uint64_t blo = 0; blo < n; blo += ORC_BLK, ++blk) {
            uint64_t bn = blo + ORC_BLK < n ? ORC_BLK : n - blo;
            uint64_t nsb = (bn + ORC_SB - 1) / ORC_SB;
            table[blk] = pbits;
            payload[pbits >> 5] = float_bits(norm);         /* the norm, b = 32 bits */
            pbits += 32;
            uint64_t len_base = pbits;                      /* u16 length table */
            pbits += 32 * ((nsb + 1) / 2);
            for (uint64_t sb = 0; sb < nsb; ++sb) {
                uint64_t slo = blo + sb * ORC_SB;
                uint64_t sn = slo + ORC_SB < blo + bn ? ORC_SB : blo + bn - slo;
                uint64_t start = pbits;
                uint64_t t_prev = 0;                        /* t_0 = 0: the run restarts */
                for (uint64_t i = 0; i < sn; ++i) {
                    if (sym[slo + i] == 0) continue;
                    uint64_t t = i + 1;                     /* 1-based position */
                    uint32_t l = nuq_oracle_erc_encode(t - t_prev, code);           /* ERC(gap)   */
                    for (uint32_t k = 0; k < l; ++k) put_bit(payload, pbits++, code[k]);
                    put_bit(payload, pbits++, sign[slo + i]);                       /* sign bit   */
                    if (mode == MODE_CODED) l = nuq_oracle_level_code(sym[slo + i], code);   /* its code word */
                    else l = nuq_oracle_erc_encode(sym[slo + i], code);             /* ERC(level) */
                    for (uint32_t k = 0; k < l; ++k) put_bit(payload, pbits++, code[k]);
                    t_prev = t;
                    ++nnz;
                }
                uint64_t len = pbits - start;
                code_bits += len;
                /* u16 number `sb` of a little-endian u16 array behind the norm word */
                payload[(len_base >> 5) + sb / 2] |= (uint32_t)len << (16u * (uint32_t)(sb & 1u));
            }
            pbits = (pbits + 31) & ~(uint64_t)31;
        }
    }
    if (mode != MODE_FIXED) table[nblk] = pbits;

    uint64_t container_bits = 32u * (uint64_t)(payload - words) + pbits;
    words[0] = ORC_MAGIC; words[1] = ORC_VERSION;
    words[2] = (uint32_t)d; words[3] = (uint32_t)(d >> 32);
    words[4] = bucket; words[5] = s; words[6] = flags & 0xffffffu; words[7] = ORC_SB;
    words[8] = (uint32_t)nblk; words[9] = (uint32_t)(nblk >> 32);
    words[10] = (uint32_t)container_bits; words[11] = (uint32_t)(container_bits >> 32);
    words[12] = (uint32_t)code_bits; words[13] = (uint32_t)(code_bits >> 32);
    words[14] = (uint32_t)nnz; words[15] = (uint32_t)(nnz >> 32);
    if (out_bits) *out_bits = container_bits;
    free(sign); free(sym);
    return ORC_OK;
}

/* DECODE (App. A) of one container into signs and level indices and the
 * per-bucket norms it carries.  Bits are consumed one at a time.              */
int nuq_oracle_decode_symbols(const void* stream, uint64_t d, uint32_t bucket, uint32_t s, uint8_t* sign,
                              uint16_t* sym, float* norms) {
    const uint32_t* words = (const uint32_t*)stream;
    if (words[0] != ORC_MAGIC || words[1] != ORC_VERSION) return ORC_ERR_STREAM;
    uint64_t hd = (uint64_t)words[2] | ((uint64_t)words[3] << 32);
    if (hd != d || words[4] != bucket || words[5] != s || words[7] != ORC_SB) return ORC_ERR_STREAM;
    uint32_t flags = words[6], levelset = (flags >> 8) & 0xff, mode = (flags >> 16) & 0xff;
    if (check_args(d, bucket, s, flags & 0xff, levelset, mode) != ORC_OK) return ORC_ERR_STREAM;
    uint64_t nb = (d + bucket - 1) / bucket;
    uint64_t nblk = (uint64_t)words[8] | ((uint64_t)words[9] << 32);
    uint64_t container_bits = (uint64_t)words[10] | ((uint64_t)words[11] << 32);
    uint32_t nlev = nuq_oracle_num_levels(levelset, s);
    uint32_t w = nuq_oracle_fixed_width(levelset, s);
    uint32_t hw = header_words(levelset, s, mode);
    level_code lc;
    if (mode == MODE_CODED && make_code((const uint8_t*)(words + hw - 2), s + 1, &lc) != ORC_OK) return ORC_ERR_STREAM;
    if (levelset == LEVELS_TABLE) {                          /* the levels must be a level sequence */
        level_table t;
        float interior[ORC_MAX_S];
        for (uint32_t j = 0; j < s; ++j) interior[j] = bits_float(words[ORC_HEADER_WORDS + j]);
        if (make_table(interior, s, &t) != ORC_OK) return ORC_ERR_STREAM;
    }
    memset(sign, 0, (size_t)d);
    memset(sym, 0, 2 * (size_t)d);

    if (mode == MODE_FIXED) {
        if (nblk != nb) return ORC_ERR_STREAM;
        uint64_t last = d - (nb - 1) * (uint64_t)bucket;
        if (container_bits != 32u * (hw + (nb - 1) * (1 + ((uint64_t)bucket * w + 31) / 32) +
                                     1 + (last * w + 31) / 32))
            return ORC_ERR_STREAM;
        const uint32_t* payload = words + hw;
        for (uint64_t b = 0; b < nb; ++b) {
            uint64_t lo = b * (uint64_t)bucket, n = lo + bucket < d ? bucket : d - lo;
            uint64_t p = b * 32u * (1 + ((uint64_t)bucket * w + 31) / 32);
            norms[b] = bits_float(payload[p >> 5]);
            p += 32;
            for (uint64_t i = 0; i < n; ++i) {
                uint32_t field = 0;
                for (uint32_t k = 0; k < w; ++k) field = (field << 1) | get_bit(payload, p++);
                uint32_t q = field & ((1u << (w - 1)) - 1u);
                if (q >= nlev) return ORC_ERR_STREAM;
                sym[lo + i] = (uint16_t)q;
                sign[lo + i] = (uint8_t)(field >> (w - 1));
            }
        }
        return ORC_OK;
    }

    if (nblk != count_blocks(d, bucket)) return ORC_ERR_STREAM;
    const uint64_t* table = (const uint64_t*)(words + hw);
    const uint32_t* payload = words + hw + 2 * (nblk + 1);
    if (container_bits != 32u * (hw + 2 * (nblk + 1)) + table[nblk]) return ORC_ERR_STREAM;
    uint64_t blk = 0;
    for (uint64_t b = 0; b < nb; ++b) {
        uint64_t lo = b * (uint64_t)bucket, n = lo + bucket < d ? bucket : d - lo;
        for (uint64_t blo = 0; blo < n; blo += ORC_BLK, ++blk) {
            uint64_t bn = blo + ORC_BLK < n ? ORC_BLK : n - blo;
            uint64_t nsb = (bn + ORC_SB - 1) / ORC_SB;
            uint64_t p = table[blk], block_end = table[blk + 1];
            if ((p & 31u) || block_end < p + 32 + 32 * ((nsb + 1) / 2)) return ORC_ERR_STREAM;
            norms[b] = bits_float(payload[p >> 5]);          /* read b = 32 bits: the norm */
            p += 32;
            uint64_t len_base = p;
            p += 32 * ((nsb + 1) / 2);
            for (uint64_t sb = 0; sb < nsb; ++sb) {
                uint64_t slo = lo + blo + sb * ORC_SB;
                uint64_t sn = sb * ORC_SB + ORC_SB < bn ? ORC_SB : bn - sb * ORC_SB;
                uint64_t len = (payload[(len_base >> 5) + sb / 2] >> (16u * (uint32_t)(sb & 1u))) & 0xffffu;
                uint64_t end = p + len;
                if (end > block_end) return ORC_ERR_STREAM;
                uint64_t t = 0;
                while (p < end) {
                    /* ERC^-1: the gap to the next nonzero coordinate */
                    uint64_t N = 1;
                    for (;;) {
                        if (p >= end) return ORC_ERR_STREAM;
                        if (get_bit(payload, p) == 0) { ++p; break; }
                        if (N + 1 > 32 || p + N + 1 > end) return ORC_ERR_STREAM;
                        uint64_t v = 0;
                        for (uint64_t i = 0; i <= N; ++i) v = (v << 1) | get_bit(payload, p + i);
                        p += N + 1; N = v;
                    }
                    t += N;
                    if (t > sn || p >= end) return ORC_ERR_STREAM;
                    uint32_t sg = get_bit(payload, p++);     /* the sign bit */
                    N = 1;
                    if (mode == MODE_CODED) {                /* the level index: bits until they spell a code word */
                        uint32_t v = 0, l = 0, found = 0;
                        while (!found) {
                            if (p >= end || l == ORC_MAX_CODED_S) return ORC_ERR_STREAM;
                            v = (v << 1) | get_bit(payload, p++);
                            ++l;
                            for (uint32_t j = 0; j < lc.n; ++j)
                                if (lc.len[j] == l && lc.word[j] == v) { N = j + 1; found = 1; }
                        }
                    } else {                                 /* ERC^-1: the level index */
                        for (;;) {
                            if (p >= end) return ORC_ERR_STREAM;
                            if (get_bit(payload, p) == 0) { ++p; break; }
                            if (N + 1 > 32 || p + N + 1 > end) return ORC_ERR_STREAM;
                            uint64_t v = 0;
                            for (uint64_t i = 0; i <= N; ++i) v = (v << 1) | get_bit(payload, p + i);
                            p += N + 1; N = v;
                        }
                    }
                    if (N >= nlev) return ORC_ERR_STREAM;
                    sym[slo + t - 1] = (uint16_t)N;
                    sign[slo + t - 1] = (uint8_t)sg;
                }
            }
        }
    }
    return ORC_OK;
}

/* DECODE each of K containers and aggregate (Algorithm 1, aggregation line,
 * without the alpha/K factor):  acc[i] = ((0 + q_0[i]) + q_1[i]) + ...  fp32. */
int nuq_oracle_decode_accumulate(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s,
                                 float* acc) {
    if (K == 0 || d == 0 || bucket == 0) return ORC_ERR_ARG;
    uint64_t nb = (d + bucket - 1) / bucket;
    uint8_t* sign = (uint8_t*)malloc((size_t)d);
    uint16_t* sym = (uint16_t*)malloc(2 * (size_t)d);
    float* norms = (float*)malloc(4 * (size_t)nb);
    for (uint64_t i = 0; i < d; ++i) acc[i] = 0.0f;
    int rc = ORC_OK;
    for (uint32_t k = 0; k < K && rc == ORC_OK; ++k) {
        rc = nuq_oracle_decode_symbols(streams[k], d, bucket, s, sign, sym, norms);
        if (rc != ORC_OK) break;
        const uint32_t* words = (const uint32_t*)streams[k];
        uint32_t levelset = (words[6] >> 8) & 0xff;
        for (uint64_t i = 0; i < d; ++i) {
            if (!sym[i]) continue;
            float q;
            if (levelset == LEVELS_TABLE) {                  /* the levels this container carries */
                float level = sym[i] <= s ? bits_float(words[ORC_HEADER_WORDS + sym[i] - 1]) : 1.0f;
                q = norms[i / bucket] * level;
                if (sign[i]) q = -q;
            } else {
                q = nuq_oracle_dequantize(norms[i / bucket], s, levelset, sign[i], sym[i]);
            }
            acc[i] = acc[i] + q;
        }
    }
    free(sign); free(sym); free(norms);
    return rc;
}

/* The aggregation step of Algorithm 1 with the momentum rule of Sec. 4 ("NUQSGD with momentum"), where the
 * gradient is the average g = (1/K) sum_i g^_i of the decoded gradients (`sum` holds sum_i g^_i):
 *     y      = w - alpha g
 *     y^l    = w - l alpha g
 *     w_next = y + mu (y^l - y^l_prev)
 * l = 0 is the heavy-ball method, l = 1 Nesterov's; mu = 0 is Algorithm 1's own line w - (alpha/K) sum_i g^_i
 * (no projection: Omega = R^d).  fp64; w and yl (y^l_prev on entry, y^l on return) are updated in place.   */
void nuq_oracle_momentum_step(double* w, double* yl, const float* sum, uint64_t d, double alpha, uint32_t K,
                              double mu, double l) {
    for (uint64_t i = 0; i < d; ++i) {
        double g = (double)sum[i] / (double)K;
        double y = w[i] - alpha * g;
        double yl_next = w[i] - l * alpha * g;
        w[i] = y + mu * (yl_next - yl[i]);
        yl[i] = yl_next;
    }
}

/* Code length of the paper's own framing (one run per bucket, no sub-block
 * restarts): 32 bits for the norm plus the tokens.  For reporting only.      */
uint64_t nuq_oracle_single_chain_bits(const uint16_t* sym, uint64_t n) {
    uint8_t code[160];
    uint64_t bits = 32, t_prev = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!sym[i]) continue;
        bits += nuq_oracle_erc_encode(i + 1 - t_prev, code) + 1 + nuq_oracle_erc_encode(sym[i], code);
        t_prev = i + 1;
    }
    return bits;
}
