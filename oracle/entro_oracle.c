/*
 * CPU oracle for the EntroLLM weight path: per-tensor quantiser, symbol histogram,
 * Huffman code lengths, canonical codes, encoder with a per-chunk bit-offset index,
 * bit-serial decoder, dequantiser, and an fp64 matrix-vector reference.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, single-purpose restatement
 * of what the method computes, written from the paper's text, and it shares no code,
 * header, table or helper with the CUDA library.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it; the product never does.
 *
 * Every function is pinned by tests that do not go through this file's own arithmetic
 * (closed forms, brute force on tiny alphabets, NumPy's float16, invariants); none is
 * "parity unpinned".
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fPIC -shared -pthread
 * (fp32 operations must be performed one at a time, no fused multiply-add, default
 * round-to-nearest-even mode).
 *
 * Conventions the paper leaves open are fixed here in one place:
 *  - Eq. 1 gives W_int = round(W_fp / s) (unsigned) and round((W_fp - z) / s)
 *    (asymmetric).  The integer-domain form is used: q = clamp(rne(w / s) + z, 0, qmax)
 *    with an integer zero-point z in [0, qmax], so that w_hat = s * (q - z).
 *  - The mode is chosen per tensor from its weight distribution (Section 3, mixed
 *    quantisation), the rule is not given: a tensor is unsigned iff all of its weights
 *    are >= 0, else asymmetric.
 *  - s comes from the tensor's min/max; round() is round-half-to-even in fp32.
 *  - Huffman (Section 3, Huffman weight encoding): repeated merging of the two
 *    smallest nodes; ties are broken by (weight, leaf-before-internal, symbol value or
 *    creation order); code length = depth; unused symbols have length 0; a single
 *    used symbol gets length 1.
 *  - Canonical codes: symbols ordered by (length, symbol); first code 0.
 *  - Bitstream: codewords concatenated MSB-first, chunk after chunk and inside a chunk in
 *    the order given under "Segments", stored in 32-bit words, stream bit i being bit
 *    (31 - i % 32) of word i / 32.
 *  - Segments (Section 3, segmentation for parallel decoding): fixed-size chunks of
 *    chunk_symbols consecutive symbols of one tensor, offsets[c] = bit position where
 *    chunk c starts, offsets[n_chunks] = total bits.  The paper fixes that segments have
 *    known boundaries and decode independently, not the order of the codewords inside
 *    one.  Here a chunk's symbols are taken in groups of 8 consecutive symbols (the last
 *    group may be short); sub-block l (0 <= l < 32) is the groups l, l + 32, l + 64, ...
 *    in that order; the chunk's codewords are stored sub-block after sub-block, and
 *    the bit length of every sub-block is recorded as well.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_SMALL 2
#define ORACLE_ERR_NONFINITE 3
#define ORACLE_ERR_TOO_LONG 4
#define ORACLE_ERR_CORRUPT 5

#define MODE_AUTO 0
#define MODE_UNSIGNED 1
#define MODE_ASYMMETRIC 2

#define MAX_SYMBOLS 256
#define MAX_LEN 32
#define SUB_BLOCKS 32
#define GROUP 8        /* symbols per group inside a chunk */

/* ------------------------------------------------------------------ fp16 <-> fp32 */

/* Exact widening of an IEEE binary16 bit pattern to a float. */
float oracle_f16_to_f32(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    int32_t expo = (h >> 10) & 0x1f;
    uint32_t frac = h & 0x3ffu;
    float mag;
    if (expo == 0x1f) {
        mag = frac ? NAN : INFINITY;
    } else if (expo == 0) {
        mag = ldexpf((float)frac, -24);              /* subnormal: frac * 2^-24 */
    } else {
        mag = ldexpf((float)(frac | 0x400u), expo - 25); /* (1024 + frac) * 2^(e-15-10) */
    }
    return sign ? -mag : mag;
}

/* Round a float to the nearest binary16 value, ties to even; overflow gives infinity. */
uint16_t oracle_f32_to_f16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t absu = u & 0x7fffffffu;
    if (absu > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);  /* NaN */
    if (absu == 0x7f800000u) return (uint16_t)(sign | 0x7c00u); /* infinity */
    double a = fabs((double)f);
    if (a == 0.0) return sign;
    /* Spacing of binary16 values around a: 2^(e-10) for normal e >= -14, else 2^-24. */
    int e;
    (void)frexp(a, &e);        /* a = m * 2^e, m in [0.5, 1)  ->  a in [2^(e-1), 2^e) */
    int e2 = e - 1;            /* floor(log2 a) */
    if (e2 < -14) e2 = -14;
    double ulp = ldexp(1.0, e2 - 10);
    double k = a / ulp;        /* exact: division by a power of two */
    double r = nearbyint(k);   /* default mode: ties to even */
    double v = r * ulp;        /* the rounded magnitude, exact */
    if (v >= 65520.0) return (uint16_t)(sign | 0x7c00u);
    if (v == 0.0) return sign;
    /* Re-derive exponent and fraction of the rounded value. */
    (void)frexp(v, &e);
    e2 = e - 1;
    if (e2 < -14) {
        uint32_t fr = (uint32_t)(v / ldexp(1.0, -24));
        return (uint16_t)(sign | fr);
    }
    uint32_t mant = (uint32_t)(v / ldexp(1.0, e2 - 10)); /* in [1024, 2048) */
    return (uint16_t)(sign | ((uint32_t)(e2 + 15) << 10) | (mant - 1024u));
}

void oracle_f16_to_f32_array(const uint16_t *h, uint64_t n, float *f)
{
    for (uint64_t i = 0; i < n; ++i) f[i] = oracle_f16_to_f32(h[i]);
}

void oracle_f32_to_f16_array(const float *f, uint64_t n, uint16_t *h)
{
    for (uint64_t i = 0; i < n; ++i) h[i] = oracle_f32_to_f16_rne(f[i]);
}

/* ------------------------------------------------------------------ quantiser (Eq. 1) */

typedef struct {
    int32_t bits;
    int32_t mode;        /* MODE_UNSIGNED or MODE_ASYMMETRIC, resolved */
    float scale;
    int32_t zero_point;
    float lo, hi;        /* tensor min / max */
} oracle_qparams;

static int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* Range, mode and (s, z) of a tensor. */
int oracle_quant_params(const uint16_t *w, uint64_t n, int bits, int mode, oracle_qparams *qp)
{
    if (!w || !qp || n == 0 || (bits != 4 && bits != 8) || mode < 0 || mode > 2) return ORACLE_ERR_ARG;
    float lo = INFINITY, hi = -INFINITY;
    for (uint64_t i = 0; i < n; ++i) {
        float x = oracle_f16_to_f32(w[i]);
        if (!isfinite(x)) return ORACLE_ERR_NONFINITE;
        if (x < lo) lo = x;
        if (x > hi) hi = x;
    }
    /* -0.0 and +0.0 compare equal; normalise so the result does not depend on which came first. */
    if (lo == 0.0f) lo = 0.0f;
    if (hi == 0.0f) hi = 0.0f;
    const int qmax = (1 << bits) - 1;
    if (mode == MODE_AUTO) mode = (lo >= 0.0f) ? MODE_UNSIGNED : MODE_ASYMMETRIC;
    float s;
    int z;
    if (mode == MODE_UNSIGNED) {
        s = hi / (float)qmax;
        if (!(s > 0.0f)) s = 1.0f;        /* degenerate range */
        z = 0;
    } else {
        float range = hi - lo;
        s = range / (float)qmax;
        if (!(s > 0.0f)) s = 1.0f;
        float zf = rintf(-lo / s);
        if (zf < 0.0f) zf = 0.0f;
        if (zf > (float)qmax) zf = (float)qmax;
        z = (int)zf;
    }
    qp->bits = bits;
    qp->mode = mode;
    qp->scale = s;
    qp->zero_point = z;
    qp->lo = lo;
    qp->hi = hi;
    return ORACLE_OK;
}

/* One weight to its integer code. */
uint8_t oracle_quantize_one(uint16_t w, float s, int z, int bits)
{
    const int qmax = (1 << bits) - 1;
    float x = oracle_f16_to_f32(w);
    float t = x / s;
    float r = rintf(t);
    /* |r| is far below 2^31 for any finite fp16 input and a min/max scale. */
    int qi = (int)r + z;
    return (uint8_t)clampi(qi, 0, qmax);
}

int oracle_quantize_tensor(const uint16_t *w, uint64_t n, int bits, int mode, uint8_t *q,
                           oracle_qparams *qp)
{
    if (!q) return ORACLE_ERR_ARG;
    int rc = oracle_quant_params(w, n, bits, mode, qp);
    if (rc) return rc;
    for (uint64_t i = 0; i < n; ++i) q[i] = oracle_quantize_one(w[i], qp->scale, qp->zero_point, bits);
    return ORACLE_OK;
}

/*
 * The grid the paper compares against (Section 3, "Mixed Quantization Scheme"; Table 2,
 * column "SOTA"): block-based quantisation, every run of `block` consecutive weights (the
 * paper's example is 32) with a range, scale and zero point of its own, by the same Eq. 1.  The last block may be shorter.  scales / zps (one per block) may be NULL.
 */
int oracle_quantize_blocks(const uint16_t *w, uint64_t n, int bits, int mode, uint64_t block, uint8_t *q,
                           float *scales, int32_t *zps)
{
    if (!w || !q || n == 0 || block == 0) return ORACLE_ERR_ARG;
    uint64_t b = 0;
    for (uint64_t first = 0; first < n; first += block, ++b) {
        const uint64_t m = n - first < block ? n - first : block;
        oracle_qparams qp;
        int rc = oracle_quant_params(w + first, m, bits, mode, &qp);
        if (rc) return rc;
        for (uint64_t i = 0; i < m; ++i) q[first + i] = oracle_quantize_one(w[first + i], qp.scale, qp.zero_point, bits);
        if (scales) scales[b] = qp.scale;
        if (zps) zps[b] = qp.zero_point;
    }
    return ORACLE_OK;
}

/* w_hat = fp16( s * (q - z) ), the product taken in fp32 and rounded once. */
uint16_t oracle_dequant_one(uint8_t q, float s, int z)
{
    float d = (float)((int)q - z);
    float p = s * d;
    return oracle_f32_to_f16_rne(p);
}

void oracle_dequant(const uint8_t *q, uint64_t n, float s, int z, uint16_t *out)
{
    for (uint64_t i = 0; i < n; ++i) out[i] = oracle_dequant_one(q[i], s, z);
}

/* ------------------------------------------------------------------ histogram */

int oracle_histogram(const uint8_t *q, uint64_t n, int nsym, uint64_t *counts)
{
    if (!counts || nsym < 1 || nsym > MAX_SYMBOLS) return ORACLE_ERR_ARG;
    for (int k = 0; k < nsym; ++k) counts[k] = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (q[i] >= nsym) return ORACLE_ERR_ARG;
        counts[q[i]]++;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ Huffman lengths */

/*
 * Repeatedly remove the two smallest live nodes and replace them by their parent.
 * "Smallest" is by (weight, leaf before internal node, symbol value for leaves or
 * creation order for internal nodes).  Written as a direct search for the minimum so
 * that the rule can be read off the code.
 */
int oracle_huffman_lengths(const uint64_t *counts, int nsym, uint8_t *len)
{
    if (!counts || !len || nsym < 1 || nsym > MAX_SYMBOLS) return ORACLE_ERR_ARG;
    enum { MAXN = 2 * MAX_SYMBOLS };
    uint64_t weight[MAXN];
    int parent[MAXN], internal[MAXN], order[MAXN], live[MAXN];
    int nn = 0, used = 0;
    int leaf_of[MAX_SYMBOLS];
    for (int k = 0; k < nsym; ++k) {
        len[k] = 0;
        leaf_of[k] = -1;
        if (counts[k] > 0) {
            weight[nn] = counts[k]; parent[nn] = -1; internal[nn] = 0; order[nn] = k; live[nn] = 1;
            leaf_of[k] = nn++;
            used++;
        }
    }
    if (used == 0) return ORACLE_OK;
    if (used == 1) {
        for (int k = 0; k < nsym; ++k) if (counts[k] > 0) len[k] = 1;
        return ORACLE_OK;
    }
    int alive = used, created = 0;
    while (alive > 1) {
        int pick[2];
        for (int p = 0; p < 2; ++p) {
            int best = -1;
            for (int i = 0; i < nn; ++i) {
                if (!live[i]) continue;
                if (best < 0) { best = i; continue; }
                int better;
                if (weight[i] != weight[best]) better = weight[i] < weight[best];
                else if (internal[i] != internal[best]) better = internal[i] < internal[best];
                else better = order[i] < order[best];
                if (better) best = i;
            }
            live[best] = 0;
            pick[p] = best;
        }
        weight[nn] = weight[pick[0]] + weight[pick[1]];
        parent[nn] = -1; internal[nn] = 1; order[nn] = created++; live[nn] = 1;
        parent[pick[0]] = nn; parent[pick[1]] = nn;
        nn++;
        alive--;
    }
    for (int k = 0; k < nsym; ++k) {
        if (leaf_of[k] < 0) continue;
        int d = 0;
        for (int i = leaf_of[k]; parent[i] >= 0; i = parent[i]) d++;
        if (d > MAX_LEN) return ORACLE_ERR_TOO_LONG;
        len[k] = (uint8_t)d;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ length-limited lengths */

/*
 * Optimal prefix-code lengths under a cap: no code longer than max_len, total cost
 * sum(count * length) minimal among such codes (the package-merge construction of Larmore
 * and Hirschberg).  This departs from the paper, which uses the unrestricted Huffman code
 * and states that no prefix code is more efficient (Section 3, Huffman weight encoding); it
 * is an optional format variant.  Steps, fixed so that exactly one answer exists:
 *   - leaves = used symbols, ascending by (count, symbol);
 *   - for level j = max_len down to 1: the level's list is the leaves merged with the
 *     packages made at level j + 1 (none at level max_len), ascending by weight; on equal
 *     weight a leaf comes before a package, leaves in their sorted order, packages in the
 *     order in which they were made;
 *   - the packages of level j are the consecutive pairs of its list (first + second,
 *     third + fourth, ...; an odd last item is dropped);
 *   - a symbol's length is the number of items among the first 2 * (n - 1) of level 1's
 *     list that contain it, a package containing what its two halves contain.
 * One used symbol gets length 1.  Fails if 2^max_len < n.
 */
int oracle_length_limited_lengths(const uint64_t *counts, int nsym, int max_len, uint8_t *len)
{
    if (!counts || !len || nsym < 1 || nsym > MAX_SYMBOLS || max_len < 1 || max_len > MAX_LEN) return ORACLE_ERR_ARG;
    int order[MAX_SYMBOLS], n = 0;
    for (int k = 0; k < nsym; ++k) { len[k] = 0; if (counts[k]) order[n++] = k; }
    if (n == 0) return ORACLE_OK;
    if (n == 1) { len[order[0]] = 1; return ORACLE_OK; }
    if (max_len < 31 && (1u << max_len) < (unsigned)n) return ORACLE_ERR_TOO_LONG;
    /* insertion sort by (count, symbol): symbols are already ascending, keep them so on ties */
    for (int i = 1; i < n; ++i) {
        int s = order[i], j = i - 1;
        while (j >= 0 && counts[order[j]] > counts[s]) { order[j + 1] = order[j]; --j; }
        order[j + 1] = s;
    }
    /* an item = its weight and, per leaf, how many times it contains that leaf */
    enum { MAXI = 2 * MAX_SYMBOLS };
    typedef struct { uint64_t w; uint8_t has[MAX_SYMBOLS]; } item;
    item *cur = (item *)calloc(MAXI, sizeof(item)), *pk = (item *)calloc(MAXI, sizeof(item));
    if (!cur || !pk) { free(cur); free(pk); return ORACLE_ERR_ARG; }
    int npk = 0;
    int ncur = 0;
    for (int level = max_len; level >= 1; --level) {
        /* merge leaves and packages */
        int a = 0, b = 0;
        ncur = 0;
        while (a < n || b < npk) {
            int take_leaf = b >= npk || (a < n && counts[order[a]] <= pk[b].w);
            if (take_leaf) {
                memset(&cur[ncur], 0, sizeof(item));
                cur[ncur].w = counts[order[a]];
                cur[ncur].has[a] = 1;
                ++a;
            } else {
                cur[ncur] = pk[b];
                ++b;
            }
            ++ncur;
        }
        if (level == 1) break;
        npk = 0;
        for (int i = 0; i + 1 < ncur; i += 2) {
            pk[npk].w = cur[i].w + cur[i + 1].w;
            for (int k = 0; k < n; ++k) pk[npk].has[k] = (uint8_t)(cur[i].has[k] + cur[i + 1].has[k]);
            ++npk;
        }
    }
    int need = 2 * (n - 1);
    if (ncur < need) { free(cur); free(pk); return ORACLE_ERR_TOO_LONG; }
    for (int i = 0; i < need; ++i)
        for (int k = 0; k < n; ++k) len[order[k]] = (uint8_t)(len[order[k]] + cur[i].has[k]);
    free(cur);
    free(pk);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ canonical codes */

/*
 * Symbols in order of (length ascending, symbol ascending); the first gets code 0;
 * each next code is (previous + 1) shifted left by the growth in length.
 */
int oracle_canonical_codes(const uint8_t *len, int nsym, uint32_t *code)
{
    if (!len || !code || nsym < 1 || nsym > MAX_SYMBOLS) return ORACLE_ERR_ARG;
    uint64_t next = 0;
    int prev_len = 0, first = 1;
    for (int k = 0; k < nsym; ++k) code[k] = 0;
    for (int l = 1; l <= MAX_LEN; ++l) {
        for (int k = 0; k < nsym; ++k) {
            if (len[k] != l) continue;
            if (first) { next = 0; first = 0; }
            else next = (next + 1) << (l - prev_len);
            prev_len = l;
            if (next >> l) return ORACLE_ERR_ARG;      /* lengths violate Kraft */
            code[k] = (uint32_t)next;
        }
    }
    for (int k = 0; k < nsym; ++k) if (len[k] > MAX_LEN) return ORACLE_ERR_TOO_LONG;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ encoder */

static void put_bit(uint32_t *stream, uint64_t pos, int bit)
{
    if (bit) stream[pos >> 5] |= 1u << (31 - (pos & 31));
}

uint64_t oracle_num_chunks(uint64_t n, uint32_t chunk_symbols)
{
    return (n + chunk_symbols - 1) / chunk_symbols;
}

/*
 * stream: cap_words 32-bit words, fully zeroed here and then filled.
 * offsets: n_chunks + 1 entries.  sub_len: n_chunks * 32 entries.
 */
int oracle_encode(const uint8_t *q, uint64_t n, const uint8_t *len, const uint32_t *code, int nsym,
                  uint32_t chunk_symbols, uint32_t *stream, uint64_t cap_words, uint64_t *offsets,
                  uint16_t *sub_len, uint64_t *total_bits)
{
    if (!q || !len || !code || !stream || !offsets || !sub_len || !total_bits) return ORACLE_ERR_ARG;
    if (chunk_symbols == 0 || chunk_symbols % SUB_BLOCKS) return ORACLE_ERR_ARG;
    const uint32_t sub = chunk_symbols / SUB_BLOCKS;
    uint64_t need = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (q[i] >= nsym || len[q[i]] == 0) return ORACLE_ERR_ARG;
        need += len[q[i]];
    }
    if ((need + 31) / 32 > cap_words) return ORACLE_ERR_SMALL;
    memset(stream, 0, cap_words * sizeof(uint32_t));
    const uint64_t nchunks = oracle_num_chunks(n, chunk_symbols);
    memset(sub_len, 0, nchunks * SUB_BLOCKS * sizeof(uint16_t));
    uint64_t pos = 0;
    (void)sub;
    for (uint64_t c = 0; c < nchunks; ++c) {
        const uint64_t first = c * chunk_symbols;
        const uint64_t m = (first + chunk_symbols <= n) ? chunk_symbols : n - first;   /* symbols in this chunk */
        offsets[c] = pos;
        for (uint32_t l = 0; l < SUB_BLOCKS; ++l) {
            for (uint64_t g = l; g * GROUP < m; g += SUB_BLOCKS) {
                for (uint64_t k = 0; k < GROUP && g * GROUP + k < m; ++k) {
                    const uint8_t sym = q[first + g * GROUP + k];
                    const int ln = len[sym];
                    const uint32_t cw = code[sym];
                    for (int b = ln - 1; b >= 0; --b) put_bit(stream, pos++, (cw >> b) & 1);
                    sub_len[c * SUB_BLOCKS + l] += (uint16_t)ln;
                }
            }
        }
    }
    offsets[nchunks] = pos;
    *total_bits = pos;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ decoder */

typedef struct {
    uint32_t count[MAX_LEN + 1];       /* symbols of each length */
    uint32_t first_code[MAX_LEN + 1];  /* canonical code of the first symbol of each length */
    uint32_t offset[MAX_LEN + 1];      /* position of that symbol in sorted[] */
    uint8_t sorted[MAX_SYMBOLS];       /* symbols by (length, symbol) */
    int max_len;
} oracle_decode_tables;

int oracle_make_tables(const uint8_t *len, int nsym, oracle_decode_tables *t)
{
    if (!len || !t || nsym < 1 || nsym > MAX_SYMBOLS) return ORACLE_ERR_ARG;
    memset(t, 0, sizeof(*t));
    for (int k = 0; k < nsym; ++k) {
        if (len[k] > MAX_LEN) return ORACLE_ERR_TOO_LONG;
        if (len[k]) { t->count[len[k]]++; if (len[k] > t->max_len) t->max_len = len[k]; }
    }
    uint32_t code = 0, off = 0;
    for (int l = 1; l <= MAX_LEN; ++l) {
        code <<= 1;
        t->first_code[l] = code;
        t->offset[l] = off;
        code += t->count[l];
        off += t->count[l];
    }
    uint32_t fill[MAX_LEN + 1];
    memcpy(fill, t->offset, sizeof(fill));
    for (int k = 0; k < nsym; ++k) if (len[k]) t->sorted[fill[len[k]]++] = (uint8_t)k;
    return ORACLE_OK;
}

static int get_bit(const uint32_t *stream, uint64_t pos)
{
    return (int)((stream[pos >> 5] >> (31 - (pos & 31))) & 1u);
}

/*
 * Decode `count` symbols starting at stream bit `pos`, one bit at a time: extend the
 * code by a bit, and stop as soon as it falls inside the range of codes of its length.
 * limit_bits is the number of valid bits in the stream.
 */
int oracle_decode_symbols(const uint32_t *stream, uint64_t limit_bits, uint64_t pos, uint64_t count,
                          const oracle_decode_tables *t, uint8_t *q, uint64_t *end_pos)
{
    for (uint64_t i = 0; i < count; ++i) {
        uint32_t code = 0;
        int l = 0, found = 0;
        while (l < t->max_len) {
            if (pos >= limit_bits) return ORACLE_ERR_CORRUPT;
            code = (code << 1) | (uint32_t)get_bit(stream, pos++);
            l++;
            if (t->count[l] && code >= t->first_code[l] && code - t->first_code[l] < t->count[l]) {
                q[i] = t->sorted[t->offset[l] + (code - t->first_code[l])];
                found = 1;
                break;
            }
        }
        if (!found) return ORACLE_ERR_CORRUPT;
    }
    if (end_pos) *end_pos = pos;
    return ORACLE_OK;
}

/* Decode one chunk on its own from its recorded start, and check where it ends. */
static int decode_dequant_chunk(const uint32_t *stream, const uint64_t *offsets, uint64_t n,
                                uint32_t chunk_symbols, const oracle_decode_tables *t, float s, int z,
                                uint64_t c, uint8_t *q_out, uint16_t *out)
{
    uint64_t nchunks = oracle_num_chunks(n, chunk_symbols);
    uint64_t first = c * chunk_symbols;
    uint64_t cnt = (first + chunk_symbols <= n) ? chunk_symbols : n - first;
    uint8_t buf[16384];
    uint64_t end = 0;
    if (cnt > sizeof(buf)) return ORACLE_ERR_ARG;
    int rc = oracle_decode_symbols(stream, offsets[nchunks], offsets[c], cnt, t, buf, &end);
    if (rc) return rc;
    if (end != offsets[c + 1]) return ORACLE_ERR_CORRUPT;
    /* buf holds the symbols in stored order: sub-block after sub-block */
    uint64_t stored = 0;
    for (uint32_t l = 0; l < SUB_BLOCKS; ++l) {
        for (uint64_t g = l; g * GROUP < cnt; g += SUB_BLOCKS) {
            for (uint64_t k = 0; k < GROUP && g * GROUP + k < cnt; ++k) {
                const uint64_t i = first + g * GROUP + k;
                if (q_out) q_out[i] = buf[stored];
                if (out) out[i] = oracle_dequant_one(buf[stored], s, z);
                ++stored;
            }
        }
    }
    return ORACLE_OK;
}

/* Whole tensor, chunk after chunk.  q_out and out may each be NULL. */
int oracle_decode_dequant(const uint32_t *stream, const uint64_t *offsets, uint64_t n,
                          uint32_t chunk_symbols, const uint8_t *len, int nsym, float s, int z,
                          uint8_t *q_out, uint16_t *out)
{
    oracle_decode_tables t;
    int rc = oracle_make_tables(len, nsym, &t);
    if (rc) return rc;
    if (chunk_symbols == 0 || chunk_symbols > 16384) return ORACLE_ERR_ARG;
    uint64_t nchunks = oracle_num_chunks(n, chunk_symbols);
    for (uint64_t c = 0; c < nchunks; ++c) {
        rc = decode_dequant_chunk(stream, offsets, n, chunk_symbols, &t, s, z, c, q_out, out);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

/* A chosen list of chunks, in the order given (segments are independent). */
int oracle_decode_dequant_chunks(const uint32_t *stream, const uint64_t *offsets, uint64_t n,
                                 uint32_t chunk_symbols, const uint8_t *len, int nsym, float s, int z,
                                 const uint64_t *chunk_ids, uint64_t n_ids, uint8_t *q_out,
                                 uint16_t *out)
{
    oracle_decode_tables t;
    int rc = oracle_make_tables(len, nsym, &t);
    if (rc) return rc;
    if (chunk_symbols == 0 || chunk_symbols > 16384) return ORACLE_ERR_ARG;
    uint64_t nchunks = oracle_num_chunks(n, chunk_symbols);
    for (uint64_t k = 0; k < n_ids; ++k) {
        if (chunk_ids[k] >= nchunks) return ORACLE_ERR_ARG;
        rc = decode_dequant_chunk(stream, offsets, n, chunk_symbols, &t, s, z, chunk_ids[k], q_out, out);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

/*
 * The paper's parallel decoder (Section 3, segmentation; Section 4, hardware efficiency):
 * independent segments dealt to threads, no synchronisation between them.  Chunks are
 * dealt round-robin to nthreads threads.
 */
typedef struct {
    const uint32_t *stream; const uint64_t *offsets; uint64_t n; uint32_t chunk_symbols;
    const oracle_decode_tables *t; float s; int z; uint16_t *out;
    uint64_t first, stride, nchunks; int rc;
} mt_job;

static void *mt_worker(void *arg)
{
    mt_job *j = (mt_job *)arg;
    for (uint64_t c = j->first; c < j->nchunks; c += j->stride) {
        int rc = decode_dequant_chunk(j->stream, j->offsets, j->n, j->chunk_symbols, j->t, j->s, j->z,
                                      c, NULL, j->out);
        if (rc) { j->rc = rc; break; }
    }
    return NULL;
}

int oracle_decode_dequant_mt(const uint32_t *stream, const uint64_t *offsets, uint64_t n,
                             uint32_t chunk_symbols, const uint8_t *len, int nsym, float s, int z,
                             uint16_t *out, int nthreads)
{
    oracle_decode_tables t;
    int rc = oracle_make_tables(len, nsym, &t);
    if (rc) return rc;
    if (nthreads < 1 || nthreads > 1024 || chunk_symbols == 0 || chunk_symbols > 16384) return ORACLE_ERR_ARG;
    uint64_t nchunks = oracle_num_chunks(n, chunk_symbols);
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    mt_job *jobs = (mt_job *)malloc(sizeof(mt_job) * (size_t)nthreads);
    if (!th || !jobs) { free(th); free(jobs); return ORACLE_ERR_ARG; }
    for (int i = 0; i < nthreads; ++i) {
        mt_job j = { stream, offsets, n, chunk_symbols, &t, s, z, out, (uint64_t)i, (uint64_t)nthreads, nchunks, 0 };
        jobs[i] = j;
        pthread_create(&th[i], NULL, mt_worker, &jobs[i]);
    }
    for (int i = 0; i < nthreads; ++i) {
        pthread_join(th[i], NULL);
        if (jobs[i].rc && !rc) rc = jobs[i].rc;
    }
    free(th);
    free(jobs);
    return rc;
}

/* ------------------------------------------------------------------ matrix-vector reference */

/*
 * y[o] = sum_i w_hat[o, i] * x[i] in fp64 over fp16 operands (W stored [rows, cols]
 * row-major), plus sum_i |w_hat[o, i] * x[i]| for the accumulation error bound.
 */
void oracle_gemv_f64(const uint16_t *w_hat, uint64_t rows, uint64_t cols, const uint16_t *x, double *y,
                     double *abs_sum)
{
    for (uint64_t o = 0; o < rows; ++o) {
        double acc = 0.0, aacc = 0.0;
        for (uint64_t i = 0; i < cols; ++i) {
            double p = (double)oracle_f16_to_f32(w_hat[o * cols + i]) * (double)oracle_f16_to_f32(x[i]);
            acc += p;
            aacc += fabs(p);
        }
        y[o] = acc;
        if (abs_sum) abs_sum[o] = aacc;
    }
}
