/*
 * sbc_oracle.c -- CPU oracle for Sparse Binary Compression (arXiv 1805.08768).
 * TEST INFRASTRUCTURE ONLY; see sbc_oracle.h for the scope, the readings of
 * the paper and the list of parity pins.  Single-threaded, plain loops, no
 * blocking or fusion beyond what the algorithms state.
 */
#include "sbc_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Scalars derived from p                                              */
/* ------------------------------------------------------------------ */

int64_t sbc_oracle_kept_count(int64_t n, double p) {
    if (n <= 0) return 0;
    double prod = p * (double)n; /* one fp64 multiply */
    int64_t k = (int64_t)floor(prod);
    if (k < 1) k = 1;
    if (k > n) k = n;
    return k;
}

int sbc_oracle_golomb_b(double p) {
    /* Algorithm 3: b* = 1 + floor(log2(log(phi - 1) / log(1 - p))). */
    const double phi = (sqrt(5.0) + 1.0) / 2.0;
    double ratio = log(phi - 1.0) / log(1.0 - p);
    int b = 1 + (int)floor(log2(ratio));
    if (b < 0) b = 0; /* p above ~0.38: pure unary code */
    return b;
}

double sbc_oracle_mean_position_bits(double p, int b) {
    /* Eq. for b_pos. */
    return (double)b + 1.0 / (1.0 - pow(1.0 - p, ldexp(1.0, b)));
}

/* ------------------------------------------------------------------ */
/* Algorithm 1, client accumulate line                                 */
/* ------------------------------------------------------------------ */

int sbc_oracle_accumulate(const float *update, float *residual, int64_t n) {
    int bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        volatile float a = residual[i] + update[i]; /* one fp32 add */
        residual[i] = a;
        if (!isfinite(a)) bad = 1;
    }
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------ */
/* Algorithm 2, top_p: full sort by (value, index), first k            */
/* ------------------------------------------------------------------ */

typedef struct {
    float v;   /* the value being ranked (a or -a) */
    int64_t i; /* flat index */
} ranked_t;

static int ranked_desc(const void *x, const void *y) {
    const ranked_t *a = (const ranked_t *)x, *b = (const ranked_t *)y;
    if (a->v > b->v) return -1; /* larger value first */
    if (a->v < b->v) return 1;
    if (a->i < b->i) return -1; /* equal values (incl. -0 vs +0): lower index */
    if (a->i > b->i) return 1;
    return 0;
}

int sbc_oracle_topk(const float *a, int64_t n, int64_t k, int negate,
                    int64_t *out_idx) {
    if (n <= 0 || k < 0 || k > n) return -2;
    ranked_t *r = (ranked_t *)malloc((size_t)n * sizeof(ranked_t));
    if (!r) return -2;
    for (int64_t i = 0; i < n; ++i) {
        r[i].v = negate ? -a[i] : a[i];
        r[i].i = i;
    }
    qsort(r, (size_t)n, sizeof(ranked_t), ranked_desc);
    for (int64_t j = 0; j < k; ++j) out_idx[j] = r[j].i;
    free(r);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Exact sum of fp32 values, rounded once to fp64                      */
/* ------------------------------------------------------------------ */
/*
 * Every finite fp32 is an integer multiple of 2^-149 below 2^128, so a sum
 * of up to 2^63 of them fits a 384-bit two's-complement integer in units of
 * 2^-149.  The integer is then rounded to nearest-even at 53 bits.
 */
#define ACC_LIMBS 6

static void acc_add_shifted(uint64_t acc[ACC_LIMBS], uint64_t m, int shift,
                            int negative) {
    /* acc +/-= m << shift, with m < 2^24 and 0 <= shift <= 253 */
    int limb = shift / 64, off = shift % 64;
    uint64_t lo = m << off;
    uint64_t hi = off ? (m >> (64 - off)) : 0;
    if (!negative) {
        uint64_t carry = 0;
        for (int l = limb; l < ACC_LIMBS; ++l) {
            uint64_t add = (l == limb) ? lo : (l == limb + 1) ? hi : 0;
            uint64_t s = acc[l] + add;
            uint64_t c1 = s < add;
            uint64_t s2 = s + carry;
            uint64_t c2 = s2 < carry;
            acc[l] = s2;
            carry = c1 | c2;
            if (l > limb && !carry) break;
        }
    } else {
        uint64_t borrow = 0;
        for (int l = limb; l < ACC_LIMBS; ++l) {
            uint64_t sub = (l == limb) ? lo : (l == limb + 1) ? hi : 0;
            uint64_t d = acc[l] - sub;
            uint64_t b1 = acc[l] < sub;
            uint64_t d2 = d - borrow;
            uint64_t b2 = d < borrow;
            acc[l] = d2;
            borrow = b1 | b2;
            if (l > limb && !borrow) break;
        }
    }
}

static int acc_bit(const uint64_t mag[ACC_LIMBS], int pos) {
    return (int)((mag[pos / 64] >> (pos % 64)) & 1u);
}

static double acc_to_double(const uint64_t acc_in[ACC_LIMBS]) {
    uint64_t mag[ACC_LIMBS];
    memcpy(mag, acc_in, sizeof(mag));
    int negative = (int)(mag[ACC_LIMBS - 1] >> 63);
    if (negative) { /* magnitude = two's complement negate */
        uint64_t carry = 1;
        for (int l = 0; l < ACC_LIMBS; ++l) {
            uint64_t v = ~mag[l] + carry;
            carry = (carry && v == 0) ? 1 : 0;
            mag[l] = v;
        }
    }
    int top = -1;
    for (int pos = ACC_LIMBS * 64 - 1; pos >= 0; --pos)
        if (acc_bit(mag, pos)) { top = pos; break; }
    if (top < 0) return 0.0;
    /* 53 significant bits: positions top .. top-52 */
    uint64_t sig = 0;
    for (int j = 0; j < 53; ++j) {
        int pos = top - j;
        sig = (sig << 1) | (uint64_t)(pos >= 0 ? acc_bit(mag, pos) : 0);
    }
    int round_pos = top - 53;
    int round_bit = round_pos >= 0 ? acc_bit(mag, round_pos) : 0;
    int sticky = 0;
    for (int pos = round_pos - 1; pos >= 0 && !sticky; --pos)
        sticky = acc_bit(mag, pos);
    if (round_bit && (sticky || (sig & 1u))) sig += 1; /* nearest, ties to even */
    /* value = sig * 2^(top-52) * 2^-149 (sig may now be 2^53: still exact) */
    double v = ldexp((double)sig, top - 52 - 149);
    return negative ? -v : v;
}

double sbc_oracle_exact_sum(const float *a, const int64_t *idx, int64_t k) {
    uint64_t acc[ACC_LIMBS];
    memset(acc, 0, sizeof(acc));
    for (int64_t j = 0; j < k; ++j) {
        uint32_t bits;
        float v = a[idx[j]];
        memcpy(&bits, &v, 4);
        int negative = (int)(bits >> 31);
        uint32_t e = (bits >> 23) & 0xffu;
        uint64_t m = bits & 0x7fffffu;
        int shift = 0;
        if (e) { m |= 0x800000u; shift = (int)e - 1; } /* normal: m*2^(e-150) */
        acc_add_shifted(acc, m, shift, negative);
    }
    return acc_to_double(acc);
}

/* ------------------------------------------------------------------ */
/* Algorithm 2 (sparse binarisation) + Algorithm 1 residual write-back */
/* ------------------------------------------------------------------ */

static int cmp_i64(const void *x, const void *y) {
    int64_t a = *(const int64_t *)x, b = *(const int64_t *)y;
    return (a > b) - (a < b);
}

void sbc_oracle_side_and_mu(double sum_top, double sum_bottom, int64_t k, int *side,
                            float *mu32, double *mu_pos, double *mu_neg) {
    /* Algorithm 2: mu+ = mean(val+), mu- = mean(val-) with val- the negated k smallest;
     * "if mu+ >= mu-" keeps the positive side; the value sent is mu+ or -mu-. */
    double mp = sum_top / (double)k;
    double mn = -sum_bottom / (double)k;
    if (mp >= mn) { *side = 0; *mu32 = (float)mp; }
    else          { *side = 1; *mu32 = (float)(-mn); }
    if (mu_pos) *mu_pos = mp;
    if (mu_neg) *mu_neg = mn;
}

int sbc_oracle_compress(float *a, int64_t n, int64_t k, int64_t *kept_sorted,
                        int *side, float *mu32, double *mu_pos,
                        double *mu_neg) {
    if (n <= 0 || k < 1 || k > n) return -2;
    int64_t *pos_idx = (int64_t *)malloc((size_t)k * sizeof(int64_t));
    int64_t *neg_idx = (int64_t *)malloc((size_t)k * sizeof(int64_t));
    if (!pos_idx || !neg_idx) { free(pos_idx); free(neg_idx); return -2; }

    /* val+ = top_p(dW), val- = top_p(-dW) */
    sbc_oracle_topk(a, n, k, 0, pos_idx);
    sbc_oracle_topk(a, n, k, 1, neg_idx);

    /* mu+ = mean(val+), mu- = mean(val-); val- holds the negated entries */
    double mp, mn;
    float mu;
    sbc_oracle_side_and_mu(sbc_oracle_exact_sum(a, pos_idx, k), sbc_oracle_exact_sum(a, neg_idx, k),
                           k, side, &mu, &mp, &mn);
    const int64_t *kept = *side ? neg_idx : pos_idx;

    /* R = dW - dW*: dW* is mu on the kept positions and 0 elsewhere */
    for (int64_t j = 0; j < k; ++j) {
        volatile float r = a[kept[j]] - mu; /* one fp32 subtract */
        a[kept[j]] = r;
    }

    memcpy(kept_sorted, kept, (size_t)k * sizeof(int64_t));
    qsort(kept_sorted, (size_t)k, sizeof(int64_t), cmp_i64);

    *mu32 = mu;
    if (mu_pos) *mu_pos = mp;
    if (mu_neg) *mu_neg = mn;
    free(pos_idx);
    free(neg_idx);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Algorithm 3: Golomb position encoding                               */
/* ------------------------------------------------------------------ */

uint64_t sbc_oracle_payload_bits_bound(int64_t n, int64_t k, int b) {
    return (uint64_t)k * (uint64_t)(1 + b) + ((uint64_t)(n - k) >> b);
}

typedef struct {
    uint8_t *bytes;
    size_t cap_bytes;
    uint64_t nbits;
    int overflow;
} bitsink_t;

static void msg_add(bitsink_t *s, int bit) {
    uint64_t i = s->nbits;
    if (i / 8 >= s->cap_bytes) { s->overflow = 1; return; }
    if (i % 8 == 0) s->bytes[i / 8] = 0;
    if (bit) s->bytes[i / 8] |= (uint8_t)(0x80u >> (i % 8)); /* MSB first */
    s->nbits = i + 1;
}

uint64_t sbc_oracle_golomb_encode(const int64_t *I, int64_t k, int b,
                                  uint8_t *payload, size_t cap_bytes) {
    bitsink_t s = {payload, cap_bytes, 0, 0};
    int64_t prev = -1; /* 0-based positions: the first distance counts from -1 */
    for (int64_t i = 0; i < k; ++i) {
        int64_t d = I[i] - prev; /* d >= 1 */
        prev = I[i];
        uint64_t q = (uint64_t)(d - 1) >> b;
        uint64_t r = (uint64_t)(d - 1) & ((1ull << b) - 1);
        for (uint64_t u = 0; u < q; ++u) msg_add(&s, 1);
        msg_add(&s, 0);
        for (int t = b - 1; t >= 0; --t) msg_add(&s, (int)((r >> t) & 1u));
        if (s.overflow) return UINT64_MAX;
    }
    return s.nbits;
}

/* ------------------------------------------------------------------ */
/* Algorithm 4: Golomb position decoding (bit-serial, as printed)      */
/* ------------------------------------------------------------------ */

static int msg_bit(const uint8_t *bytes, uint64_t i) {
    return (bytes[i / 8] >> (7 - (i % 8))) & 1;
}

int64_t sbc_oracle_golomb_decode(const uint8_t *msg, uint64_t nbits, int b,
                                 float mu, float *dense, int64_t n) {
    uint64_t i = 0, q = 0;
    int64_t j = 0; /* 1-based running position, as in the paper */
    int64_t count = 0;
    while (i < nbits) {
        if (msg_bit(msg, i) == 0) {
            if (i + (uint64_t)b >= nbits)
                return -1; /* message ends inside the remainder field */
            uint64_t r = 0;
            for (int t = 1; t <= b; ++t) r = (r << 1) | (uint64_t)msg_bit(msg, i + t);
            j = j + (int64_t)(q << b) + (int64_t)r + 1;
            if (j < 1 || j > n) return -1;
            dense[j - 1] += mu; /* dW*_j <- mu on a zeroed tensor; += to aggregate */
            q = 0;
            i = i + (uint64_t)b + 1;
            ++count;
        } else {
            q = q + 1;
            i = i + 1;
        }
    }
    if (q != 0) return -1; /* trailing ones without a terminator */
    return count;
}

/* ------------------------------------------------------------------ */
/* Container: header | chunk table | payload (project convention)      */
/* ------------------------------------------------------------------ */
/*
 * The paper's message is the Golomb bit string plus one fp32 mean per tensor
 * ("Optimal Position Encoding"); shapes are known to both sides.  The
 * container adds what a parallel decoder needs and nothing that changes the
 * payload: a 64-byte little-endian header and, for every run of C codewords
 * ("chunk"), the bit offset of the run's first codeword and the position
 * decoded just before it (-1 for the first run).  C depends on the number of
 * positions k alone (sbc_oracle_chunk_codewords): short messages get short
 * chunks, so that a decoder that gives every chunk to one worker still has
 * many chunks to hand out.
 *
 *   0  u32 magic      4  u32 version     8  u64 numel      16 u64 k
 *   24 u64 nbits      32 u64 payload_offset (bytes)        40 u32 b
 *   44 u32 side       48 f32 mu          52 u32 chunk_codewords
 *   56 u32 n_chunks   60 u32 status (0 = ok)
 */

static void put_u32(uint8_t *p, uint32_t v) {
    for (int i = 0; i < 4; ++i) p[i] = (uint8_t)(v >> (8 * i));
}
static void put_u64(uint8_t *p, uint64_t v) {
    for (int i = 0; i < 8; ++i) p[i] = (uint8_t)(v >> (8 * i));
}
static uint32_t get_u32(const uint8_t *p) {
    uint32_t v = 0;
    for (int i = 0; i < 4; ++i) v |= (uint32_t)p[i] << (8 * i);
    return v;
}
static uint64_t get_u64(const uint8_t *p) {
    uint64_t v = 0;
    for (int i = 0; i < 8; ++i) v |= (uint64_t)p[i] << (8 * i);
    return v;
}

/* Codewords per chunk-table entry (project convention): 32 below 2^17
 * positions, 64 below 2^21, 256 from there on. */
uint32_t sbc_oracle_chunk_codewords(int64_t k) {
    if (k < ((int64_t)1 << 17)) return 32u;
    if (k < ((int64_t)1 << 21)) return 64u;
    return 256u;
}

static uint64_t n_chunks_for(int64_t k) {
    uint64_t c = sbc_oracle_chunk_codewords(k);
    return ((uint64_t)k + c - 1) / c;
}

static size_t round_up16(size_t x) { return (x + 15u) & ~(size_t)15u; }

size_t sbc_oracle_container_bytes(int64_t k, uint64_t nbits) {
    size_t payload_offset =
        SBC_ORACLE_HEADER_BYTES + SBC_ORACLE_CHUNK_ENTRY_BYTES * (size_t)n_chunks_for(k);
    return payload_offset + round_up16((size_t)((nbits + 7) / 8));
}

size_t sbc_oracle_stream_bytes(int64_t n, double p) {
    int64_t k = sbc_oracle_kept_count(n, p);
    int b = sbc_oracle_golomb_b(p);
    return sbc_oracle_container_bytes(k, sbc_oracle_payload_bits_bound(n, k, b));
}

int sbc_oracle_container(const int64_t *I, int64_t k, int64_t n, int b, int side, float mu,
                         uint8_t *out, size_t cap, size_t *out_len) {
    /* Algorithm 3 into the payload area */
    uint64_t nchunks = n_chunks_for(k);
    size_t payload_offset = SBC_ORACLE_HEADER_BYTES + SBC_ORACLE_CHUNK_ENTRY_BYTES * (size_t)nchunks;
    if (cap < payload_offset) return -3;
    uint64_t nbits = sbc_oracle_golomb_encode(I, k, b, out + payload_offset, cap - payload_offset);
    if (nbits == UINT64_MAX) return -3;
    size_t total = sbc_oracle_container_bytes(k, nbits);
    if (cap < total) return -3;
    for (size_t z = payload_offset + (size_t)((nbits + 7) / 8); z < total; ++z) out[z] = 0;

    /* chunk table: bit offset of codeword c*C and the position before it */
    uint64_t bit_off = 0;
    int64_t prev = -1;
    const int64_t chunk = (int64_t)sbc_oracle_chunk_codewords(k);
    for (int64_t i = 0; i < k; ++i) {
        if (i % chunk == 0) {
            uint8_t *e = out + SBC_ORACLE_HEADER_BYTES +
                         SBC_ORACLE_CHUNK_ENTRY_BYTES * (size_t)(i / chunk);
            put_u64(e, bit_off);
            put_u64(e + 8, (uint64_t)prev);
        }
        uint64_t g = (uint64_t)(I[i] - prev - 1);
        bit_off += (g >> b) + 1 + (uint64_t)b;
        prev = I[i];
    }

    uint32_t mu_bits;
    memcpy(&mu_bits, &mu, 4);
    put_u32(out + 0, SBC_ORACLE_MAGIC);
    put_u32(out + 4, SBC_ORACLE_VERSION);
    put_u64(out + 8, (uint64_t)n);
    put_u64(out + 16, (uint64_t)k);
    put_u64(out + 24, nbits);
    put_u64(out + 32, (uint64_t)payload_offset);
    put_u32(out + 40, (uint32_t)b);
    put_u32(out + 44, (uint32_t)side);
    put_u32(out + 48, mu_bits);
    put_u32(out + 52, sbc_oracle_chunk_codewords(k));
    put_u32(out + 56, (uint32_t)nchunks);
    put_u32(out + 60, 0u);
    if (out_len) *out_len = total;
    return 0;
}

int sbc_oracle_encode(const float *update, float *residual, int64_t n, double p,
                      uint8_t *out, size_t cap, size_t *out_len, float *out_mu) {
    if (!update || !residual || !out || n <= 0 || n >= ((int64_t)1 << 31) ||
        !(p > 0.0 && p < 1.0))
        return -2;
    int64_t k = sbc_oracle_kept_count(n, p);
    int b = sbc_oracle_golomb_b(p);
    if (b > 30) return -2;

    /* Algorithm 1: dW_i = R_i + (SGD_n(W_i) - W_i) */
    if (sbc_oracle_accumulate(update, residual, n) != 0) return -1;

    /* Algorithm 2 and R_i = dW_i - dW_i* */
    int64_t *I = (int64_t *)malloc((size_t)k * sizeof(int64_t));
    if (!I) return -2;
    int side;
    float mu;
    sbc_oracle_compress(residual, n, k, I, &side, &mu, NULL, NULL);

    int rc = sbc_oracle_container(I, k, n, b, side, mu, out, cap, out_len);
    if (rc == 0 && out_mu) *out_mu = mu;
    free(I);
    return rc;
}

/* ------------------------------------------------------------------ */
/* Gradient Dropping (the paper's sparsification baseline, Section 1   */
/* and Table 1): top-p by magnitude, the values themselves are sent    */
/* ------------------------------------------------------------------ */

static int ranked_abs_desc(const void *x, const void *y) {
    return ranked_desc(x, y); /* v already holds |a| */
}

int sbc_oracle_topk_abs(const float *a, int64_t n, int64_t k, int64_t *out_idx) {
    if (n <= 0 || k < 0 || k > n) return -2;
    ranked_t *r = (ranked_t *)malloc((size_t)n * sizeof(ranked_t));
    if (!r) return -2;
    for (int64_t i = 0; i < n; ++i) { r[i].v = fabsf(a[i]); r[i].i = i; }
    qsort(r, (size_t)n, sizeof(ranked_t), ranked_abs_desc);
    for (int64_t j = 0; j < k; ++j) out_idx[j] = r[j].i;
    free(r);
    return 0;
}

/* Algorithm 4 with one value per position instead of one mean: dense[j] += values[i] at the
 * i-th decoded position.  values: k little-endian fp32. */
int64_t sbc_oracle_golomb_decode_values(const uint8_t *msg, uint64_t nbits, int b,
                                        const uint8_t *values, int64_t k, float *dense, int64_t n) {
    uint64_t i = 0, q = 0;
    int64_t j = 0, count = 0;
    while (i < nbits) {
        if (msg_bit(msg, i) == 0) {
            if (i + (uint64_t)b >= nbits) return -1;
            uint64_t r = 0;
            for (int t = 1; t <= b; ++t) r = (r << 1) | (uint64_t)msg_bit(msg, i + t);
            j = j + (int64_t)(q << b) + (int64_t)r + 1;
            if (j < 1 || j > n || count >= k) return -1;
            uint32_t bits = get_u32(values + 4 * (size_t)count);
            float v;
            memcpy(&v, &bits, 4);
            dense[j - 1] += v;
            q = 0;
            i = i + (uint64_t)b + 1;
            ++count;
        } else {
            q = q + 1;
            i = i + 1;
        }
    }
    if (q != 0) return -1;
    return count;
}

size_t sbc_oracle_stream_bytes_values(int64_t n, double p) {
    int64_t k = sbc_oracle_kept_count(n, p);
    return sbc_oracle_stream_bytes(n, p) + round_up16((size_t)k * 4);
}

int sbc_oracle_encode_values(const float *update, float *residual, int64_t n, double p,
                             uint8_t *out, size_t cap, size_t *out_len) {
    if (!update || !residual || !out || n <= 0 || n >= ((int64_t)1 << 31) || !(p > 0.0 && p < 1.0))
        return -2;
    int64_t k = sbc_oracle_kept_count(n, p);
    int b = sbc_oracle_golomb_b(p);
    if (b > 30) return -2;
    if (sbc_oracle_accumulate(update, residual, n) != 0) return -1; /* dW = R + update */
    int64_t *I = (int64_t *)malloc((size_t)k * sizeof(int64_t));
    if (!I) return -2;
    sbc_oracle_topk_abs(residual, n, k, I);                /* the fraction p with the biggest magnitude */
    qsort(I, (size_t)k, sizeof(int64_t), cmp_i64);

    uint64_t nchunks = n_chunks_for(k);
    size_t values_offset = SBC_ORACLE_HEADER_BYTES + SBC_ORACLE_CHUNK_ENTRY_BYTES * (size_t)nchunks;
    size_t payload_offset = values_offset + round_up16((size_t)k * 4);
    if (cap < payload_offset) { free(I); return -3; }
    memset(out + values_offset, 0, payload_offset - values_offset);
    for (int64_t i = 0; i < k; ++i) {
        uint32_t bits;
        float v = residual[I[i]];                          /* dW*_j = dW_j on the kept positions */
        memcpy(&bits, &v, 4);
        put_u32(out + values_offset + 4 * (size_t)i, bits);
        volatile float r = v - v;                          /* R = dW - dW* */
        residual[I[i]] = r;
    }
    uint64_t nbits = sbc_oracle_golomb_encode(I, k, b, out + payload_offset, cap - payload_offset);
    if (nbits == UINT64_MAX) { free(I); return -3; }
    size_t total = payload_offset + round_up16((size_t)((nbits + 7) / 8));
    if (cap < total) { free(I); return -3; }
    for (size_t z = payload_offset + (size_t)((nbits + 7) / 8); z < total; ++z) out[z] = 0;
    uint64_t bit_off = 0;
    int64_t prev = -1;
    const int64_t chunk = (int64_t)sbc_oracle_chunk_codewords(k);
    for (int64_t i = 0; i < k; ++i) {
        if (i % chunk == 0) {
            uint8_t *e = out + SBC_ORACLE_HEADER_BYTES +
                         SBC_ORACLE_CHUNK_ENTRY_BYTES * (size_t)(i / chunk);
            put_u64(e, bit_off);
            put_u64(e + 8, (uint64_t)prev);
        }
        uint64_t g = (uint64_t)(I[i] - prev - 1);
        bit_off += (g >> b) + 1 + (uint64_t)b;
        prev = I[i];
    }
    put_u32(out + 0, SBC_ORACLE_MAGIC);
    put_u32(out + 4, SBC_ORACLE_VERSION);
    put_u64(out + 8, (uint64_t)n);
    put_u64(out + 16, (uint64_t)k);
    put_u64(out + 24, nbits);
    put_u64(out + 32, (uint64_t)payload_offset);
    put_u32(out + 40, (uint32_t)b);
    put_u32(out + 44, SBC_ORACLE_SIDE_VALUES);
    put_u32(out + 48, 0u);
    put_u32(out + 52, sbc_oracle_chunk_codewords(k));
    put_u32(out + 56, (uint32_t)nchunks);
    put_u32(out + 60, 0u);
    if (out_len) *out_len = total;
    free(I);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Sparse binarisation with thresholds from a random subsample         */
/* (Section 2, "Sparse Binarization": subsampling reduces the cost of  */
/* the selection and adds noise to the amount of sparsity)             */
/* ------------------------------------------------------------------ */

static int cmp_float_desc(const void *x, const void *y) {
    float a = *(const float *)x, b = *(const float *)y;
    return (a < b) - (a > b);
}

int sbc_oracle_encode_sampled(const float *update, float *residual, int64_t n, double p,
                              const uint32_t *sample_idx, int64_t m, uint8_t *out, size_t cap,
                              size_t *out_len, float *out_mu) {
    if (!update || !residual || !out || !sample_idx || m <= 0 || n <= 0 || n >= ((int64_t)1 << 31) ||
        !(p > 0.0 && p < 1.0))
        return -2;
    int64_t k = sbc_oracle_kept_count(n, p);
    int b = sbc_oracle_golomb_b(p);
    if (b > 30) return -2;
    if (sbc_oracle_accumulate(update, residual, n) != 0) return -1;
    float *a = residual;

    /* thresholds: the floor(p*m)-th largest and smallest of the sampled entries */
    float *sv = (float *)malloc((size_t)m * sizeof(float));
    if (!sv) return -2;
    for (int64_t i = 0; i < m; ++i) {
        if (sample_idx[i] >= (uint64_t)n) { free(sv); return -2; }
        sv[i] = a[sample_idx[i]];
    }
    qsort(sv, (size_t)m, sizeof(float), cmp_float_desc);
    int64_t j = (int64_t)floor(p * (double)m);
    if (j < 1) j = 1;
    float t_pos = sv[j - 1], t_neg = sv[m - j];
    free(sv);

    /* val+ = everything at or above t+, val- = everything at or below t- */
    int64_t limit = 2 * k + 1024;
    if (limit > n) limit = n;
    int64_t n_pos = 0, n_neg = 0;
    for (int64_t i = 0; i < n; ++i) { n_pos += a[i] >= t_pos; n_neg += a[i] <= t_neg; }
    int64_t *I;
    int side;
    float mu;
    int64_t kept_count;
    if (n_pos >= 1 && n_pos <= limit && n_neg >= 1 && n_neg <= limit) {
        int64_t *P = (int64_t *)malloc((size_t)n_pos * sizeof(int64_t));
        int64_t *N = (int64_t *)malloc((size_t)n_neg * sizeof(int64_t));
        if (!P || !N) { free(P); free(N); return -2; }
        int64_t ip = 0, in = 0;
        for (int64_t i = 0; i < n; ++i) {
            if (a[i] >= t_pos) P[ip++] = i;
            if (a[i] <= t_neg) N[in++] = i;
        }
        double mp = sbc_oracle_exact_sum(a, P, n_pos) / (double)n_pos;   /* mean(val+) */
        double mn = -sbc_oracle_exact_sum(a, N, n_neg) / (double)n_neg;  /* mean(val-) */
        if (mp >= mn) { side = 0; mu = (float)mp; I = P; kept_count = n_pos; free(N); }
        else          { side = 1; mu = (float)(-mn); I = N; kept_count = n_neg; free(P); }
        for (int64_t q = 0; q < kept_count; ++q) {
            volatile float r = a[I[q]] - mu;
            a[I[q]] = r;
        }
    } else { /* estimate rejected: Algorithm 2 with exactly k entries per side */
        I = (int64_t *)malloc((size_t)k * sizeof(int64_t));
        if (!I) return -2;
        sbc_oracle_compress(a, n, k, I, &side, &mu, NULL, NULL);
        kept_count = k;
    }
    int rc = sbc_oracle_container(I, kept_count, n, b, side, mu, out, cap, out_len);
    if (rc == 0 && out_mu) *out_mu = mu;
    free(I);
    return rc;
}

int sbc_oracle_decode_accumulate(const uint8_t *const *streams, int n_clients,
                                 float *out_dense, int64_t n) {
    if (!streams || !out_dense || n_clients < 0 || n <= 0) return -2;
    for (int c = 0; c < n_clients; ++c) { /* sum over i in I_t, client order */
        const uint8_t *s = streams[c];
        if (!s) return -2;
        if (get_u32(s + 0) != SBC_ORACLE_MAGIC || get_u32(s + 4) != SBC_ORACLE_VERSION ||
            get_u32(s + 60) != 0u || get_u64(s + 8) != (uint64_t)n)
            return -4;
        uint64_t k = get_u64(s + 16), nbits = get_u64(s + 24), off = get_u64(s + 32);
        uint32_t b = get_u32(s + 40), mu_bits = get_u32(s + 48);
        if (b > 30 || k > (uint64_t)n) return -4;
        float mu;
        memcpy(&mu, &mu_bits, 4);
        int64_t got;
        if (get_u32(s + 44) == SBC_ORACLE_SIDE_VALUES) /* one fp32 value per position, before the payload */
            got = sbc_oracle_golomb_decode_values(s + off, nbits, (int)b,
                                                  s + SBC_ORACLE_HEADER_BYTES + SBC_ORACLE_CHUNK_ENTRY_BYTES * n_chunks_for((int64_t)k),
                                                  (int64_t)k, out_dense, n);
        else
            got = sbc_oracle_golomb_decode(s + off, nbits, (int)b, mu, out_dense, n);
        if (got < 0 || (uint64_t)got != k) return -4;
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Algorithm 1, server lines: dW = 1/|I_t| * sum dW_i*,  W = W + dW    */
/* and momentum masking (Supplement): zero the momentum where a weight */
/* was updated by a transmitted entry                                  */
/* ------------------------------------------------------------------ */

int sbc_oracle_decode_apply(const uint8_t *const *streams, int n_clients, float scale,
                            float *weights, float *momentum, int64_t n) {
    if (!streams || !weights || n_clients < 0 || n <= 0) return -2;
    float *sum = (float *)calloc((size_t)n, sizeof(float));
    float *hit = (float *)calloc((size_t)n, sizeof(float));
    if (!sum || !hit) { free(sum); free(hit); return -2; }
    int rc = sbc_oracle_decode_accumulate(streams, n_clients, sum, n); /* sum over i in I_t */
    for (int c = 0; rc == 0 && c < n_clients; ++c) { /* positions any client transmitted */
        const uint8_t *s = streams[c];
        int64_t got = sbc_oracle_golomb_decode(s + get_u64(s + 32), get_u64(s + 24),
                                               (int)get_u32(s + 40), 1.0f, hit, n);
        if (got < 0) rc = -4;
    }
    for (int64_t j = 0; rc == 0 && j < n; ++j) {
        volatile float d = scale * sum[j];      /* dW_j = 1/|I_t| * sum */
        volatile float w = weights[j] + d;      /* W_j = W_j + dW_j */
        weights[j] = w;
        if (momentum && hit[j] != 0.0f) momentum[j] = 0.0f;
    }
    free(sum);
    free(hit);
    return rc;
}
