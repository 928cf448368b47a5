/*
 * sbc_oracle.h -- CPU oracle for Sparse Binary Compression (arXiv 1805.08768).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded statement
 * of what the method computes, written from the paper so that a reader can
 * check it by eye.  It shares no code with the CUDA library, is never linked
 * into it and is never called by it.  Only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may use it.
 *
 * Steps follow the paper's order and notation:
 *   Algorithm 1 (client lines: residual accumulate, residual write-back,
 *                server line: sum of the decoded updates)
 *   Algorithm 2 (sparse binarisation: two-sided top-p, means, side choice)
 *   Algorithm 3 (Golomb position encoding, b* from p)
 *   Algorithm 4 (Golomb position decoding, supplement)
 *   Eq. for the mean position bits  b_pos = b* + 1 / (1 - (1-p)^(2^b*)).
 *
 * Readings taken where the paper is silent:
 *   k = max(1, floor(p*n)) (fp64 product), exactly k entries kept per side,
 *   equal values ordered by lower flat index first, -0 == +0, signed top-k as
 *   Algorithm 2 writes it, the two sums exact (rounded once to fp64), mean =
 *   sum / k in fp64, ">=" picks the positive side, the transmitted value is
 *   the fp32 rounding of the chosen mean (negated for the negative side) and
 *   that same fp32 value is subtracted from the kept residual entries,
 *   0-based positions with the first gap counted from -1, remainder bits
 *   MSB-first, stream bit i in byte i/8 at bit 7-(i%8).
 *
 * Parity pins (tests/test_oracle_*.py): brute-force stable argsort, Python
 * big-integer / math.fsum exact sums, hand-computed Golomb codes, the
 * paper's b* / b_pos closed forms, decode(encode(x)) round trip, the residual
 * identity of Eq. (residual), the least-squares property of Theorem 2.1.
 * Unpinned conventions (no statement in the paper to check against): the
 * rounding of p*n, the bit/byte order, and the container around the payload
 * (header + chunk table) -- "parity unpinned" for those three.
 */
#ifndef SBC_ORACLE_H
#define SBC_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Container constants (a convention of this project, not of the paper). */
#define SBC_ORACLE_MAGIC 0x31434253u /* "SBC1" little-endian */
#define SBC_ORACLE_VERSION 1u
#define SBC_ORACLE_HEADER_BYTES 64u
#define SBC_ORACLE_CHUNK_ENTRY_BYTES 16u
#define SBC_ORACLE_SIDE_VALUES 2u /* header 'side' of a stream that carries one value per position */

/* Codewords per chunk-table entry of a message with k positions: 32 below
 * 2^17 positions, 64 below 2^21, 256 from there on (a convention of this
 * project, "parity unpinned"; the header carries the value). */
uint32_t sbc_oracle_chunk_codewords(int64_t k);

/* k = max(1, floor(p*n)), at most n.  (Algorithm 2, "top p%"; reading S1.) */
int64_t sbc_oracle_kept_count(int64_t n, double p);

/* b* = 1 + floor(log2(log(phi-1)/log(1-p))), clamped at 0.  (Algorithm 3.) */
int sbc_oracle_golomb_b(double p);

/* Mean position bits b + 1/(1-(1-p)^(2^b)).  (Eq. for b_pos.) */
double sbc_oracle_mean_position_bits(double p, int b);

/* A_i = fl32(R_i + dW_i), written over the residual.  (Algorithm 1, client
 * accumulate line.)  Returns 0, or -1 if any A_i is not finite. */
int sbc_oracle_accumulate(const float *update, float *residual, int64_t n);

/* Indices of the k largest entries of a (negate = 0) or of -a (negate = 1),
 * in rank order; equal values: lower index first.  Full sort, then the first
 * k.  (Algorithm 2, top_p(dW) and top_p(-dW).) */
int sbc_oracle_topk(const float *a, int64_t n, int64_t k, int negate,
                    int64_t *out_idx);

/* Correctly rounded fp64 value of the exact sum of a[idx[0..k)]. */
double sbc_oracle_exact_sum(const float *a, const int64_t *idx, int64_t k);

/* Algorithm 2 + the residual line of Algorithm 1 on an accumulated tensor A
 * (in: A, out: R_new in place).  kept_sorted receives the k kept positions in
 * ascending order.  side: 0 positive, 1 negative.  mu_pos / mu_neg are the
 * two fp64 means (mu_neg is the mean of the negated k smallest). */
int sbc_oracle_compress(float *a_inout, int64_t n, int64_t k,
                        int64_t *kept_sorted, int *side, float *mu32,
                        double *mu_pos, double *mu_neg);

/* Algorithm 2's decision from the two (exactly rounded) sums: sum_top over the
 * k largest entries, sum_bottom over the k smallest.  mu+ = sum_top/k,
 * mu- = -sum_bottom/k; side 0 iff mu+ >= mu-; mu32 = (float)mu+ or (float)(-mu-). */
void sbc_oracle_side_and_mu(double sum_top, double sum_bottom, int64_t k, int *side,
                            float *mu32, double *mu_pos, double *mu_neg);

/* Upper bound on payload bits: k(1+b) + floor((n-k)/2^b). */
uint64_t sbc_oracle_payload_bits_bound(int64_t n, int64_t k, int b);

/* Algorithm 3 on an ascending position list.  Writes ceil(nbits/8) bytes
 * (zero pad bits), returns nbits, or UINT64_MAX if cap_bytes is too small. */
uint64_t sbc_oracle_golomb_encode(const int64_t *sorted_idx, int64_t k, int b,
                                  uint8_t *payload, size_t cap_bytes);

/* Algorithm 4, bit by bit, on nbits of payload: dense[j] += mu at every
 * decoded position (the dense tensor is the caller's; zero it to get the
 * paper's dW*).  Returns the number of positions decoded, or -1 if a position
 * falls outside [0, n) or the message ends inside a codeword. */
int64_t sbc_oracle_golomb_decode(const uint8_t *payload, uint64_t nbits, int b,
                                 float mu, float *dense, int64_t n);

/* Bytes of a container holding nbits of payload for k codewords. */
size_t sbc_oracle_container_bytes(int64_t k, uint64_t nbits);
/* Capacity bound for (n, p): container_bytes(k, payload_bits_bound). */
size_t sbc_oracle_stream_bytes(int64_t n, double p);

/* Container (header, chunk table, Algorithm 3 payload) for an ascending
 * position list.  Returns 0, or -3 if cap is too small. */
int sbc_oracle_container(const int64_t *sorted_idx, int64_t k, int64_t n, int b, int side,
                         float mu, uint8_t *out, size_t cap, size_t *out_len);

/* Whole client step: accumulate, compress, residual write-back, encode into a
 * container (header, chunk table, payload).  Returns 0 on success, -1 for
 * non-finite input, -2 for bad arguments, -3 if cap is too small.
 * out_len: bytes written.  out_mu: the signed fp32 value transmitted. */
int sbc_oracle_encode(const float *update, float *residual, int64_t n, double p,
                      uint8_t *out_stream, size_t cap, size_t *out_len,
                      float *out_mu);

/* Server step: for every client in order, parse its container and add its
 * decoded sparse tensor into out_dense (fp32 adds).  (Algorithm 1, server sum
 * line without the 1/|I_t| factor; Algorithm 4.)  Returns 0 or a negative
 * error (-4 corrupt container). */
int sbc_oracle_decode_accumulate(const uint8_t *const *streams, int n_clients,
                                 float *out_dense, int64_t n);

/* Gradient Dropping, the sparsification baseline the paper compares with (Section 1: "only
 * communicate the fraction p entries of the gradient with the biggest magnitude, while also
 * collecting all other gradients in a residual"; Table 1: 32 value bits + position bits):
 * A = R + update; kept = the k entries of largest |A| (equal magnitudes: lower index first);
 * the kept values themselves are sent; R_new = A off the kept set and A - A on it.
 * Container: header (side = 2, mu = 0) | chunk table | k fp32 values in position order, padded
 * to 16 bytes | Algorithm 3 payload.  Decoding such a stream adds values[i] at the i-th position. */
int sbc_oracle_topk_abs(const float *a, int64_t n, int64_t k, int64_t *out_idx);
size_t sbc_oracle_stream_bytes_values(int64_t n, double p);
int sbc_oracle_encode_values(const float *update, float *residual, int64_t n, double p,
                             uint8_t *out, size_t cap, size_t *out_len);
int64_t sbc_oracle_golomb_decode_values(const uint8_t *payload, uint64_t nbits, int b,
                                        const uint8_t *values, int64_t k, float *dense, int64_t n);

/* Sparse binarisation with thresholds from a subsample (Section 2, "Sparse Binarization": the
 * selection can be made cheaper "by randomly subsampling from W", which adds noise to the amount
 * of sparsity).  The caller supplies the m sample positions.  j = max(1, floor(p*m)); t+ / t- =
 * the j-th largest / smallest sampled entry of A = R + update; val+ = ALL entries >= t+, val- =
 * ALL entries <= t-; means over those sets, side choice, binarisation, residual and container as
 * in the exact method, with k = size of the kept set.  If either set is empty or larger than
 * min(n, 2*kept_count(n,p) + 1024) the estimate is rejected and the exact method is used.
 * cap: at least sbc_oracle_container_bytes(limit, limit*(1+b) + 2*(n >> b)). */
int sbc_oracle_encode_sampled(const float *update, float *residual, int64_t n, double p,
                              const uint32_t *sample_idx, int64_t m, uint8_t *out, size_t cap,
                              size_t *out_len, float *out_mu);

/* Server / client apply step (Algorithm 1: "dW <- 1/|I_t| sum dW_i*", "W <- W + dW") with
 * momentum masking (Supplement): weights[j] = fl32(weights[j] + fl32(scale * sum_j)) for every
 * j, sum_j the fp32 sum of the decoded client tensors in client order; momentum[j] = 0 at every
 * position some client transmitted (momentum may be NULL).  scale is 1/|I_t| for the paper's
 * average.  Returns 0 or a negative error. */
int sbc_oracle_decode_apply(const uint8_t *const *streams, int n_clients, float scale,
                            float *weights, float *momentum, int64_t n);

#ifdef __cplusplus
}
#endif
#endif /* SBC_ORACLE_H */
