/*
 * sbc.h -- C ABI of the B200 Sparse Binary Compression library.
 *
 * Sparse Binary Compression (Sattler, Wiedemann, Mueller, Samek,
 * arXiv 1805.08768) sends, per tensor and per communication round, the
 * positions of a p-fraction of a client's accumulated weight update plus ONE
 * fp32 value.  This library is the per-tensor hot path of that scheme on one
 * NVIDIA B200 (sm_100a): the client-side encode and the server-side
 * decode-and-sum.  Everything below runs as CUDA kernels on the caller's
 * stream; there is no CPU fallback.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA global-memory addresses on the current
 *     device, "host" pointers are ordinary process memory.
 *   - The caller owns every buffer.  Except where an entry point says
 *     otherwise the library allocates nothing and keeps no state between
 *     calls.
 *   - Device work is enqueued on `stream` and the call returns without
 *     waiting for it, unless the entry point says that it synchronises.
 *   - Return value: SBC_OK or a negative sbc_status code.  Errors the host
 *     can see (null or misaligned pointer, size out of range, capacity too
 *     small) are returned at once and nothing is enqueued.  Errors only the
 *     device can see (non-finite input, corrupt stream) are recorded in the
 *     stream header's status word / the status word passed to the decoder
 *     and the kernels stop writing results; they never trap.
 *   - Positions are flat 0-based element indices, numel < 2^31.
 */
#ifndef SBC_H
#define SBC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Same type as cudaStream_t (an opaque driver handle); 0 is the default stream. */
typedef struct CUstream_st *sbc_cuda_stream_t;

enum sbc_status {
    SBC_OK = 0,
    SBC_EINVAL = -1,     /* bad argument */
    SBC_ECAPACITY = -2,  /* an output or workspace buffer is too small */
    SBC_ENONFINITE = -3, /* residual + update holds an Inf or NaN */
    SBC_ECORRUPT = -4,   /* a stream failed validation while decoding */
    SBC_ETIMEOUT = -5,   /* a bounded device-side wait gave up (the exact route's grid barrier) */
    SBC_ECUDA = -6       /* a CUDA runtime call failed */
};

/* Bits of the device-side status words (stream header offset 60, decoder status word). */
#define SBC_STATUS_NONFINITE 0x1u
#define SBC_STATUS_CORRUPT 0x2u
#define SBC_STATUS_RANGE 0x4u /* a decoded position fell outside [0, numel) */
#define SBC_STATUS_INTERNAL 0x8u
#define SBC_STATUS_TIMEOUT 0x10u /* a bounded device-side wait gave up; the stream holds no payload */

/*
 * Stream container (little-endian).  The paper's message is the Golomb bit
 * string of the position gaps plus one mean value per tensor (Section 2,
 * "Optimal Position Encoding"); tensor shapes are known to both sides
 * (Supplement, "Golomb Position Decoding").  The container keeps that bit
 * string unchanged as its payload and adds what a parallel decoder needs:
 *
 *   bytes 0..63   header
 *      0 u32 magic "SBC1"      4 u32 version (1)     8 u64 numel
 *     16 u64 k (positions)    24 u64 nbits (payload bits)
 *     32 u64 payload_offset   40 u32 b (Golomb parameter b*)
 *     44 u32 side (0: +mu kept, 1: -mu kept, 2: values follow the table)  48 f32 mu (signed)
 *     52 u32 chunk_codewords  56 u32 n_chunks         60 u32 status
 *   bytes 64..    chunk table, n_chunks = ceil(k / chunk_codewords) entries of
 *                 { u64 bit offset of codeword c*chunk_codewords,
 *                   i64 position decoded just before it (-1 for c = 0) }
 *                 chunk_codewords depends on k alone (32 below 2^17 positions,
 *                 64 below 2^21, 256 from there on): a decoder that hands
 *                 every chunk to one worker then has enough chunks to hand
 *                 out for short messages too, at 4, 2 or 0.5 table bits per
 *                 position
 *   payload_offset..  payload: codeword i = q ones, a zero, r in b bits
 *                 (MSB first), where gap-1 = q*2^b + r (Algorithm 3); stream
 *                 bit j is bit 7-(j%8) of byte j/8; zero padded to 16 bytes.
 */
#define SBC_MAGIC 0x31434253u
#define SBC_VERSION 1u
#define SBC_HEADER_BYTES 64u
#define SBC_CHUNK_CODEWORDS_MAX 256u /* chunk_codewords is 32 for k < 2^17 positions, 64 for k < 2^21, else 256 */
#define SBC_CHUNK_ENTRY_BYTES 16u
#define SBC_SIDE_VALUES 2u /* header 'side' of a stream written by sbc_encode_values */

typedef struct sbc_stream_info {
    uint32_t magic, version;
    uint64_t numel, k, nbits, payload_offset;
    uint32_t b, side;
    float mu;
    uint32_t chunk_codewords, n_chunks, status;
    uint64_t total_bytes; /* payload_offset + payload bytes rounded up to 16 */
} sbc_stream_info;

/* ---- host-side pure functions (no CUDA calls) ------------------------- */

/* Number of positions sent for a tensor of numel elements at sparsity p:
 * k = max(1, floor(p * numel)), at most numel.  The paper's top_p% (Algorithm
 * 2) does not say how p*|W| is rounded; this is the convention used here.
 * Returns 0 if numel <= 0 or p is not in (0, 1). */
int64_t sbc_kept_count(int64_t numel, double p);

/* Golomb parameter b* = 1 + floor(log2(log(phi-1)/log(1-p))), phi the golden
 * ratio (Algorithm 3), clamped at 0.  Returns -1 if p is not in (0, 1). */
int sbc_golomb_b(double p);

/* Mean position bits b + 1/(1-(1-p)^(2^b)) (Section 2, equation for b_pos):
 * the expected codeword length when gaps are geometric. */
double sbc_mean_position_bits(double p, int b);

/* Capacity, in bytes, that out_stream must have for sbc_encode(numel, p):
 * header + chunk table + the largest possible payload,
 * k(1+b) + floor((numel-k)/2^b) bits, rounded up to 16 bytes.  0 on bad
 * arguments. */
size_t sbc_stream_bytes(int64_t numel, double p);

/* Bytes of device scratch sbc_encode(numel, p) needs.  0 on bad arguments. */
size_t sbc_workspace_bytes(int64_t numel, double p);

/* ---- client side ------------------------------------------------------- */

/*
 * One client step for one tensor (Algorithm 1, client lines
 * "dW_i <- R_i + ...", "dW_i* <- compress(dW_i)", "R_i <- dW_i - dW_i*",
 * "msg_i <- encode(dW_i*)"; Algorithm 2; Algorithm 3):
 *
 *   A      = residual + update                 (fp32, elementwise)
 *   val+   = the k largest entries of A,  val- = the k largest of -A
 *            (equal values: lower index first; exactly k each)
 *   mu+    = mean(val+), mu- = mean(val-)      (sums exact, one fp64 divide)
 *   kept   = positions of val+ if mu+ >= mu-, else of val-
 *   mu     = (float)mu+  or  (float)(-mu-)
 *   residual = A, except residual[j] = A[j] - mu for j in kept
 *   out_stream = container(kept positions in ascending order, mu)
 *   *out_mu = mu
 *
 * update     device, numel floats, read only, 4-byte aligned (16 preferred)
 * residual   device, numel floats, in: R_old, out: R_new; must not alias update
 * numel      1 .. 2^31-1
 * p          sparsity, 0 < p < 1, with sbc_golomb_b(p) <= 30
 * out_stream device, 16-byte aligned, out_capacity >= sbc_stream_bytes(numel, p)
 * out_mu     device, one float (may be NULL)
 * workspace  device, 256-byte aligned, workspace_bytes >= sbc_workspace_bytes
 *            (numel, p); contents are scratch, nothing carries between calls
 * stream     CUDA stream the work is enqueued on
 *
 * Asynchronous.  If A holds a non-finite value the header's status word gets
 * SBC_STATUS_NONFINITE, residual holds A and no payload is produced; read the
 * header with sbc_stream_info to find out.
 */
int sbc_encode(const float *update, float *residual, int64_t numel, double p,
               void *out_stream, size_t out_capacity, float *out_mu,
               void *workspace, size_t workspace_bytes, sbc_cuda_stream_t stream);

/*
 * Gradient Dropping, the sparsification baseline the paper measures SBC against
 * (Section 1: send the fraction p of entries with the biggest magnitude, collect
 * the rest in a residual; Table 1: 32 value bits per entry), with the same
 * Golomb position code (Algorithm 3):
 *
 *   A        = residual + update
 *   kept     = the k entries of largest |A| (equal magnitudes: lower index first)
 *   residual = A, except residual[j] = 0 for j in kept
 *   out_stream = header (side = SBC_SIDE_VALUES, mu = 0) | chunk table |
 *                k fp32 values A[j] in position order, zero padded to 16 bytes |
 *                Golomb payload of the kept positions
 *
 * out_capacity >= sbc_stream_bytes_values(numel, p); workspace as sbc_encode
 * (sbc_workspace_bytes).  sbc_decode_accumulate / sbc_decode_apply accept such
 * streams and add values[i] (times scale) at the i-th position.  Lets the
 * paper's accounting -- about x3 from binarisation, up to x2 from Golomb coding
 * (Figure 2) -- be measured on the same tensors.
 */
size_t sbc_stream_bytes_values(int64_t numel, double p);
int sbc_encode_values(const float *update, float *residual, int64_t numel, double p,
                      void *out_stream, size_t out_capacity, void *workspace,
                      size_t workspace_bytes, sbc_cuda_stream_t stream);

/*
 * sbc_encode with thresholds estimated from a random subsample (Section 2,
 * "Sparse Binarization": the cost of the selection can be reduced "by randomly
 * subsampling from W", at the price of noise in the amount of sparsity).  The
 * caller draws the sample positions; everything else is deterministic:
 *
 *   j  = max(1, floor(p * sample_count))
 *   t+ = j-th largest, t- = j-th smallest of A[sample_idx[0..sample_count)]
 *   val+ = ALL entries A_i >= t+,  val- = ALL entries A_i <= t-   (about k each)
 *   means over those sets, side choice, binarisation, residual, stream: as
 *   sbc_encode, with the header's k = the size of the kept set.
 *
 * The estimate is accepted if both sets hold between 1 and min(numel, 2k+1024)
 * entries (k = sbc_kept_count); otherwise the call produces exactly what
 * sbc_encode produces.  The selection stage of sbc_encode is skipped, so the
 * call is cheaper by that stage.
 *
 * sample_idx   device, sample_count positions in [0, numel), 4-byte aligned;
 *              a position >= numel sets SBC_STATUS_RANGE in the header
 * sample_count 1 .. 2^20
 * out_capacity >= sbc_stream_bytes_sampled(numel, p)
 * workspace    >= sbc_workspace_bytes_sampled(numel, p, sample_count)
 */
size_t sbc_stream_bytes_sampled(int64_t numel, double p);
size_t sbc_workspace_bytes_sampled(int64_t numel, double p, int64_t sample_count);
int sbc_encode_sampled(const float *update, float *residual, int64_t numel, double p,
                       const uint32_t *sample_idx, int64_t sample_count, void *out_stream,
                       size_t out_capacity, float *out_mu, void *workspace,
                       size_t workspace_bytes, sbc_cuda_stream_t stream);

/*
 * sbc_encode for many tensors at once (a model's parameter tensors in one
 * communication round; the paper applies the method per tensor, with one mean
 * per tensor -- Section 2, "Optimal Position Encoding").  Exactly the results
 * of n_tensors separate sbc_encode calls, but every kernel is launched once
 * for the whole batch, so small tensors do not pay a launch sequence each.
 *
 * descs      HOST array of n_tensors descriptors (fields as the sbc_encode
 *            arguments of the same name; p may differ per tensor).  Read
 *            before the call returns.
 * workspace  device, 256-byte aligned, >= sbc_workspace_bytes_batch(...)
 * If any tensor has a host-visible argument error nothing is enqueued.
 * Device-side errors are reported per tensor in its stream header.
 */
typedef struct sbc_tensor_desc {
    const float *update;
    float *residual;
    int64_t numel;
    double p;
    void *out_stream;
    size_t out_capacity;
    float *out_mu;
} sbc_tensor_desc;
size_t sbc_workspace_bytes_batch(int n_tensors, const sbc_tensor_desc *descs);
int sbc_encode_batch(int n_tensors, const sbc_tensor_desc *descs, void *workspace,
                     size_t workspace_bytes, sbc_cuda_stream_t stream);

/*
 * sbc_encode with timing marks: the same work, plus, when `marks` is not NULL,
 * a cudaEventRecord on `stream` at each stage boundary.  marks is a host array
 * of SBC_MARK_COUNT events the caller created (entries may be NULL).  The
 * interval BOUNDS->COLLECT holds exactly one kernel, the streaming pass that
 * reads update and residual and writes the residual (Algorithm 1's accumulate
 * fused with the candidate gathering for Algorithm 2).
 */
typedef struct CUevent_st *sbc_cuda_event_t; /* same type as cudaEvent_t */
enum sbc_mark {
    SBC_MARK_BEGIN = 0, /* before anything is enqueued */
    SBC_MARK_BOUNDS,    /* scratch cleared, threshold bounds estimated from the sample */
    SBC_MARK_COLLECT,   /* residual = A written, candidate lists gathered */
    SBC_MARK_EXACT,     /* exact-select route over A done (a no-op unless the bounds failed) */
    SBC_MARK_SELECT,    /* k-th entries, means, side and mu found */
    SBC_MARK_END,       /* kept positions walked in order: residual written back, Golomb payload, chunk table and header written */
    SBC_MARK_COUNT
};
int sbc_encode_ex(const float *update, float *residual, int64_t numel, double p,
                  void *out_stream, size_t out_capacity, float *out_mu,
                  void *workspace, size_t workspace_bytes, sbc_cuda_stream_t stream,
                  const sbc_cuda_event_t *marks);

/*
 * Host-buffer form of sbc_encode for callers whose update lives in host
 * memory: copies update_host to update_dev, encodes, copies the finished
 * container (its true length, *out_bytes_host) and mu back, and synchronises
 * `stream`.  The residual is the encoder's persistent state (Algorithm 1) and
 * stays on the device.  update_dev: device scratch of numel floats;
 * stream_dev: device scratch of out_capacity bytes.  Pinned host memory makes
 * the copies asynchronous up to the final synchronise.  With page-locked
 * out_stream_host the container is written to the host by a kernel instead of
 * a copy engine (so that it does not queue behind another stream's large
 * transfer in the same direction); sbc_decode_accumulate_host fetches
 * page-locked containers the same way.  Two such calls on two streams, from
 * two host threads, then use both directions of the link at once.  The first
 * host-buffer call of a host thread page-locks a 256-byte landing pad for the
 * header and status words it reads back (kept for the life of the thread).
 */
int sbc_encode_host(const float *update_host, float *update_dev, float *residual_dev,
                    int64_t numel, double p, void *out_stream_host, void *stream_dev,
                    size_t out_capacity, size_t *out_bytes_host, float *out_mu_host,
                    void *workspace, size_t workspace_bytes, sbc_cuda_stream_t stream);

/*
 * sbc_encode without a workspace argument, for callers that must not allocate.
 * (The paper has no counterpart; this is a packaging variant of sbc_encode.)
 *
 * Who needs it: code that is handed a stream and its tensors but no allocator
 * -- a compression hook called from inside a training framework's
 * communication step, a plug-in in a serving process, a control loop that is
 * forbidden to allocate once it is running.  For them cudaMalloc is either
 * unavailable or harmful (it can synchronise the whole device and stall
 * streams that belong to someone else), and they have no pool to carve the
 * scratch of sbc_encode from.
 *
 * The scratch of this variant is a fixed array of SBC_STATIC_WORKSPACE_BYTES
 * that is part of the library image: every GPU that loads the library holds
 * those bytes until the process exits.  Consequences the caller must know:
 *   - Only problems with sbc_workspace_bytes(numel, p) <=
 *     SBC_STATIC_WORKSPACE_BYTES fit (up to about 2.6 M elements at p = 0.01,
 *     10.7 M at p = 0.001);
 *     larger ones are refused with SBC_ECAPACITY and nothing is enqueued.
 *   - There is ONE array per GPU, shared by every call in the process.  Two
 *     calls whose device work can overlap (different streams, different
 *     threads) race on it and corrupt each other; issue them on one stream or
 *     order them with events.  The array keeps whatever the previous call
 *     left; each call clears the parts that must start at zero itself.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and remembers it; make that first call outside any
 *     stream capture.  The remembered address belongs to the device's primary
 *     context: after cudaDeviceReset it is stale, and the library must not be
 *     used on that device again in the same process.  No call allocates or
 *     frees memory.
 * Everything else (arguments, results, errors, asynchrony) is as sbc_encode.
 */
#define SBC_STATIC_WORKSPACE_BYTES (8u << 20)
int sbc_encode_static(const float *update, float *residual, int64_t numel, double p,
                      void *out_stream, size_t out_capacity, float *out_mu,
                      sbc_cuda_stream_t stream);

/* Copies the header of a device-resident stream to the host and fills
 * *host_out.  Synchronises `stream`.  Returns SBC_OK, SBC_ECORRUPT if the
 * magic/version are wrong, SBC_ENONFINITE or SBC_ETIMEOUT if the status word
 * says so. */
int sbc_stream_info_get(const void *stream_dev, sbc_stream_info *host_out,
                        sbc_cuda_stream_t stream);

/* ---- server side ------------------------------------------------------- */

/*
 * Decode n_clients streams and add them into a dense tensor (Algorithm 4 for
 * each stream; Algorithm 1, server line "dW <- 1/|I_t| sum dW_i*", without
 * the 1/|I_t| factor, which is the caller's):
 *
 *   out_dense[j] += mu_c   for every client c and every position j it sent.
 *
 * streams    HOST array of n_clients DEVICE pointers to containers written
 *            by sbc_encode for the same numel (16-byte aligned)
 * n_clients  >= 0
 * out_dense  device, numel floats, in/out (zero it first for a plain sum)
 * numel      must equal the numel in every header
 * status_dev device, one uint32 the kernels OR error bits into (may be NULL;
 *            the caller zeroes it).  A stream whose header fails validation
 *            contributes nothing; a chunk whose codewords run out of the
 *            payload or past numel stops there; a chunk that does not end
 *            where the table says the next one starts is reported after its
 *            (in-range) positions were added.  When the word is non-zero
 *            out_dense is not to be trusted.
 * Asynchronous.  The order of the fp32 additions into one element is not
 * fixed, so sums over several clients agree with a sequential sum to
 * rounding (<= n_clients ulps of the partial sums), not bit for bit.
 */
int sbc_decode_accumulate(const void *const *streams, int n_clients,
                          float *out_dense, int64_t numel, uint32_t *status_dev,
                          sbc_cuda_stream_t stream);

/*
 * sbc_decode_accumulate for messages the caller does not vouch for (received
 * from another process or machine): Algorithm 4 reads "while i < size(msg)",
 * and this form is told size(msg).
 *
 * stream_bytes  HOST array of n_clients sizes: stream_bytes[c] bytes are
 *               readable behind streams[c] (the received length, or the
 *               capacity of the slot the message sits in); each >= 64.
 * A header whose size fields (k, n_chunks, payload_offset, nbits) describe a
 * container longer than stream_bytes[c] fails validation BEFORE any chunk-table
 * entry or payload word is read: the stream contributes nothing and
 * SBC_STATUS_CORRUPT is set.  sbc_decode_accumulate itself checks the size
 * fields only against each other and against numel, i.e. it trusts that the
 * buffer is as long as its header says -- true for a container sbc_encode
 * wrote into a buffer of sbc_stream_bytes(numel, p) bytes.
 * Everything else as sbc_decode_accumulate.
 */
int sbc_decode_accumulate_sized(const void *const *streams, const size_t *stream_bytes,
                                int n_clients, float *out_dense, int64_t numel,
                                uint32_t *status_dev, sbc_cuda_stream_t stream);

/*
 * Decode, scale and apply in one pass (Algorithm 1: server lines
 * "dW <- 1/|I_t| sum dW_i*" and "W <- W + dW", equally the client line
 * "W_i <- W_i + dW"; momentum masking, Supplement "Momentum Correction, Warm-up
 * Training and Momentum Masking": the momentum of every updated weight is set
 * to zero):
 *
 *   weights[j]  += scale * mu_c   for every client c and every position j it sent
 *   momentum[j]  = 0              at those positions (if momentum != NULL)
 *
 * scale is 1/|I_t| for the paper's average, 1 for a plain sum.  Each client's
 * contribution fl32(scale * mu_c) is added with an fp32 atomic, so the result
 * agrees with "sum, then scale, then add" to rounding (a few ulps of
 * |weights[j]| + scale * sum_c |mu_c|), not bit for bit.  Other arguments,
 * validation and status reporting as sbc_decode_accumulate, which is this call
 * with scale = 1 and momentum = NULL.
 */
int sbc_decode_apply(const void *const *streams, int n_clients, float scale, float *weights,
                     float *momentum, int64_t numel, uint32_t *status_dev,
                     sbc_cuda_stream_t stream);
/* sbc_decode_apply with the readable size of every message stated, as
 * sbc_decode_accumulate_sized. */
int sbc_decode_apply_sized(const void *const *streams, const size_t *stream_bytes, int n_clients,
                           float scale, float *weights, float *momentum, int64_t numel,
                           uint32_t *status_dev, sbc_cuda_stream_t stream);

/*
 * sbc_decode_accumulate for many tensors at once: for every tensor t,
 * out_dense[t][j] += mu_{c,t} over the n_clients streams of that tensor
 * (Algorithm 1, server sum line, per tensor).  One launch for the batch.
 *
 * descs      HOST array of n_tensors descriptors; descs[t].streams is a HOST
 *            array of n_clients DEVICE pointers.  Read before the call returns.
 * n_clients  1 .. 32 (the same for every tensor)
 * workspace  device, 256-byte aligned, >= sbc_decode_workspace_bytes_batch(n_tensors)
 * status_dev as in sbc_decode_accumulate (one word for the whole batch)
 */
typedef struct sbc_decode_desc {
    const void *const *streams;
    float *out_dense;
    int64_t numel;
    const size_t *stream_bytes; /* HOST array of n_clients readable sizes as in
                                   sbc_decode_accumulate_sized, or NULL (not stated) */
} sbc_decode_desc;
size_t sbc_decode_workspace_bytes_batch(int n_tensors);
int sbc_decode_accumulate_batch(int n_tensors, int n_clients, const sbc_decode_desc *descs,
                                uint32_t *status_dev, void *workspace, size_t workspace_bytes,
                                sbc_cuda_stream_t stream);

/*
 * Host-buffer form of sbc_decode_accumulate: copies the n_clients containers
 * (streams_host[c], stream_bytes[c] bytes each) into staging_dev (device
 * scratch of staging_bytes >= sum of the sizes rounded up to 16 each), zeroes
 * dense_dev (device, numel floats), decodes and sums into it, copies the
 * result to out_dense_host and the status word to *status_host, and
 * synchronises `stream`.  Returns SBC_ECORRUPT if the status word is non-zero.
 * The headers are first checked on the host against stream_bytes[c] (magic,
 * version, numel, and that the container they describe ends inside the bytes
 * given): if one fails, SBC_ECORRUPT is returned, *status_host gets
 * SBC_STATUS_CORRUPT, nothing is enqueued and out_dense_host is not touched.
 * The device decode is the _sized form with the same lengths.
 */
int sbc_decode_accumulate_host(const void *const *streams_host, const size_t *stream_bytes,
                               int n_clients, float *out_dense_host, float *dense_dev,
                               int64_t numel, void *staging_dev, size_t staging_bytes,
                               uint32_t *status_host, sbc_cuda_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* SBC_H */
