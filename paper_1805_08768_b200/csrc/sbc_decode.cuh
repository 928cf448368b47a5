// Golomb position decoding and server-side sum (Algorithm 4; Algorithm 1,
// server lines "dW <- 1/|I_t| sum of the decoded client updates", "W <- W + dW";
// momentum masking of the Supplement as an optional second target).
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

constexpr int kMaxClientsPerLaunch = 32;

struct DecodeArgs {
    const uint8_t* streams[kMaxClientsPerLaunch];
    // bytes the caller vouches for behind streams[c]; 0: not stated (the header's own size fields are trusted)
    unsigned long long bytes[kMaxClientsPerLaunch];
    int n_clients;
    float* out;
    long long n;
    uint32_t* status;  // may be null
    float scale;       // every transmitted value is multiplied by this before it is added
    float* momentum;   // may be null: zeroed at every decoded position (momentum masking)
};

__device__ __forceinline__ uint32_t load_u32(const uint8_t* p) { return *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ unsigned long long load_u64(const uint8_t* p) {
    return *reinterpret_cast<const unsigned long long*>(p);
}

struct StreamView {
    const uint32_t* words;        // payload as stored (byte-swapped MSB-first words)
    const uint8_t* table;
    unsigned long long k, nbits, n_words;
    uint32_t b, n_chunks, chunk_cw;
    float mu;
    const float* values;  // one value per position (values stream), else null
};

// 32 stream bits starting at bit `pos`, MSB first; bits past the payload read as 0.
__device__ __forceinline__ uint32_t peek32(const StreamView& v, unsigned long long pos) {
    const unsigned long long w = pos >> 5;
    const int sh = (int)(pos & 31ull);
    const uint32_t hi = (w < v.n_words) ? __byte_perm(__ldg(v.words + w), 0u, 0x0123) : 0u;
    const uint32_t lo = (w + 1 < v.n_words) ? __byte_perm(__ldg(v.words + w + 1), 0u, 0x0123) : 0u;
    return __funnelshift_l(lo, hi, sh);
}

// out[j] += mu.  The hardware fp32 atomic add treats subnormal inputs and results as zero, which
// is harmless (far below the stated tolerance) unless the transmitted value itself is tiny; then
// an IEEE add is done with a compare-and-swap retry instead.  The retry count is bounded: every
// failed attempt means another thread's add succeeded.
__device__ __forceinline__ uint32_t add_at(float* p, float mu, bool ieee_path) {
    if (!ieee_path) { atomicAdd(p, mu); return 0u; }
    unsigned int* u = reinterpret_cast<unsigned int*>(p);
    unsigned int old = *u;
    for (int tries = 0; tries < (1 << 20); ++tries) {
        const unsigned int assumed = old;
        old = atomicCAS(u, assumed, __float_as_uint(__fadd_rn(__uint_as_float(assumed), mu)));
        if (old == assumed) return 0u;
    }
    return SBC_STATUS_INTERNAL;
}

constexpr int kDecodeThreads = 64;            // two warps per block
constexpr int kDecodeWarpWords = 4608;        // staged payload words per warp (18 KB)
constexpr unsigned long long kInOrderPositions = 1ull << 21;   // streams from this many positions on add in list order

// Sequential MSB-first bit reader over a warp's staged (byte-swapped) words, or over global memory when the group's payload did not fit the stage.
// `cur` holds the next 64 - (32 - avail) ... bits left-aligned: bits [63, 64-avail)
// are valid; one word is always fetched ahead so that its latency is hidden.
struct BitReader {
    const uint32_t* sw;
    const StreamView* v;
    unsigned long long first_word;  // stream word index of sw[0]
    uint32_t n_staged;
    bool staged;
    unsigned long long cur;   // unread bits, left-aligned
    int avail;                // valid bits in cur (>= 32 after every refill)
    unsigned long long next_index;  // stream word index of `ahead`
    uint32_t ahead;           // word already fetched, not yet in cur

    __device__ __forceinline__ uint32_t fetch(unsigned long long w) const {
        if (staged) {
            const unsigned long long r = w - first_word;
            return (r < n_staged) ? sw[r] : 0u;
        }
        return (w < v->n_words) ? __byte_perm(__ldg(v->words + w), 0u, 0x0123) : 0u;
    }
    __device__ __forceinline__ void start(unsigned long long pos) {
        const unsigned long long w = pos >> 5;
        const int sh = (int)(pos & 31ull);
        cur = (((unsigned long long)fetch(w) << 32) | (unsigned long long)fetch(w + 1)) << sh;
        avail = 64 - sh;
        next_index = w + 2;
        ahead = fetch(next_index);
    }
    __device__ __forceinline__ uint32_t top32() const { return (uint32_t)(cur >> 32); }
    __device__ __forceinline__ void skip(int count) {  // count <= 32 <= avail
        cur <<= count;
        avail -= count;
        if (avail <= 32) {
            cur |= (unsigned long long)ahead << (32 - avail);
            avail += 32;
            ++next_index;
            ahead = fetch(next_index);
        }
    }
};

// One codeword from the warp's staged (MSB-first) words at relative bit `rel`: q ones, a zero,
// b remainder bits (Algorithm 4).  Bit positions relative to the stage fit 32 bits and the
// codeword is cut out of a 64-bit window rebuilt from three staged words.  The common case (fewer
// than 32 ones, everything in range) is decided by ONE predicate and runs without any other branch;
// long unary runs and every kind of error take the general step.  On success returns 0, advances
// `rel`, sets *at to the decoded position and `nxt` to the position after it; else an error status.
__device__ __forceinline__ uint32_t parse_staged(const uint32_t* sw, uint32_t& rel, uint32_t rel_end, uint32_t b,
                                                 uint32_t n32, uint32_t& nxt, uint32_t* at) {
    uint32_t w = rel >> 5;
    const int sh = (int)(rel & 31u);
    const uint32_t x0 = sw[w], x1 = sw[w + 1], x2 = sw[w + 2];
    uint32_t hi = __funnelshift_l(x1, x0, sh);
    uint32_t lo = __funnelshift_l(x2, x1, sh);
    uint32_t ones = __clz(~hi);
    const uint32_t q_max = n32 >> b;  // a larger quotient cannot stay inside the tensor
    {
        const unsigned long long win = ((unsigned long long)hi << 32) | (unsigned long long)lo;
        const uint32_t r = (uint32_t)(((win << (ones & 31u) << 1) >> 1) >> (63u - b));  // b bits after the zero
        const uint32_t stp = (ones << b) + r;       // meaningful when ones <= q_max: no overflow then
        const bool ok = (rel < rel_end) & (ones < 32u) & (ones <= q_max) & (stp < n32 - nxt);
        if (ok) {
            *at = nxt + stp;
            nxt = *at + 1u;
            rel += ones + 1u + b;
            return 0u;
        }
    }
    // general step: a run of 32 or more ones, or something is wrong
    if (rel >= rel_end) return SBC_STATUS_CORRUPT;
    unsigned long long q = ones;
    while (ones == 32u) {
        rel += 32u;
        if (rel >= rel_end) break;
        w = rel >> 5;
        hi = __funnelshift_l(sw[w + 1], sw[w], sh);
        lo = __funnelshift_l(sw[w + 2], sw[w + 1], sh);
        ones = __clz(~hi);
        q += ones;
    }
    if (rel >= rel_end) return SBC_STATUS_CORRUPT;
    const unsigned long long win = ((unsigned long long)hi << 32) | (unsigned long long)lo;
    const uint32_t r = b ? (uint32_t)((win << (ones + 1u)) >> (64u - b)) : 0u;
    rel += ones + 1u + b;
    const unsigned long long step = (q << b) + r;
    if (q > (unsigned long long)n32 || (unsigned long long)(n32 - nxt) <= step) return SBC_STATUS_RANGE;
    *at = nxt + (uint32_t)step;
    nxt = *at + 1u;
    return 0u;
}

// One warp per group of 32 consecutive chunks: the group's payload is one
// contiguous bit range, copied once (coalesced) into shared memory; then every
// lane parses its chunk's codewords (32, 64 or 256 of them, by the header) from there (Algorithm 4)
// and adds mu at each position (Algorithm 1, server sum).
__device__ __forceinline__ void decode_body(const DecodeArgs& args) {
    __shared__ StreamView s_view[kMaxClientsPerLaunch];
    __shared__ uint32_t s_first[kMaxClientsPerLaunch + 1];  // first work item (group) of each client
    __shared__ uint32_t s_words[kDecodeThreads / 32][kDecodeWarpWords];
    __shared__ uint32_t s_at[kDecodeThreads / 32][32][33];  // decoded positions of a step, [chunk lane][codeword], padded
    __shared__ uint32_t s_n[kDecodeThreads / 32][32];       // how many each lane decoded in the step
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < args.n_clients) {
        const uint8_t* h = args.streams[tid];
        StreamView v;
        v.k = load_u64(h + 16);
        v.nbits = load_u64(h + 24);
        const unsigned long long payload_offset = load_u64(h + 32);
        v.b = load_u32(h + 40);
        v.mu = __uint_as_float(load_u32(h + 48));
        v.n_chunks = load_u32(h + 56);
        v.chunk_cw = load_u32(h + 52);
        v.n_words = (v.nbits + 31ull) >> 5;
        v.words = reinterpret_cast<const uint32_t*>(h + payload_offset);
        v.table = h + SBC_HEADER_BYTES;
        const uint32_t side = load_u32(h + 44);
        const unsigned long long values_bytes = (side == SBC_SIDE_VALUES) ? ((v.k * 4ull + 15ull) & ~15ull) : 0ull;
        v.values = (side == SBC_SIDE_VALUES)
            ? reinterpret_cast<const float*>(h + SBC_HEADER_BYTES + (unsigned long long)v.n_chunks * SBC_CHUNK_ENTRY_BYTES)
            : nullptr;
        const bool good =
            load_u32(h + 0) == SBC_MAGIC && load_u32(h + 4) == SBC_VERSION &&
            load_u64(h + 8) == (unsigned long long)args.n && load_u32(h + 60) == 0u &&
            v.chunk_cw == chunk_codewords_for(v.k) && v.b <= 30u && v.k <= (unsigned long long)args.n &&
            (unsigned long long)v.n_chunks == (v.k + v.chunk_cw - 1ull) / v.chunk_cw &&
            side <= SBC_SIDE_VALUES &&
            payload_offset == SBC_HEADER_BYTES + (unsigned long long)v.n_chunks * SBC_CHUNK_ENTRY_BYTES + values_bytes &&
            v.nbits >= v.k * (1ull + v.b) &&
            v.nbits <= v.k * (1ull + v.b) + ((unsigned long long)args.n >> v.b) &&
            // the whole container (chunk table, values, payload padded to 16 bytes) lies inside the bytes the
            // caller stated: checked before any table entry or payload word is read (k <= n < 2^31 and
            // nbits < 2^37 by the lines above, so nothing here overflows)
            (args.bytes[tid] == 0ull ||
             payload_offset + ((((v.nbits + 7ull) >> 3) + 15ull) & ~15ull) <= args.bytes[tid]);
        if (!good) {
            v.n_chunks = 0u;  // contributes nothing
            v.chunk_cw = (uint32_t)kChunkCodewords;
            if (args.status && blockIdx.x == 0) atomicOr(args.status, SBC_STATUS_CORRUPT);
        }
        s_view[tid] = v;
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0u;
        for (int c = 0; c < args.n_clients; ++c) { s_first[c] = run; run += (s_view[c].n_chunks + 31u) / 32u; }
        s_first[args.n_clients] = run;
    }
    __syncthreads();
    const uint32_t total = s_first[args.n_clients];
    const uint32_t warps_total = gridDim.x * (kDecodeThreads / 32);
    uint32_t* sw = s_words[warp];
    for (uint32_t item = blockIdx.x * (kDecodeThreads / 32) + warp; item < total; item += warps_total) {
        int c = 0;
        while (item >= s_first[c + 1]) ++c;
        const StreamView& v = s_view[c];
        const uint32_t chunk0 = (item - s_first[c]) * 32u;
        const uint32_t chunk = chunk0 + lane;
        const bool has = chunk < v.n_chunks;
        const uint8_t* e = v.table + (size_t)(has ? chunk : chunk0) * SBC_CHUNK_ENTRY_BYTES;
        unsigned long long pos = load_u64(e);
        long long prev = (long long)load_u64(e + 8);
        // bit range of the whole group: from its first chunk to the next group's first chunk
        const unsigned long long gbeg = __shfl_sync(0xffffffffu, pos, 0);
        const uint32_t chunk_end = min(chunk0 + 32u, v.n_chunks);
        const unsigned long long gend =
            (chunk_end < v.n_chunks) ? load_u64(v.table + (size_t)chunk_end * SBC_CHUNK_ENTRY_BYTES) : v.nbits;
        uint32_t err = 0u;
        const bool range_ok = gbeg <= gend && gend <= v.nbits;  // warp-uniform
        if (!range_ok) err = SBC_STATUS_CORRUPT;
        const unsigned long long first_word = gbeg >> 5;
        const unsigned long long n_group_words = range_ok ? ((gend + 31ull) >> 5) - first_word : 0ull;
        const bool staged = range_ok && n_group_words + 2ull <= (unsigned long long)kDecodeWarpWords;
        const uint32_t n_staged = staged ? (uint32_t)n_group_words : 0u;
        __syncwarp();
        // asynchronous 4-byte copies: all of the group's words are in flight at once
        for (uint32_t i = lane; i < n_staged; i += 32) {
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(sw + i);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(v.words + first_word + i));
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        // MSB-first words for the parser, and two zero words so that a 96-bit read never leaves the stage
        for (uint32_t i = lane; i < n_staged; i += 32) sw[i] = __byte_perm(sw[i], 0u, 0x0123);
        if (staged && lane < 2) sw[n_staged + lane] = 0u;
        __syncwarp();
        // Plain sums (one value per stream, no second target, no tiny value) of long streams are
        // added in list order: every lane parses 32 codewords of its chunk into shared memory, then
        // the warp adds chunk after chunk, one instruction covering 32 neighbouring positions of the
        // tensor.  Lanes that add as they parse send each instruction to 32 places a chunk apart,
        // and DRAM serves neighbours that arrive together far better: 0.44 -> 0.40 ms for 10.7 M
        // positions over 4 GiB.  Short streams are bound by the latency of a chunk's serial parse
        // instead, which the extra step lengthens (60 -> 63 us at 1 M positions), so only streams
        // of at least kInOrderPositions positions are decoded this way.
        const float mu_w = __fmul_rn(v.mu, args.scale);
        const bool in_order = staged && v.k >= kInOrderPositions && v.values == nullptr &&
                              args.momentum == nullptr && !(fabsf(mu_w) < 7.888609052e-31f);  // warp-uniform
        if (in_order) {
            uint32_t count = 0u, rel = 0u, rel_end = 0u, nxt = 0u, done = 0u;
            const uint32_t n32 = (uint32_t)args.n;
            bool live = has && !err;
            if (live) {
                const unsigned long long first_cw = (unsigned long long)chunk * v.chunk_cw;
                count = (uint32_t)min((unsigned long long)v.chunk_cw, v.k - first_cw);
                if (pos >= v.nbits || pos < gbeg || pos > gend || prev < -1 || prev >= args.n) {
                    err = SBC_STATUS_CORRUPT;
                    live = false;
                }
                rel = (uint32_t)(pos - (first_word << 5));
                rel_end = (uint32_t)(gend - (first_word << 5));
                nxt = (uint32_t)(prev + 1);
            }
            const bool checked = live;  // the end of the chunk is compared with the table below
            for (uint32_t step = 0; step < v.chunk_cw / 32u; ++step) {
                if (!__any_sync(0xffffffffu, live && done < count)) break;  // warp-uniform
                uint32_t got = 0u;
                if (live) {
                    const uint32_t lim = min(32u, count - done);
                    for (; got < lim; ++got) {
                        uint32_t at;
                        const uint32_t bad = parse_staged(sw, rel, rel_end, v.b, n32, nxt, &at);
                        if (bad) { err = bad; live = false; break; }
                        s_at[warp][lane][got] = at;
                    }
                    done += got;
                }
                s_n[warp][lane] = got;
                __syncwarp();
#pragma unroll 4
                for (int c = 0; c < 32; ++c)
                    if ((uint32_t)lane < s_n[warp][c]) atomicAdd(args.out + s_at[warp][c][lane], mu_w);
                __syncwarp();
            }
            if (checked && !err) {
                // the chunk must end exactly where the table says the next one starts
                const unsigned long long end_pos = (first_word << 5) + rel;
                const long long end_prev = (long long)nxt - 1;
                if (chunk + 1u < v.n_chunks) {
                    if (load_u64(e + SBC_CHUNK_ENTRY_BYTES) != end_pos ||
                        (long long)load_u64(e + SBC_CHUNK_ENTRY_BYTES + 8) != end_prev)
                        err = SBC_STATUS_CORRUPT;
                } else if (end_pos != v.nbits) {
                    err = SBC_STATUS_CORRUPT;
                }
            }
        } else if (has && !err) {
            const unsigned long long first_cw = (unsigned long long)chunk * v.chunk_cw;
            const uint32_t count = (uint32_t)min((unsigned long long)v.chunk_cw, v.k - first_cw);
            const bool entry_ok = !(pos >= v.nbits || pos < gbeg || pos > gend || prev < -1 || prev >= args.n);
            if (!entry_ok) err = SBC_STATUS_CORRUPT;
            const uint32_t b = v.b;
            const float mu = __fmul_rn(v.mu, args.scale);
            float* __restrict__ momentum = args.momentum;
            const float* __restrict__ vals = v.values ? v.values + (size_t)chunk * v.chunk_cw : nullptr;
            const bool tiny = fabsf(mu) < 7.888609052e-31f;  // 2^-100
            if (!entry_ok) {
                // nothing is decoded from a chunk whose table entry is out of range
            } else if (staged) {
                uint32_t rel = (uint32_t)(pos - (first_word << 5));
                const uint32_t rel_end = (uint32_t)(gend - (first_word << 5));
                const uint32_t n32 = (uint32_t)args.n;
                uint32_t nxt = (uint32_t)(prev + 1);      // first position the next codeword can name
                float* __restrict__ out = args.out;
                const bool plain = vals == nullptr && momentum == nullptr && !tiny;  // warp-uniform
                for (uint32_t i = 0; i < count; ++i) {
                    uint32_t at;
                    const uint32_t bad = parse_staged(sw, rel, rel_end, b, n32, nxt, &at);
                    if (bad) { err = bad; break; }
                    if (plain) {  // the usual case: nothing but the add in the loop
                        atomicAdd(out + at, mu);
                        continue;
                    }
                    if (vals) {
                        const float x = __fmul_rn(vals[i], args.scale);
                        err |= add_at(args.out + at, x, fabsf(x) < 7.888609052e-31f);
                    } else {
                        err |= add_at(args.out + at, mu, tiny);
                    }
                    if (momentum) momentum[at] = 0.f;
                }
                prev = (long long)nxt - 1;
                pos = (first_word << 5) + rel;
            } else {
                // Long unary runs made the group larger than the stage: read global memory.
                BitReader br;
                br.sw = sw; br.v = &v; br.first_word = first_word; br.n_staged = 0u; br.staged = false;
                br.start(pos);
                const unsigned long long room = v.nbits - pos;  // no codeword of this chunk may reach past it
                unsigned long long used = 0ull;
                for (uint32_t i = 0; i < count; ++i) {
                    uint32_t ones = __clz(~br.top32());
                    unsigned long long q = ones;
                    while (ones == 32u) {
                        br.skip(32);
                        used += 32ull;
                        if (used > room) break;
                        ones = __clz(~br.top32());
                        q += ones;
                    }
                    if (used > room) { err = SBC_STATUS_CORRUPT; break; }
                    br.skip((int)ones + 1);  // the rest of the ones and the zero
                    const uint32_t r = b ? (br.top32() >> (32 - b)) : 0u;
                    br.skip((int)b);
                    used += ones + 1u + b;
                    const unsigned long long step = (q << b) + r + 1ull;
                    if (q > (unsigned long long)args.n || (unsigned long long)(args.n - 1 - prev) < step) {
                        err = SBC_STATUS_RANGE;
                        break;
                    }
                    prev += (long long)step;
                    if (vals) {
                        const float x = __fmul_rn(vals[i], args.scale);
                        err |= add_at(args.out + prev, x, fabsf(x) < 7.888609052e-31f);
                    } else {
                        err |= add_at(args.out + prev, mu, tiny);
                    }
                    if (momentum) momentum[prev] = 0.f;
                }
                if (!err && used > room) err = SBC_STATUS_CORRUPT;
                pos += used;
            }
            if (!err) {
                // the chunk must end exactly where the table says the next one starts
                if (chunk + 1u < v.n_chunks) {
                    if (load_u64(e + SBC_CHUNK_ENTRY_BYTES) != pos ||
                        (long long)load_u64(e + SBC_CHUNK_ENTRY_BYTES + 8) != prev)
                        err = SBC_STATUS_CORRUPT;
                } else if (pos != v.nbits) {
                    err = SBC_STATUS_CORRUPT;
                }
            }
        }
        if (err && args.status) atomicOr(args.status, err);
    }
}

__global__ void __launch_bounds__(kDecodeThreads) k_decode_accumulate(const DecodeArgs args) { decode_body(args); }

// Batch form: blockIdx.y selects the tensor; its arguments sit in device memory.
__global__ void __launch_bounds__(kDecodeThreads) k_decode_accumulate_batch(const DecodeArgs* __restrict__ all) {
    decode_body(all[blockIdx.y]);
}

}  // namespace sbc
