// Golomb position decoding and server-side sum (Algorithm 4; Algorithm 1,
// server line "dW <- sum of the decoded client updates").
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

constexpr int kMaxClientsPerLaunch = 32;

struct DecodeArgs {
    const uint8_t* streams[kMaxClientsPerLaunch];
    int n_clients;
    float* out;
    long long n;
    uint32_t* status;  // may be null
};

__device__ __forceinline__ uint32_t load_u32(const uint8_t* p) { return *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ unsigned long long load_u64(const uint8_t* p) {
    return *reinterpret_cast<const unsigned long long*>(p);
}

struct StreamView {
    const uint32_t* words;        // payload as stored (byte-swapped MSB-first words)
    const uint8_t* table;
    unsigned long long k, nbits, n_words;
    uint32_t b, n_chunks;
    float mu;
};

// 32 stream bits starting at bit `pos`, MSB first; bits past the payload read as 0.
__device__ __forceinline__ uint32_t peek32(const StreamView& v, unsigned long long pos) {
    const unsigned long long w = pos >> 5;
    const int sh = (int)(pos & 31ull);
    const uint32_t hi = (w < v.n_words) ? __byte_perm(__ldg(v.words + w), 0u, 0x0123) : 0u;
    const uint32_t lo = (w + 1 < v.n_words) ? __byte_perm(__ldg(v.words + w + 1), 0u, 0x0123) : 0u;
    return __funnelshift_l(lo, hi, sh);
}

__global__ void __launch_bounds__(128) k_decode_accumulate(const DecodeArgs args) {
    __shared__ StreamView s_view[kMaxClientsPerLaunch];
    __shared__ uint32_t s_first[kMaxClientsPerLaunch + 1];  // first work item of each client
    const int tid = threadIdx.x;
    if (tid < args.n_clients) {
        const uint8_t* h = args.streams[tid];
        StreamView v;
        v.k = load_u64(h + 16);
        v.nbits = load_u64(h + 24);
        const unsigned long long payload_offset = load_u64(h + 32);
        v.b = load_u32(h + 40);
        v.mu = __uint_as_float(load_u32(h + 48));
        v.n_chunks = load_u32(h + 56);
        v.n_words = (v.nbits + 31ull) >> 5;
        v.words = reinterpret_cast<const uint32_t*>(h + payload_offset);
        v.table = h + SBC_HEADER_BYTES;
        const bool good =
            load_u32(h + 0) == SBC_MAGIC && load_u32(h + 4) == SBC_VERSION &&
            load_u64(h + 8) == (unsigned long long)args.n && load_u32(h + 60) == 0u &&
            load_u32(h + 52) == SBC_CHUNK_CODEWORDS && v.b <= 30u && v.k <= (unsigned long long)args.n &&
            v.n_chunks == (uint32_t)((v.k + kChunkCodewords - 1) / kChunkCodewords) &&
            payload_offset == SBC_HEADER_BYTES + (unsigned long long)v.n_chunks * SBC_CHUNK_ENTRY_BYTES &&
            v.nbits >= v.k * (1ull + v.b) &&
            v.nbits <= v.k * (1ull + v.b) + ((unsigned long long)args.n >> v.b);
        if (!good) {
            v.n_chunks = 0u;  // contributes nothing
            if (args.status && blockIdx.x == 0) atomicOr(args.status, SBC_STATUS_CORRUPT);
        }
        s_view[tid] = v;
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0u;
        for (int c = 0; c < args.n_clients; ++c) { s_first[c] = run; run += s_view[c].n_chunks; }
        s_first[args.n_clients] = run;
    }
    __syncthreads();
    const uint32_t total = s_first[args.n_clients];
    for (uint32_t item = blockIdx.x * blockDim.x + tid; item < total; item += gridDim.x * blockDim.x) {
        int c = 0;
        while (item >= s_first[c + 1]) ++c;
        const StreamView& v = s_view[c];
        const uint32_t chunk = item - s_first[c];
        const uint8_t* e = v.table + (size_t)chunk * SBC_CHUNK_ENTRY_BYTES;
        unsigned long long pos = load_u64(e);
        long long prev = (long long)load_u64(e + 8);
        const unsigned long long first_cw = (unsigned long long)chunk * kChunkCodewords;
        const uint32_t count = (uint32_t)min((unsigned long long)kChunkCodewords, v.k - first_cw);
        uint32_t err = 0u;
        if (pos >= v.nbits || prev < -1 || prev >= args.n) err = SBC_STATUS_CORRUPT;
        for (uint32_t i = 0; i < count && !err; ++i) {
            // unary part: count ones up to the first zero
            unsigned long long q = 0ull;
            while (true) {
                const uint32_t ones = __clz(~peek32(v, pos));  // 32 when the window is all ones
                q += ones;
                pos += ones;
                if (ones < 32u) break;
                if (pos >= v.nbits) { err = SBC_STATUS_CORRUPT; break; }
            }
            if (err) break;
            pos += 1ull;  // the zero
            const uint32_t r = v.b ? (peek32(v, pos) >> (32 - v.b)) : 0u;
            pos += v.b;
            if (pos > v.nbits) { err = SBC_STATUS_CORRUPT; break; }
            const unsigned long long step = (q << v.b) + r + 1ull;
            if (q > (unsigned long long)args.n || (unsigned long long)(args.n - 1 - prev) < step) {
                err = SBC_STATUS_RANGE;
                break;
            }
            prev += (long long)step;
            atomicAdd(args.out + prev, v.mu);
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
        if (err && args.status) atomicOr(args.status, err);
    }
}

}  // namespace sbc
