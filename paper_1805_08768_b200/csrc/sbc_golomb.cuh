// Golomb position coding (Algorithm 3) and decoding (Algorithm 4).
//
// Encode: kept-position bitmask -> ascending position list (popcount scan)
// -> per-codeword lengths q + 1 + b -> exclusive scan = bit offsets ->
// every codeword ORs its own bits into the pre-zeroed payload.
// Decode: one thread per chunk of kChunkCodewords codewords, started from the
// chunk table (bit offset, previous position), adds mu into the dense tensor.
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// ---------------------------------------------------------------- mask -> sorted positions

// In-place exclusive scan of the kept-position counts per mask tile (one block).
__global__ void __launch_bounds__(kBlock) k_mask_scan(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status) return;
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    constexpr int kPer = 8;
    uint32_t carry = 0u;
    for (uint32_t base = 0; base < P.n_mask_tiles; base += kBlock * kPer) {
        uint32_t v[kPer];
        uint32_t sum = 0u;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t t = base + threadIdx.x * kPer + j;
            v[j] = (t < P.n_mask_tiles) ? P.mask_tile_cnt[t] : 0u;
            sum += v[j];
        }
        uint32_t total;
        uint32_t run = carry + block_exclusive_scan<uint32_t>(sum, s_scan, &total);
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t t = base + threadIdx.x * kPer + j;
            if (t < P.n_mask_tiles) P.mask_tile_cnt[t] = run;
            run += v[j];
        }
        carry += total;
    }
    if (threadIdx.x == 0) {
        ctl->kept_total = carry;
        if (carry != (uint32_t)P.k) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
}

// Mask -> ascending position list.
__global__ void __launch_bounds__(kBlock) k_mask_compact(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    if (P.ctl->status) return;
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    static_assert(kMaskTileWords / kBlock == 8, "eight words per thread");
    constexpr int kPer = kMaskTileWords / kBlock;
    for (uint32_t tile = S.bx; tile < P.n_mask_tiles; tile += S.nb) {
        uint32_t words[kPer];
        uint32_t c = 0u;
        const uint32_t w0 = tile * kMaskTileWords + threadIdx.x * kPer;
        if (w0 + kPer <= P.n_mask_words) {
            const uint4 lo = *reinterpret_cast<const uint4*>(P.mask + w0);
            const uint4 hi = *reinterpret_cast<const uint4*>(P.mask + w0 + 4);
            words[0] = lo.x; words[1] = lo.y; words[2] = lo.z; words[3] = lo.w;
            words[4] = hi.x; words[5] = hi.y; words[6] = hi.z; words[7] = hi.w;
        } else {
#pragma unroll
            for (int j = 0; j < kPer; ++j) words[j] = (w0 + j < P.n_mask_words) ? P.mask[w0 + j] : 0u;
        }
#pragma unroll
        for (int j = 0; j < kPer; ++j) c += __popc(words[j]);
        uint32_t pos = P.mask_tile_cnt[tile] + block_exclusive_scan<uint32_t>(c, s_scan, nullptr);
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            uint32_t w = words[j];
            const uint32_t first = (w0 + j) << 5;
            while (w) {
                const uint32_t idx = first + (__ffs(w) - 1);
                w &= w - 1u;
                if (pos < (uint32_t)P.k) P.idx[pos] = idx;
                ++pos;
            }
        }
    }
}

// ---------------------------------------------------------------- lengths, offsets, header

__device__ __forceinline__ unsigned long long codeword_len(const Prob& P, uint32_t i, uint32_t* gap) {
    const long long prev = i ? (long long)P.idx[i - 1] : -1ll;
    const uint32_t g = (uint32_t)((long long)P.idx[i] - prev - 1);  // gap - 1 of Algorithm 3
    *gap = g;
    return (unsigned long long)(g >> P.b) + 1ull + (unsigned long long)P.b;
}

// Bits of each block of kLenBlock codewords, and -- since this is the first
// walk over the ordered position list -- the residual write-back
// R_j = A_j - mu at the kept positions (Algorithm 1), in address order.
__global__ void __launch_bounds__(kBlock) k_len_sum_residual(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    if (P.ctl->status) return;
    __shared__ unsigned long long s_scan[kBlock / 32 + 1];
    constexpr int kPer = kLenBlock / kBlock;
    const float mu = P.ctl->mu32;
    const uint32_t k = (uint32_t)P.k;
    for (uint32_t blk = S.bx; blk < P.n_len_blocks; blk += S.nb) {
        const uint32_t i0 = blk * kLenBlock + threadIdx.x * kPer;
        uint32_t pos[kPer];
        float r[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) pos[j] = (i0 + j < k) ? P.idx[i0 + j] : 0u;
#pragma unroll
        for (int j = 0; j < kPer; ++j) r[j] = (i0 + j < k) ? P.residual[pos[j]] : 0.f;
        long long prev = (i0 && i0 < k) ? (long long)P.idx[i0 - 1] : -1ll;
        unsigned long long sum = 0ull;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            if (i0 + j < k) {
                P.residual[pos[j]] = __fsub_rn(r[j], mu);
                const uint32_t g = (uint32_t)((long long)pos[j] - prev - 1);
                sum += (unsigned long long)(g >> P.b) + 1ull + (unsigned long long)P.b;
                prev = pos[j];
            }
        }
        unsigned long long total;
        block_exclusive_scan<unsigned long long>(sum, s_scan, &total);
        if (threadIdx.x == 0) P.blk_len[blk] = total;
    }
}

__device__ __forceinline__ void store_u32(uint8_t* p, uint32_t v) { *reinterpret_cast<uint32_t*>(p) = v; }
__device__ __forceinline__ void store_u64(uint8_t* p, unsigned long long v) {
    *reinterpret_cast<unsigned long long*>(p) = v;
}

// Scan of the per-block bit counts; also writes the container header, always,
// so that a failed encode still leaves a header that says why.
__global__ void __launch_bounds__(kBlock) k_len_scan_header(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    __shared__ unsigned long long s_scan[kBlock / 32 + 1];
    const bool ok = ctl->status == 0u;  // uniform: nothing writes status while this kernel runs
    unsigned long long total = 0ull;
    if (ok) {
        constexpr int kPer = 8;
        for (uint32_t base = 0; base < P.n_len_blocks; base += kBlock * kPer) {
            unsigned long long v[kPer];
            unsigned long long sum = 0ull;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t t = base + threadIdx.x * kPer + j;
                v[j] = (t < P.n_len_blocks) ? P.blk_len[t] : 0ull;
                sum += v[j];
            }
            unsigned long long part;
            unsigned long long run = total + block_exclusive_scan<unsigned long long>(sum, s_scan, &part);
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t t = base + threadIdx.x * kPer + j;
                if (t < P.n_len_blocks) P.blk_len[t] = run;
                run += v[j];
            }
            total += part;
        }
    }
    if (threadIdx.x == 0) {
        ctl->nbits = total;
        uint8_t* h = P.stream;
        store_u32(h + 0, SBC_MAGIC);
        store_u32(h + 4, SBC_VERSION);
        store_u64(h + 8, (unsigned long long)P.n);
        store_u64(h + 16, ok ? (unsigned long long)P.k : 0ull);
        store_u64(h + 24, total);
        store_u64(h + 32, ok ? P.payload_offset : (unsigned long long)SBC_HEADER_BYTES);
        store_u32(h + 40, (uint32_t)P.b);
        store_u32(h + 44, ok ? ctl->side : 0u);
        store_u32(h + 48, ok ? __float_as_uint(ctl->mu32) : 0u);
        store_u32(h + 52, SBC_CHUNK_CODEWORDS);
        store_u32(h + 56, ok ? P.n_chunks : 0u);
        store_u32(h + 60, ctl->status);
    }
}

// ---------------------------------------------------------------- bit packer

// OR `count` (1..32) bits, given right-aligned in `value`, into the payload at
// stream bit `off`.  Stream bit j lives in byte j/8 at bit 7-(j%8); a 32-bit
// word assembled MSB-first is therefore stored byte-swapped.
__device__ __forceinline__ void or_bits(uint32_t* words, unsigned long long off, int count,
                                        uint32_t value) {
    const unsigned long long w = off >> 5;
    const int sh = (int)(off & 31ull);
    const unsigned long long window = (unsigned long long)value << (64 - count - sh);
    const uint32_t hi = (uint32_t)(window >> 32), lo = (uint32_t)window;
    if (hi) atomicOr(words + w, __byte_perm(hi, 0u, 0x0123));
    if (lo) atomicOr(words + w + 1, __byte_perm(lo, 0u, 0x0123));
}

__global__ void __launch_bounds__(kBlock) k_pack(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    if (P.ctl->status) return;
    __shared__ unsigned long long s_scan[kBlock / 32 + 1];
    constexpr int kPer = kLenBlock / kBlock;
    uint32_t* words = reinterpret_cast<uint32_t*>(P.stream + P.payload_offset);
    uint8_t* table = P.stream + SBC_HEADER_BYTES;
    const int b = P.b;
    for (uint32_t blk = S.bx; blk < P.n_len_blocks; blk += S.nb) {
        unsigned long long len[kPer];
        uint32_t gap[kPer];
        unsigned long long sum = 0ull;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t i = blk * kLenBlock + threadIdx.x * kPer + j;
            len[j] = 0ull;
            gap[j] = 0u;
            if (i < (uint32_t)P.k) len[j] = codeword_len(P, i, &gap[j]);
            sum += len[j];
        }
        unsigned long long off = P.blk_len[blk] + block_exclusive_scan<unsigned long long>(sum, s_scan, nullptr);
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t i = blk * kLenBlock + threadIdx.x * kPer + j;
            if (i >= (uint32_t)P.k) continue;
            if (i % kChunkCodewords == 0) {
                uint8_t* e = table + (size_t)(i / kChunkCodewords) * SBC_CHUNK_ENTRY_BYTES;
                store_u64(e, off);
                store_u64(e + 8, (unsigned long long)(i ? (long long)P.idx[i - 1] : -1ll));
            }
            unsigned long long pos = off;
            uint32_t q = gap[j] >> b;
            // q ones: head up to a word boundary, whole words, then the rest
            if (q) {
                const int head = min((uint32_t)(32 - (int)(pos & 31ull)) & 31u, q);
                if (head) { or_bits(words, pos, head, 0xffffffffu >> (32 - head)); pos += head; q -= head; }
                while (q >= 32u) { words[pos >> 5] = 0xffffffffu; pos += 32; q -= 32u; }
                if (q) { or_bits(words, pos, (int)q, 0xffffffffu >> (32 - q)); pos += q; }
            }
            // the terminating zero and r in b bits, MSB first: 1 + b <= 31 bits
            or_bits(words, pos, 1 + b, gap[j] & ((1u << b) - 1u));
            off += len[j];
        }
    }
}

}  // namespace sbc
