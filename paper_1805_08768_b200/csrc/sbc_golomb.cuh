// Golomb position coding (Algorithm 3) and decoding (Algorithm 4).
//
// Encode: kept positions bucketed by tile and ordered inside each tile -> ascending position list
// -> per-codeword lengths q + 1 + b -> exclusive scan = bit offsets ->
// every codeword ORs its own bits into the pre-zeroed payload.
// Decode: one thread per chunk of kChunkCodewords codewords, started from the
// chunk table (bit offset, previous position), adds mu into the dense tensor.
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// ---------------------------------------------------------------- block-wide sort in registers

// Compare-exchange stage of a bitonic network between registers r and r | STRIDE of one thread
// (element index = first + r); ascending where (index & size) == 0.
template <int E, int STRIDE>
__device__ __forceinline__ void bitonic_in_thread(uint32_t (&x)[E], uint32_t size, uint32_t first) {
#pragma unroll
    for (int r = 0; r < E; ++r) {
        if ((r & STRIDE) == 0 && (r | STRIDE) < E) {
            const bool ascending = ((first + (uint32_t)r) & size) == 0u;
            const uint32_t a = x[r], b = x[r | STRIDE];
            const bool swap = (a > b) == ascending;
            x[r] = swap ? b : a;
            x[r | STRIDE] = swap ? a : b;
        }
    }
}

// Ascending sort of E * kBlock values (E = 2, 4, 8 or 16), thread t holding elements E t .. E t + E - 1
// in registers (bitonic network): exchanges between threads of a warp by shuffle, between warps
// through `s_swap` (E * kBlock words, transposed so that accesses are conflict-free), the rest in
// registers.  All threads call.
template <int E>
__device__ __forceinline__ void block_sort(uint32_t (&x)[E], uint32_t* s_swap) {
    static_assert(E == 2 || E == 4 || E == 8 || E == 16, "power-of-two share per thread");
    constexpr uint32_t kCount = (uint32_t)E * kBlock;
    const uint32_t tid = threadIdx.x, first = tid * (uint32_t)E;
    for (uint32_t size = 2u; size <= kCount; size <<= 1) {
        const bool ascending = (first & size) == 0u;  // used where the partner is another thread (size >= 2 E)
        for (uint32_t stride = size >> 1; stride >= 32u * E; stride >>= 1) {  // partner in another warp
            const uint32_t d = stride / E;
#pragma unroll
            for (int r = 0; r < E; ++r) s_swap[r * kBlock + tid] = x[r];
            __syncthreads();
            const bool take_min = ((tid & d) == 0u) == ascending;
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const uint32_t o = s_swap[r * kBlock + (tid ^ d)];
                x[r] = take_min ? min(x[r], o) : max(x[r], o);
            }
            __syncthreads();
        }
        for (uint32_t stride = min(size >> 1, 16u * E); stride >= (uint32_t)E; stride >>= 1) {  // partner in this warp
            const uint32_t d = stride / E;
            const bool take_min = ((tid & d) == 0u) == ascending;
#pragma unroll
            for (int r = 0; r < E; ++r) {
                const uint32_t o = __shfl_xor_sync(0xffffffffu, x[r], (int)d);
                x[r] = take_min ? min(x[r], o) : max(x[r], o);
            }
        }
        if (E > 8 && size >= 16u) bitonic_in_thread<E, 8>(x, size, first);
        if (E > 4 && size >= 8u) bitonic_in_thread<E, 4>(x, size, first);
        if (E > 2 && size >= 4u) bitonic_in_thread<E, 2>(x, size, first);
        bitonic_in_thread<E, 1>(x, size, first);
    }
}

// ---------------------------------------------------------------- mask -> sorted positions

// Exclusive scan of the kept positions per tile (both counters of k_tile_count together) into
// the bucket starts, in place over the second counter (one block); entry n_tiles receives the total.
__global__ void __launch_bounds__(kBlock) k_tile_scan(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status) return;
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    uint32_t* __restrict__ cnt = P.tile_base;
    const uint32_t* __restrict__ cnt_in = P.tile_in;
    const uint32_t n_tiles = P.n_tiles;
    constexpr int kPer = 8;
    uint32_t carry = 0u;
    for (uint32_t base = 0; base < n_tiles; base += kBlock * kPer) {
        uint32_t v[kPer];
        uint32_t sum = 0u;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t t = base + threadIdx.x * kPer + j;
            v[j] = (t < n_tiles) ? cnt[t] + cnt_in[t] : 0u;
            sum += v[j];
        }
        uint32_t total;
        uint32_t run = carry + block_exclusive_scan<uint32_t>(sum, s_scan, &total);
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t t = base + threadIdx.x * kPer + j;
            if (t < n_tiles) cnt[t] = run;
            run += v[j];
        }
        carry += total;
    }
    if (threadIdx.x == 0) {
        cnt[n_tiles] = carry;
        ctl->kept_total = carry;
        if (carry != (uint32_t)P.k) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
}

// One bucket of up to E * kBlock positions, ordered in registers and written back.  All threads call.
template <int E>
__device__ __forceinline__ void sort_bucket_in_registers(uint32_t* list, uint32_t beg, uint32_t count, uint32_t* s_swap) {
    uint32_t x[E];
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const uint32_t i = (uint32_t)r * kBlock + threadIdx.x;  // any assignment will do before the sort
        x[r] = (i < count) ? list[beg + i] : 0xffffffffu;        // padding sorts to the end
    }
    block_sort<E>(x, s_swap);  // contains block-wide barriers: every load above precedes every store below
#pragma unroll
    for (int r = 0; r < E; ++r) {
        const uint32_t i = threadIdx.x * (uint32_t)E + (uint32_t)r;
        if (i < count) list[beg + i] = x[r];
    }
    __syncthreads();
}

// Put every tile's bucket of the position list in ascending order.  Up to 256 entries: each thread
// ranks its entry against the others in shared memory.  Up to 1024: a bitonic network in
// registers.  More: the entries set bits in a shared-memory bitmask of the tile, which is then read
// out in order (popcount scan).
__global__ void __launch_bounds__(kBlock) k_tile_sort(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    if (P.ctl->status) return;
    // the bitmask is stored with one pad word per 32 so that thread t's 32 consecutive words
    // (t*32 .. t*32+31 -> slots t*33 .. t*33+31) fall into 32 different banks for every t
    __shared__ uint32_t s_mask[kTileWords + kTileWords / 32];
    __shared__ uint32_t s_small[kBlock];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    static_assert(kTileWords == 32 * kBlock, "one thread reads out 32 words of the tile's bitmask");
    const uint32_t* __restrict__ tile_base = P.tile_base;
    uint32_t* __restrict__ list = P.idx;
    const uint32_t n_tiles = P.n_tiles;
    for (uint32_t tile = S.bx; tile < n_tiles; tile += S.nb) {
        const uint32_t beg = tile_base[tile], end = tile_base[tile + 1];
        const uint32_t count = end - beg;
        if (count <= 1u) continue;  // block-uniform
        if (count <= (uint32_t)kBlock) {
            const uint32_t x = (threadIdx.x < count) ? list[beg + threadIdx.x] : 0xffffffffu;
            s_small[threadIdx.x] = x;
            __syncthreads();
            uint32_t rank = 0u;
            for (uint32_t j = 0; j < count; ++j) rank += (s_small[j] < x) ? 1u : 0u;
            if (threadIdx.x < count) list[beg + rank] = x;
            __syncthreads();
            continue;
        }
        if (count <= 4u * kBlock) {  // block-uniform: a bitonic network in registers (larger ones lose to the bitmask)
            if (count <= 2u * kBlock) sort_bucket_in_registers<2>(list, beg, count, s_mask);
            else sort_bucket_in_registers<4>(list, beg, count, s_mask);
            continue;
        }
        for (int w = threadIdx.x; w < kTileWords + kTileWords / 32; w += kBlock) s_mask[w] = 0u;
        __syncthreads();
        for (uint32_t base = beg; base < end; base += 4 * kBlock) {  // four loads in flight per thread
            uint32_t v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t i = base + j * kBlock + threadIdx.x;
                v[j] = (i < end) ? list[i] : 0xffffffffu;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (v[j] != 0xffffffffu) {
                    const uint32_t r = v[j] & ((1u << kTileShift) - 1u);
                    const uint32_t word = r >> 5;
                    atomicOr(&s_mask[word + (word >> 5)], 1u << (r & 31u));
                }
            }
        }
        __syncthreads();
        // read-out in position order: thread t owns words t*32 .. t*32+31
        const uint32_t* mine_words = s_mask + threadIdx.x * 33;
        uint32_t mine = 0u;
#pragma unroll 8
        for (int j = 0; j < 32; ++j) mine += __popc(mine_words[j]);
        uint32_t total;
        uint32_t at = beg + block_exclusive_scan<uint32_t>(mine, s_scan, &total);
        if (mine) {
            const uint32_t first = (tile << kTileShift) + ((uint32_t)threadIdx.x << 10);
            for (int j = 0; j < 32; ++j) {
                uint32_t w = mine_words[j];
                while (w) {
                    const uint32_t idx = first + ((uint32_t)j << 5) + (__ffs(w) - 1);
                    w &= w - 1u;
                    if (at < end) list[at] = idx;
                    ++at;
                }
            }
        }
        __syncthreads();  // s_mask is cleared again for the next tile
    }
}

// ---------------------------------------------------------------- lengths, offsets, header

__device__ __forceinline__ unsigned long long codeword_len(const Prob& P, uint32_t i, uint32_t* gap) {
    const long long prev = i ? (long long)P.idx[i - 1] : -1ll;
    const uint32_t g = (uint32_t)((long long)P.idx[i] - prev - 1);  // gap - 1 of Algorithm 3
    *gap = g;
    return (unsigned long long)(g >> P.b) + 1ull + (unsigned long long)P.b;
}

__device__ __forceinline__ void store_u32(uint8_t* p, uint32_t v) { *reinterpret_cast<uint32_t*>(p) = v; }
__device__ __forceinline__ void store_u64(uint8_t* p, unsigned long long v) {
    *reinterpret_cast<unsigned long long*>(p) = v;
}

// The container header (one thread).  Written always, so that a failed encode still leaves a
// header that says why.
__device__ __forceinline__ void write_header(const Prob& P, Ctl* ctl, bool ok, unsigned long long nbits) {
    ctl->nbits = nbits;
    uint8_t* h = P.stream;
    store_u32(h + 0, SBC_MAGIC);
    store_u32(h + 4, SBC_VERSION);
    store_u64(h + 8, (unsigned long long)P.n);
    store_u64(h + 16, ok ? (unsigned long long)P.k : 0ull);
    store_u64(h + 24, nbits);
    store_u64(h + 32, ok ? P.payload_offset : (unsigned long long)SBC_HEADER_BYTES);
    store_u32(h + 40, (uint32_t)P.b);
    store_u32(h + 44, ok ? (P.mode == kModeValues ? SBC_SIDE_VALUES : __ldcg(&ctl->side)) : 0u);
    store_u32(h + 48, ok ? __float_as_uint(__ldcg(&ctl->mu32)) : 0u);
    store_u32(h + 52, SBC_CHUNK_CODEWORDS);
    store_u32(h + 56, ok ? P.n_chunks : 0u);
    store_u32(h + 60, __ldcg(&ctl->status));
}

// Scan of the per-block bit counts (written by other blocks: read from L2) and the container
// header, which is written always, so that a failed encode still leaves a header that says why.
// One block.
__device__ __forceinline__ void block_len_scan_header(const Prob& P, Ctl* ctl, unsigned long long* s_scan) {
    const bool ok = __ldcg(&ctl->status) == 0u;  // uniform: nothing writes status while this kernel runs
    unsigned long long total = 0ull;
    if (ok) {
        constexpr int kPer = 8;
        for (uint32_t base = 0; base < P.n_len_blocks; base += kBlock * kPer) {
            unsigned long long v[kPer];
            unsigned long long sum = 0ull;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t t = base + threadIdx.x * kPer + j;
                v[j] = (t < P.n_len_blocks) ? __ldcg(P.blk_len + t) : 0ull;
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
    if (threadIdx.x == 0) write_header(P, ctl, ok, total);
}

// Bits of each block of kLenBlock codewords, and -- since this is the first
// walk over the ordered position list -- the residual write-back
// R_j = A_j - mu at the kept positions (Algorithm 1), in address order.  The block that finishes
// last scans the block bit counts and writes the container header.
__global__ void __launch_bounds__(kBlock) k_len_sum_residual(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    const bool failed = ctl->status != 0u;  // uniform over the grid: no kernel of this stage sets it
    __shared__ unsigned long long s_scan[kBlock / 32 + 1];
    constexpr int kPer = kLenBlock / kBlock;
    const float mu = ctl->mu32;
    const uint32_t k = (uint32_t)P.k;
    // values mode: the kept values themselves are sent (they sit between the chunk table and the
    // payload, in position order) and nothing of them stays in the residual
    float* values = (P.mode == kModeValues)
        ? reinterpret_cast<float*>(P.stream + SBC_HEADER_BYTES + (size_t)P.n_chunks * SBC_CHUNK_ENTRY_BYTES)
        : nullptr;
    // R_j - mu as a fire-and-forget atomic add of -mu (no load round trip): the same single fp32
    // rounding as the subtraction.  The hardware's atomic adder treats subnormal operands and
    // results as zero, which cannot change the result while |mu| >= 2^-100: a subnormal R_j is less
    // than a quarter ulp of mu, and a non-zero difference of two values that close is a multiple of
    // 2^-124.  Smaller |mu| (zero included) takes the load / subtract / store path.
    const bool by_atomic = values == nullptr && fabsf(mu) >= 7.888609052e-31f;  // 2^-100
    for (uint32_t blk = S.bx; blk < (failed ? 0u : P.n_len_blocks); blk += S.nb) {
        const uint32_t i0 = blk * kLenBlock + threadIdx.x * kPer;
        uint32_t pos[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) pos[j] = (i0 + j < k) ? P.idx[i0 + j] : 0u;
        if (by_atomic) {
            // lane-contiguous: one warp instruction covers 32 neighbouring positions of the list, so
            // that updates of the same DRAM row reach the memory together (0.43 -> 0.39 ms for
            // 10.7 M positions over 4 GiB against four consecutive positions per thread)
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t i = blk * kLenBlock + (uint32_t)j * kBlock + threadIdx.x;
                if (i < k) atomicAdd(P.residual + P.idx[i], -mu);
            }
        } else {
            float r[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) r[j] = (i0 + j < k) ? P.residual[pos[j]] : 0.f;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                if (i0 + j < k) {
                    if (values) values[i0 + j] = r[j];
                    P.residual[pos[j]] = __fsub_rn(r[j], values ? r[j] : mu);
                }
            }
        }
        long long prev = (i0 && i0 < k) ? (long long)P.idx[i0 - 1] : -1ll;
        unsigned long long sum = 0ull;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            if (i0 + j < k) {
                const uint32_t g = (uint32_t)((long long)pos[j] - prev - 1);
                sum += (unsigned long long)(g >> P.b) + 1ull + (unsigned long long)P.b;
                prev = pos[j];
            }
        }
        unsigned long long total;
        block_exclusive_scan<unsigned long long>(sum, s_scan, &total);
        if (threadIdx.x == 0) P.blk_len[blk] = total;
    }
    // by the block that finishes last: bit offset of every block, total bits, header
    if (last_block_ticket(&ctl->done[ST_LEN], S.nb)) block_len_scan_header(P, ctl, s_scan);
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

// Codeword i (gap g, Golomb parameter b) at stream bit `off`: q = g >> b ones, a zero, then g's low
// b bits MSB first (Algorithm 3), ORed into the zeroed payload; the first codeword of a chunk also
// writes the chunk's table entry (bit offset, position of the codeword before it, taken from the
// ascending position list).
// `words` holds the payload from stream bit `bit_base` on (the payload itself: 0; a staging buffer
// in shared memory: the bit at which the buffer starts, a multiple of 32).
__device__ __forceinline__ void pack_codeword(uint32_t* words, unsigned long long bit_base, uint8_t* table, uint32_t i,
                                              unsigned long long off, uint32_t g, int b, const uint32_t* positions) {
    if (i % kChunkCodewords == 0) {
        uint8_t* e = table + (size_t)(i / kChunkCodewords) * SBC_CHUNK_ENTRY_BYTES;
        store_u64(e, off);
        store_u64(e + 8, (unsigned long long)(i ? (long long)positions[i - 1] : -1ll));
    }
    unsigned long long pos = off - bit_base;
    uint32_t q = g >> b;
    // q ones: head up to a word boundary, whole words, then the rest
    if (q) {
        const int head = min((uint32_t)(32 - (int)(pos & 31ull)) & 31u, q);
        if (head) { or_bits(words, pos, head, 0xffffffffu >> (32 - head)); pos += head; q -= head; }
        while (q >= 32u) { words[pos >> 5] = 0xffffffffu; pos += 32; q -= 32u; }
        if (q) { or_bits(words, pos, (int)q, 0xffffffffu >> (32 - q)); pos += q; }
    }
    // the terminating zero and r in b bits, MSB first: 1 + b <= 31 bits
    or_bits(words, pos, 1 + b, g & ((1u << b) - 1u));
}

// Bit offset of every codeword (block scan over the lengths) and the payload bits themselves, every
// codeword ORed into the zeroed payload on its own.  (Putting a block's bit range together in
// shared memory first and storing whole words was measured slower: 79 instead of 62 us for 10.7 M
// codewords; the atomics of many blocks on the L2-resident payload do not wait for one another.)
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
            pack_codeword(words, 0ull, table, i, off, gap[j], b, P.idx);
            off += len[j];
        }
    }
}

}  // namespace sbc
