// Golomb position coding (Algorithm 3) of the kept positions, and the residual write-back at
// those positions (Algorithm 1).
//
// The candidates of the chosen side lie in position order, span by span (see k_add_collect).  Two
// kernels walk them with the same split into warp ranges: k_span_count adds up, per range, how
// many entries are kept and how many payload bits they take, and its last block turns the range
// sums into the rank, bit offset and previous position every range starts from (and writes the
// header); k_span_emit walks again and, for every kept entry, subtracts mu from the residual,
// ORs the codeword into the pre-zeroed payload and writes the chunk-table entries.
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

// ---------------------------------------------------------------- header

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
    store_u32(h + 52, P.chunk_cw);
    store_u32(h + 56, ok ? P.n_chunks : 0u);
    store_u32(h + 60, __ldcg(&ctl->status));
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
// writes the chunk's table entry (bit offset, position of the codeword before it: prev_plus1 - 1).
__device__ __forceinline__ void pack_codeword(uint32_t* words, uint8_t* table, uint32_t chunk_cw, uint32_t i,
                                              unsigned long long off, uint32_t g, int b, uint32_t prev_plus1) {
    if (i % chunk_cw == 0u) {
        uint8_t* e = table + (size_t)(i / chunk_cw) * SBC_CHUNK_ENTRY_BYTES;
        store_u64(e, off);
        store_u64(e + 8, (unsigned long long)((long long)prev_plus1 - 1ll));
    }
    unsigned long long pos = off;
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

// ---------------------------------------------------------------- candidates in position order

// Calls on_batch(composite, valid) for every 32 consecutive entries of the position-ordered
// candidates of spans [span0, span1) of side `s`, in ascending order; lane j of a call holds entry
// 32 * call + j.  All 32 lanes call and on_batch runs warp-uniformly.  The records of 32 spans are
// read at once; a batch may straddle spans (lane j finds its span by a search over the scanned counts).
template <typename F>
__device__ __forceinline__ void walk_spans(const Prob& P, int s, uint32_t span0, uint32_t span1, F&& on_batch) {
    const uint2* __restrict__ rec = P.span_rec[s];
    const unsigned long long* __restrict__ list = P.list[s];
    const uint32_t lane = lane_id();
    const uint32_t list_cap = P.list_cap;
    for (uint32_t sp = span0; sp < span1; sp += 32u) {
        uint2 r = make_uint2(0u, 0u);
        if (sp + lane < span1) r = rec[sp + lane];
        if (r.x > list_cap || r.y > list_cap - r.x) r.y = 0u;  // a record that points outside the list holds nothing
        const uint32_t incl = warp_inclusive_scan(r.y);
        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
        const uint32_t excl = incl - r.y;
        for (uint32_t t0 = 0u; t0 < total; t0 += 32u) {
            const uint32_t t = t0 + lane;
            const bool valid = t < total;
            // the span of entry t: the last lane whose exclusive count is <= t
            uint32_t at = 0u;
#pragma unroll
            for (uint32_t step = 16u; step > 0u; step >>= 1) {
                const uint32_t e = __shfl_sync(0xffffffffu, excl, (int)((at + step) & 31u));
                if (at + step < 32u && e <= t) at += step;
            }
            const uint32_t off = __shfl_sync(0xffffffffu, r.x, (int)at);
            const uint32_t ex = __shfl_sync(0xffffffffu, excl, (int)at);
            const unsigned long long c = valid ? list[off + (t - ex)] : 0ull;
            on_batch(c, valid);
        }
    }
}

// Spans [first, last) of warp range `r` when n_spans spans are split evenly over n_ranges ranges.
__device__ __forceinline__ void range_spans(uint32_t n_spans, uint32_t n_ranges, uint32_t r, uint32_t* first, uint32_t* last) {
    const uint32_t per = (n_spans + n_ranges - 1u) / n_ranges;
    *first = min(n_spans, r * per);
    *last = min(n_spans, *first + per);
}

// `A` followed by `B` (ranges that lie one after the other): the code lengths of B's first entry,
// whose gap reaches back to A's last, becomes an inner one.
__device__ __forceinline__ RangeSum fold_ranges(RangeSum A, const RangeSum& B, int b) {
    if (B.cnt == 0u) return A;
    if (A.cnt == 0u) return B;
    const uint32_t g = B.first - (A.last + 1u);
    A.inner_bits += (unsigned long long)(g >> b) + 1ull + (unsigned long long)b + B.inner_bits;
    A.cnt += B.cnt;
    A.last = B.last;
    return A;
}
__device__ __forceinline__ RangeSum load_range_sum(const RangeSum* p) {
    RangeSum r;
    r.cnt = __ldcg(&p->cnt); r.first = __ldcg(&p->first); r.last = __ldcg(&p->last); r.pad_ = 0u;
    r.inner_bits = __ldcg(&p->inner_bits);
    return r;
}

// Per warp range (the spans one warp of k_span_emit will walk): number of kept entries, first and
// last kept position, and the code lengths of all kept entries but the first (its gap reaches back
// into an earlier range); the same for the block's eight ranges together.  The last block to
// finish combines the blocks in order: for every block the rank of its first kept entry, the
// position kept just before it and the bit offset of its first codeword; then the header.
template <bool DENSE_SPANS>
__global__ void __launch_bounds__(kBlock, 6) k_span_count(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    const bool failed = ctl->status != 0u;  // uniform over the grid: no kernel of this stage sets it before the ticket
    const int s = (int)ctl->side;
    const unsigned long long thr = ctl->thr[s];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    constexpr uint32_t kWarps = kBlock / 32;
    const uint32_t n_ranges = S.nb * kWarps;
    const uint32_t range = S.bx * kWarps + warp;
    const int b = P.b;
    // one buffer for two phases: the lanes' sums of this block's warps (long spans), then (last block only) all blocks' sums
    __shared__ RangeSum s_buf[kOrderBlocksMax > kWarps * 32u ? kOrderBlocksMax : kWarps * 32u];
    RangeSum (*s_lane)[32] = reinterpret_cast<RangeSum (*)[32]>(s_buf);
    __shared__ RangeSum s_rs[kWarps];
    // DENSE_SPANS (the host's choice: sixteen kept entries or more per span on average, and spans
    // enough to give most threads of the machine one): one THREAD
    // walks a span by itself -- a compare and a handful of integer operations per entry, no
    // shuffles; a thread's loads stay within a few cache lines.  Otherwise the warp walks its range
    // 32 entries at a time, as k_span_emit does (with a thread per span nearly every load would be
    // a sector of its own and the work of the lanes uneven).  Same result either way.
    if (!failed) {
        uint32_t span0, span1;
        range_spans(P.n_spans, n_ranges, range, &span0, &span1);
        if (DENSE_SPANS) {
            // lane i takes spans [span0 + i * per_lane, span0 + (i + 1) * per_lane) of the range
            const uint32_t per_lane = (span1 - span0 + 31u) / 32u;
            const uint32_t my0 = min(span1, span0 + lane * per_lane), my1 = min(span1, my0 + per_lane);
            const uint2* __restrict__ rec = P.span_rec[s];
            const unsigned long long* __restrict__ list = P.list[s];
            const uint32_t list_cap = P.list_cap;
            RangeSum mine;
            mine.cnt = 0u; mine.first = 0u; mine.last = 0u; mine.pad_ = 0u; mine.inner_bits = 0ull;
            uint32_t pp1 = 0u;
            for (uint32_t sp = my0; sp < my1; ++sp) {
                uint2 r = rec[sp];
                if (r.x > list_cap || r.y > list_cap - r.x) r.y = 0u;  // a record that points outside the list holds nothing
                const unsigned long long* __restrict__ e = list + r.x;
                auto take = [&](unsigned long long c) {
                    if (c >= thr) {
                        const uint32_t pos = composite_index(c);
                        if (mine.cnt == 0u) mine.first = pos;
                        else mine.inner_bits += (unsigned long long)((pos - pp1) >> b) + 1ull + (unsigned long long)b;
                        pp1 = pos + 1u;
                        ++mine.cnt;
                    }
                };
                // two entries per load (every lane's load is a sector of its own here, and the load
                // unit takes such an instruction apart lane by lane: half as many instructions, half
                // the time): an odd first entry and an odd last one by themselves
                uint32_t j0 = 0u;
                if ((r.x & 1u) && r.y) { take(e[0]); j0 = 1u; }
                const ulonglong2* __restrict__ e2 = reinterpret_cast<const ulonglong2*>(e + j0);   // the lists start on 256-byte boundaries
                const uint32_t pairs = (r.y - j0) >> 1;
                constexpr int kLoads = 4;   // loads in flight per thread
                for (uint32_t q0 = 0u; q0 < pairs; q0 += kLoads) {
                    ulonglong2 v[kLoads];
#pragma unroll
                    for (int j = 0; j < kLoads; ++j) v[j] = (q0 + j < pairs) ? e2[q0 + j] : make_ulonglong2(0ull, 0ull);
#pragma unroll
                    for (int j = 0; j < kLoads; ++j)
                        if (q0 + j < pairs) { take(v[j].x); take(v[j].y); }
                }
                if ((r.y - j0) & 1u) take(e[r.y - 1u]);
            }
            mine.last = pp1 - 1u;
            // the lanes' sums in order, by lane 0
            s_lane[warp][lane] = mine;
            __syncwarp();
            if (lane == 0u) {
                RangeSum all = s_lane[warp][0];
                for (uint32_t l = 1u; l < 32u; ++l) all = fold_ranges(all, s_lane[warp][l], b);
                P.rng_sum[range] = all;
                s_rs[warp] = all;
            }
        } else {
        const unsigned lt = (1u << lane) - 1u;
        uint32_t cnt = 0u, first = 0u, prev_plus1 = 0u;   // the same in all lanes
        unsigned long long inner = 0ull;                   // each lane adds up the code lengths of the entries it sees
        walk_spans(P, s, span0, span1, [&](unsigned long long c, bool valid) {
            const bool kept = valid && c >= thr;
            const unsigned m = __ballot_sync(0xffffffffu, kept);
            if (m == 0u) return;  // warp-uniform
            const uint32_t pos = composite_index(c);
            const unsigned lower = m & lt;
            const uint32_t before = __shfl_sync(0xffffffffu, pos, lower ? 31 - __clz((int)lower) : 0);
            const bool opens = cnt == 0u && lower == 0u;   // the range's first kept entry: its gap reaches into an earlier range
            if (kept && !opens) {
                const uint32_t pp = lower ? before + 1u : prev_plus1;   // previous kept position, plus one
                inner += (unsigned long long)((pos - pp) >> b) + 1ull + (unsigned long long)b;
            }
            if (cnt == 0u) first = __shfl_sync(0xffffffffu, pos, __ffs((int)m) - 1);
            prev_plus1 = __shfl_sync(0xffffffffu, pos, 31 - __clz((int)m)) + 1u;
            cnt += (uint32_t)__popc(m);
        });
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) inner += __shfl_down_sync(0xffffffffu, inner, d);
        if (lane == 0u) {
            RangeSum all;
            all.cnt = cnt; all.first = first; all.last = prev_plus1 - 1u; all.pad_ = 0u; all.inner_bits = inner;
            P.rng_sum[range] = all;
            s_rs[warp] = all;
        }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            RangeSum all = s_rs[0];
            for (uint32_t w = 1; w < kWarps; ++w) all = fold_ranges(all, s_rs[w], b);
            P.blk_sum[S.bx] = all;
        }
    }
    if (!last_block_ticket(&ctl->done[ST_ORDER], S.nb)) return;
    // ---- the last block: blocks in order.  Thread t takes blocks [t * per, (t + 1) * per).
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ unsigned long long s_scan64[kBlock / 32 + 1];
    __shared__ uint32_t s_last[kBlock / 32];   // per warp: last kept position + 1 within its threads' blocks (0: none)
    RangeSum* const s_blk = s_buf;   // the ticket's barriers lie between the two uses
    if (failed || S.nb > kOrderBlocksMax) {
        if (threadIdx.x == 0) {
            if (!failed) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            write_header(P, ctl, false, 0ull);
        }
        return;
    }
    for (uint32_t i = threadIdx.x; i < S.nb; i += kBlock) s_blk[i] = load_range_sum(P.blk_sum + i);
    __syncthreads();
    const uint32_t per = (S.nb + kBlock - 1u) / kBlock;
    const uint32_t r0 = min(S.nb, threadIdx.x * per), r1 = min(S.nb, r0 + per);
    RangeSum mine;
    mine.cnt = 0u; mine.first = 0u; mine.last = 0u; mine.pad_ = 0u; mine.inner_bits = 0ull;
    for (uint32_t r = r0; r < r1; ++r) mine = fold_ranges(mine, s_blk[r], b);
    uint32_t total_cnt;
    uint32_t rank = block_exclusive_scan<uint32_t>(mine.cnt, s_scan, &total_cnt);
    // last kept position (plus one) before this thread's blocks: positions only grow from thread to
    // thread, so it is the maximum over the earlier threads
    uint32_t pp;
    {
        const uint32_t mine_last = mine.cnt ? mine.last + 1u : 0u;
        uint32_t incl = mine_last;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
            if ((int)lane >= d) incl = max(incl, o);
        }
        if (lane == 31u) s_last[warp] = incl;
        __syncthreads();
        uint32_t before = 0u;
        for (uint32_t w = 0; w < warp; ++w) before = max(before, s_last[w]);
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, 1);
        pp = max(before, lane ? up : 0u);
    }
    // bits of this thread's blocks, now that the gap of its first entry is known
    const unsigned long long my_bits =
        mine.cnt ? (unsigned long long)((mine.first - pp) >> b) + 1ull + (unsigned long long)b + mine.inner_bits : 0ull;
    unsigned long long total_bits;
    unsigned long long bit = block_exclusive_scan<unsigned long long>(my_bits, s_scan64, &total_bits);
    for (uint32_t r = r0; r < r1; ++r) {
        RangeBase rb;
        rb.rank = rank; rb.prev_plus1 = pp; rb.bit = bit;
        P.blk_base[r] = rb;
        const RangeSum& q = s_blk[r];
        if (q.cnt == 0u) continue;
        bit += (unsigned long long)((q.first - pp) >> b) + 1ull + (unsigned long long)b + q.inner_bits;
        pp = q.last + 1u;
        rank += q.cnt;
    }
    if (threadIdx.x == 0) {
        ctl->kept_total = total_cnt;
        const bool ok = total_cnt == (uint32_t)P.k;
        if (!ok) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
        write_header(P, ctl, ok, ok ? total_bits : 0ull);
    }
}

// Second walk: every kept entry gets its rank and bit offset from the range's start values and
// does its three jobs -- R_j -= mu (Algorithm 1), its codeword into the payload, and, if it
// opens a chunk, the chunk's table entry (Algorithm 3).  A warp instruction covers 32 neighbouring
// list entries, i.e. neighbouring positions of the tensor, so that updates of the same DRAM row
// reach the memory together.
__global__ void __launch_bounds__(kBlock) k_span_emit(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status != 0u) return;
    const int s = (int)ctl->side;
    const unsigned long long thr = ctl->thr[s];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    const uint32_t n_ranges = S.nb * (kBlock / 32);
    const uint32_t range = S.bx * (kBlock / 32) + warp;
    const int b = P.b;
    const float mu = ctl->mu32;
    const uint32_t k = (uint32_t)P.k, chunk_cw = P.chunk_cw;
    uint32_t* words = reinterpret_cast<uint32_t*>(P.stream + P.payload_offset);
    uint8_t* table = P.stream + SBC_HEADER_BYTES;
    float* __restrict__ R = P.residual;
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
    uint32_t span0, span1;
    range_spans(P.n_spans, n_ranges, range, &span0, &span1);
    // where this warp's range starts: the block's start values, advanced over the block's earlier ranges
    const RangeBase rb = P.blk_base[S.bx];
    uint32_t rank = rb.rank, prev_plus1 = rb.prev_plus1;
    unsigned long long bit = rb.bit;
    {
        RangeSum mine;
        mine.cnt = 0u; mine.first = 0u; mine.last = 0u; mine.pad_ = 0u; mine.inner_bits = 0ull;
        if (lane < kBlock / 32) mine = P.rng_sum[S.bx * (kBlock / 32) + lane];
        for (uint32_t w = 0; w < warp; ++w) {  // warp-uniform bound
            const uint32_t c = __shfl_sync(0xffffffffu, mine.cnt, (int)w);
            const uint32_t f = __shfl_sync(0xffffffffu, mine.first, (int)w);
            const uint32_t l = __shfl_sync(0xffffffffu, mine.last, (int)w);
            const unsigned long long in = __shfl_sync(0xffffffffu, mine.inner_bits, (int)w);
            if (c == 0u) continue;
            bit += (unsigned long long)((f - prev_plus1) >> b) + 1ull + (unsigned long long)b + in;
            prev_plus1 = l + 1u;
            rank += c;
        }
    }
    walk_spans(P, s, span0, span1, [&](unsigned long long c, bool valid) {
        const bool kept = valid && c >= thr;
        const unsigned m = __ballot_sync(0xffffffffu, kept);
        if (m == 0u) return;  // warp-uniform
        const uint32_t pos = composite_index(c);
        const unsigned lower = m & lt;
        const uint32_t before = __shfl_sync(0xffffffffu, pos, lower ? 31 - __clz((int)lower) : 0);
        const uint32_t pp = lower ? before + 1u : prev_plus1;   // previous kept position, plus one
        const uint32_t g = kept ? pos - pp : 0u;
        const unsigned long long len = kept ? (unsigned long long)(g >> b) + 1ull + (unsigned long long)b : 0ull;
        // bit offsets: 32-bit scan unless a long unary run is among the 32 (then 64-bit)
        unsigned long long off;
        if (__any_sync(0xffffffffu, len >= (1ull << 26))) {
            const unsigned long long incl = warp_inclusive_scan(len);
            off = bit + incl - len;
            bit += __shfl_sync(0xffffffffu, incl, 31);
        } else {
            const uint32_t incl = warp_inclusive_scan((uint32_t)len);
            off = bit + (incl - (uint32_t)len);
            bit += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (kept) {
            const uint32_t i = rank + (uint32_t)__popc(lower);
            if (i < k && pos < (uint32_t)P.n) {
                if (by_atomic) {
                    atomicAdd(R + pos, -mu);
                } else {
                    const float r = R[pos];
                    if (values) values[i] = r;
                    R[pos] = __fsub_rn(r, values ? r : mu);
                }
                pack_codeword(words, table, chunk_cw, i, off, g, b, pp);
            }
        }
        prev_plus1 = __shfl_sync(0xffffffffu, pos, 31 - __clz((int)m)) + 1u;
        rank += (uint32_t)__popc(m);
    });
}

}  // namespace sbc
