// Exact k-th largest composite of each side's candidates (Algorithm 2: exactly k
// kept entries, equal values ordered by index), by MSB-first radix selection
// with 11-bit digits over the 64-bit composites, and, on the way, the exact sums
// of the kept values, the two means, the side choice and mu (Algorithm 2).
//
// A first kernel (k_select_hist0) takes the histogram of the first digit over the list that is
// ranked and picks the bucket of the k-th largest entry.  A second one over the list
// (k_select_filter0) then adds up everything in the buckets above (kept for sure) and
// keeps the entries of the picked bucket, which are few: the last block of each side to finish
// ranks those and adds the kept ones among them, and the block that completes the second side
// turns the sums into the means and takes the side decision.
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// Rank `rank` (1 = largest) among the cnt <= PER * kBlock composites a block holds in registers
// (slot j of thread t = entry j * kBlock + t; SelectDigits::sub already taken off), which agree in
// every digit before `first_level` (`prefix` holds those digits).  Radix selection, 11-bit digits
// from bit `top` down, on shared-memory histograms; stops at the first bucket with a single entry.
// Returns false if the histogram walk failed (inconsistent counts).  All threads call; result
// identical in all.
template <int PER>
__device__ __forceinline__ bool block_select_registers(const unsigned long long (&c)[PER], uint32_t cnt, uint32_t rank,
                                                       int top, int first_level, unsigned long long prefix, uint32_t* s_hist,
                                                       uint32_t* s_scan, Pick* s_pick, unsigned long long* s_result,
                                                       unsigned long long* out) {
    unsigned alive = 0u;  // entries that still match the prefix
#pragma unroll
    for (int j = 0; j < PER; ++j) alive |= ((uint32_t)j * kBlock + threadIdx.x < cnt) ? (1u << j) : 0u;
    const int levels = digit_levels(top);
    for (int level = first_level; level < levels; ++level) {
        for (int i = threadIdx.x; i < kHistBins; i += kBlock) s_hist[i] = 0u;
        __syncthreads();
        // a thread's entries mostly share their leading digits: one atomic per run of equal digits
        uint32_t run_digit = 0u, run_len = 0u;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if ((alive >> j) & 1u) {
                const uint32_t d = digit_of(c[j], level, top);
                if (run_len && d != run_digit) { atomicAdd(&s_hist[run_digit], run_len); run_len = 0u; }
                run_digit = d;
                ++run_len;
            }
        }
        if (run_len) atomicAdd(&s_hist[run_digit], run_len);
        __syncthreads();
        block_pick_desc<true>(s_hist, 1 << digit_bits(level, top), false, rank, s_scan, s_pick);
        if (!s_pick->found) return false;  // uniform
        const uint32_t sel = s_pick->bin;
        const bool single = s_pick->count == 1u;
        rank = s_pick->rank;
        prefix |= (unsigned long long)sel << digit_shift(level, top);
#pragma unroll
        for (int j = 0; j < PER; ++j)
            if (((alive >> j) & 1u) && digit_of(c[j], level, top) != sel) alive &= ~(1u << j);
        if (single) {  // the one entry left is the answer; its owner publishes it
#pragma unroll
            for (int j = 0; j < PER; ++j)
                if ((alive >> j) & 1u) *s_result = c[j];
            __syncthreads();
            *out = *s_result;
            return true;
        }
        __syncthreads();  // s_pick and s_hist are reused
    }
    *out = prefix;  // every digit fixed
    return true;
}

// Highest bit set in any of a block's values (all threads call, result in all; s_tmp: one word per
// warp).  A list that is ranked by one block starts its digits there: with no upper bound on its
// keys the range the digits were laid out for is mostly empty at the top.
__device__ __forceinline__ int block_top_bit(unsigned long long any_bits, unsigned long long* s_tmp) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) any_bits |= __shfl_xor_sync(0xffffffffu, any_bits, d);
    __syncthreads();  // s_tmp may still be read from an earlier use
    if (lane_id() == 0) s_tmp[threadIdx.x >> 5] = any_bits;
    __syncthreads();
    unsigned long long all = 0ull;
#pragma unroll
    for (int w = 0; w < kBlock / 32; ++w) all |= s_tmp[w];
    return all ? 63 - __clzll((long long)all) : 0;
}

constexpr int kFinishPer = 8;  // entries per thread the short rest of a side is ranked from in registers
constexpr uint32_t kFinishList = kFinishPer * kBlock;

// The fp32 bit pattern behind a composite of side s (binarised form: the key is the ordered image
// of the signed value, complemented for the negative side).
__device__ __forceinline__ uint32_t value_bits_of(int s, unsigned long long c) {
    return bits_of_key(side_key(s, (uint32_t)(c >> 32)));
}

// ---------------------------------------------------------------- exact sums, means, side

// Which of a block's 256 bins (bins[threadIdx.x]) are not zero, one bit each, into nonzero[0..8)
// (shared).  All kBlock threads call; valid after the next barrier.
__device__ __forceinline__ void bins_nonzero_masks(long long mine, uint32_t* nonzero) {
    const unsigned m = __ballot_sync(0xffffffffu, mine != 0);
    if (lane_id() == 0) nonzero[threadIdx.x >> 5] = m;
}

// Round the exact integer sum_s bins[s] * 2^s (units of 2^-149) to fp64,
// nearest-even.  One thread.  `nonzero` has bit (s & 31) of word s >> 5 set for every bin that is
// not zero (8 words, from bins_nonzero_masks): only those are visited.
__device__ double bins_to_double(const long long* bins, const uint32_t* nonzero) {
    unsigned long long acc[6] = {0, 0, 0, 0, 0, 0};  // 384-bit two's complement
    for (int word = 0; word < 8; ++word)
    for (uint32_t left = nonzero[word]; left; left &= left - 1u) {
        const int s = word * 32 + __ffs(left) - 1;
        if (s >= kSumBins) continue;
        const long long v = bins[s];
        const int limb = s >> 6, off = s & 63;
        unsigned long long part[3];
        part[0] = (unsigned long long)v << off;
        part[1] = off ? (unsigned long long)(v >> (64 - off)) : (v < 0 ? ~0ull : 0ull);
        part[2] = v < 0 ? ~0ull : 0ull;
        unsigned long long carry = 0;
        for (int l = limb; l < 6; ++l) {
            const unsigned long long add = part[min(l - limb, 2)];
            const unsigned long long t = acc[l] + add;
            const unsigned long long c1 = t < add;
            const unsigned long long t2 = t + carry;
            const unsigned long long c2 = t2 < carry;
            acc[l] = t2;
            carry = c1 | c2;
        }
    }
    const bool neg = (acc[5] >> 63) != 0;
    if (neg) {
        unsigned long long carry = 1;
        for (int l = 0; l < 6; ++l) {
            acc[l] = ~acc[l] + carry;
            carry = (carry && acc[l] == 0) ? 1 : 0;
        }
    }
    int top = -1;
    for (int l = 5; l >= 0; --l)
        if (acc[l]) { top = l * 64 + 63 - __clzll((long long)acc[l]); break; }
    if (top < 0) return 0.0;
    // shift right so that bit `top` lands on bit 52, tracking round and sticky bits
    const int drop = top - 52;
    unsigned long long sig = 0;
    bool round_bit = false, sticky = false;
    if (drop <= 0) {
        sig = acc[0] << (-drop);  // top <= 52: everything sits in limb 0
    } else {
        const int limb = drop >> 6, off = drop & 63;
        const unsigned long long lo = acc[limb];
        const unsigned long long hi = (limb + 1 < 6) ? acc[limb + 1] : 0ull;
        sig = off ? ((lo >> off) | (hi << (64 - off))) : lo;
        sig &= (1ull << 53) - 1ull;
        const int rpos = drop - 1;
        round_bit = (acc[rpos >> 6] >> (rpos & 63)) & 1ull;
        for (int l = 0; l < (rpos >> 6); ++l) sticky |= acc[l] != 0;
        if (rpos & 63) sticky |= (acc[rpos >> 6] & ((1ull << (rpos & 63)) - 1ull)) != 0;
    }
    if (round_bit && (sticky || (sig & 1ull))) sig += 1ull;
    const double mag = scalbn((double)sig, drop - 149);  // sig <= 2^53: exact
    return neg ? -mag : mag;
}

// The bins of both sides are complete: the two means, Algorithm 2's side decision, mu.  One block,
// all threads call.  On the fast route the entries above the sample's upper bound of the threshold
// were summed while the streaming pass flushed them (pre_bins).
__device__ __forceinline__ void sums_decide_finish(const Prob& P, const Slot& S, Ctl* ctl, unsigned long long (&s_bins)[2][256],
                                                   uint32_t (&s_nonzero)[2][8]) {
    if (__ldcg(&ctl->status) != 0u) return;  // uniform: read after the ticket's barrier, nothing sets it any more
    const bool values_mode = P.mode == kModeValues;
    const bool pre = !ctl->use_fallback && !values_mode;
    const long long b0 = __ldcg(&ctl->bins[0][threadIdx.x]) + (pre ? __ldcg(&ctl->pre_bins[0][threadIdx.x]) : 0ll);
    const long long b1 = __ldcg(&ctl->bins[1][threadIdx.x]) + (pre ? __ldcg(&ctl->pre_bins[1][threadIdx.x]) : 0ll);
    __syncthreads();  // the caller's own use of s_bins is over
    s_bins[0][threadIdx.x] = (unsigned long long)b0;
    s_bins[1][threadIdx.x] = (unsigned long long)b1;
    bins_nonzero_masks(b0, s_nonzero[0]);
    bins_nonzero_masks(b1, s_nonzero[1]);
    __syncthreads();
    if (threadIdx.x < 2) {  // one thread per side rounds its exact sum
        const double sum = bins_to_double(reinterpret_cast<const long long*>(s_bins[threadIdx.x]), s_nonzero[threadIdx.x]);
        // mean over the k selected entries, or over however many the sampled threshold let through
        const double count = ctl->sampled_ok ? (double)__ldcg(&ctl->cand_cnt[threadIdx.x]) : (double)P.k;
        ctl->mu64[threadIdx.x] = threadIdx.x ? -sum / count : sum / count;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const double mu_pos = ctl->mu64[0];
        const double mu_neg = ctl->mu64[1];  // val- holds the negated entries
        const uint32_t side = values_mode ? 0u : ((mu_pos >= mu_neg) ? 0u : 1u);
        const float mu = values_mode ? 0.f : (side ? (float)(-mu_neg) : (float)mu_pos);
        ctl->side = side;
        ctl->mu32 = mu;
        if (P.out_mu) *P.out_mu = mu;
        const uint32_t k_final = ctl->sampled_ok ? __ldcg(&ctl->cand_cnt[side]) : (uint32_t)P.k;
        ctl->k_final = k_final;
        if (P.sampled) {  // the kernels that follow size their work from the descriptor
            const uint32_t cw = chunk_codewords_for(k_final);
            S.G->k = k_final;
            S.G->chunk_cw = cw;
            S.G->n_chunks = (k_final + cw - 1u) / cw;
            S.G->payload_offset = SBC_HEADER_BYTES + (unsigned long long)S.G->n_chunks * SBC_CHUNK_ENTRY_BYTES;
        }
    }
}

// ---------------------------------------------------------------- first digit

// Histogram of the first digit over the list that is ranked; the last block of a side to finish
// picks the bucket of the k-th largest entry (b_prefix, b_rank).  grid.z = side.
__global__ void __launch_bounds__(kBlock) k_select_hist0(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status || ctl->sampled_ok) return;  // sampled thresholds: every candidate is kept
    const int s = blockIdx.z;
    if (s == 1 && P.mode == kModeValues) return;  // magnitude selection has one side only
    if (ctl->sel_done[s]) return;                 // exact route: the gathered list is the kept set
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) s_hist[i] = 0u;
    __syncthreads();
    const BandView view = band_view(P, ctl, s);
    const uint32_t cnt = view.count;
    const SelectDigits dg = select_digits(ctl, s);
    constexpr int kItems = 4;  // loads in flight per thread
    for (uint32_t base = S.bx * (kBlock * kItems); base < cnt; base += S.nb * (kBlock * kItems)) {
        unsigned long long c[kItems];
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const uint32_t i = base + j * kBlock + threadIdx.x;
            c[j] = (i < cnt) ? view.src[i] : dg.sub;
        }
#pragma unroll
        for (int j = 0; j < kItems; ++j)
            if (base + j * kBlock + threadIdx.x < cnt) atomicAdd(&s_hist[digit_of(c[j] - dg.sub, 0, dg.top)], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&P.hists->b0[s][i], v);
    }
    if (last_block_ticket(&ctl->done[ST_HIST_S0 + s], S.nb)) select_pick0(P, ctl, s, view.rank, dg.top, s_scan, &s_pick);
}

// ---------------------------------------------------------------- one pass over the ranked list

// Shared memory of the block that ranks the short rest of a side.
struct RestShared {
    uint32_t hist[kHistBins];
    uint32_t scan[kBlock / 32 + 1];
    Pick pick;
    unsigned long long result;
    uint32_t fill;
};

// Ranks what the pass over the list left (the entries that share the first digit with the k-th
// largest): at most kFinishList entries in registers, all remaining digits at once; a longer rest
// (many entries with the same value around the threshold) digit by digit from global memory.  Adds
// the values of the kept ones to the side's sums (s_bins, zeroed by the caller; added to the
// control block's here).  One block, all threads call.
__device__ __forceinline__ void select_rest_side(const Prob& P, Ctl* ctl, int s, RestShared& sh, unsigned long long* s_bins) {
    const bool values_mode = P.mode == kModeValues;
    const SelectDigits dg = select_digits(ctl, s);
    const int top = dg.top, levels = digit_levels(top);
    ExactSum sum;
    sum.start(value_bits_of(s, dg.sub));
    const unsigned long long* src = P.buf[s][0];
    unsigned long long* dst = P.buf[s][1];
    uint32_t n = min(__ldcg(&ctl->list_cnt[s]), P.cap), rank = __ldcg(&ctl->b_rank[s]);
    unsigned long long prefix = __ldcg(&ctl->b_prefix[s]), thr_rel = 0ull;
    bool good = true;
    for (int level = 1; ; ++level) {
        if (n <= kFinishList) {
            unsigned long long c[kFinishPer];
#pragma unroll
            for (int j = 0; j < kFinishPer; ++j) {
                const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
                c[j] = (i < n) ? __ldcg(src + i) : 0ull;   // written by other blocks of this kernel
            }
            good = block_select_registers<kFinishPer>(c, n, rank, top, level, prefix, sh.hist, sh.scan, &sh.pick, &sh.result, &thr_rel);
            if (good && !values_mode) {
#pragma unroll
                for (int j = 0; j < kFinishPer; ++j)
                    if ((uint32_t)j * kBlock + threadIdx.x < n && c[j] >= thr_rel) sum.add(value_bits_of(s, c[j] + dg.sub), s_bins);
            }
            break;
        }
        if (level >= levels) { good = false; break; }  // cannot happen: composites are distinct
        // a long rest: histogram of this level's digit, pick, then filter, this block alone
        for (int i = threadIdx.x; i < kHistBins; i += kBlock) sh.hist[i] = 0u;
        if (threadIdx.x == 0) sh.fill = 0u;
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < n; i += kBlock) atomicAdd(&sh.hist[digit_of(__ldcg(src + i), level, top)], 1u);
        __syncthreads();
        block_pick_desc<true>(sh.hist, 1 << digit_bits(level, top), false, rank, sh.scan, &sh.pick);
        if (!sh.pick.found) { good = false; break; }  // uniform
        const uint32_t sel = sh.pick.bin;
        rank = sh.pick.rank;
        prefix |= (unsigned long long)sel << digit_shift(level, top);
        const bool last = level + 1 == levels;  // every digit fixed after this one: the entry in `sel` is the k-th largest itself
        for (uint32_t base = 0u; base < n; base += kBlock) {
            const uint32_t i = base + threadIdx.x;
            const unsigned long long c = (i < n) ? __ldcg(src + i) : 0ull;
            const uint32_t d = digit_of(c, level, top);
            const bool keep = i < n && (d > sel || (last && d == sel));
            const bool match = i < n && !last && d == sel;
            if (keep && !values_mode) sum.add(value_bits_of(s, c + dg.sub), s_bins);
            uint32_t total;
            const uint32_t excl = block_exclusive_scan<uint32_t>(match ? 1u : 0u, sh.scan, &total);
            if (match) dst[sh.fill + excl] = c;   // at most n entries: fits wherever src did
            __syncthreads();
            if (threadIdx.x == 0) sh.fill += total;
            __syncthreads();
        }
        if (last) { thr_rel = prefix; break; }
        n = sh.fill;
        const unsigned long long* t = src; src = dst; dst = const_cast<unsigned long long*>(t);
        __threadfence_block();
        __syncthreads();  // this block's own stores to the new src are visible to all its threads
    }
    sum.finish(s_bins);
    if (threadIdx.x == 0) {
        if (good) ctl->thr[s] = thr_rel + dg.sub;
        else atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
    __syncthreads();
    const unsigned long long v = s_bins[threadIdx.x];
    if (v) atomicAdd(reinterpret_cast<unsigned long long*>(&ctl->bins[s][threadIdx.x]), v);
}

// The bucket of the k-th largest entry's first digit is known (b_prefix).  Entries in the buckets
// above it are kept: their values are added up here.  Entries in that bucket (a hundredth of the
// list or so) go to a short list, with SelectDigits::sub taken off, which the last block of the
// side to finish ranks (select_rest_side).  Where the threshold is already final (exact route: the
// gathered list is the kept set) or every candidate is kept (accepted sampled thresholds) the pass
// only adds up.  The block that completes the second side turns the sums into the means and takes
// the side decision.  grid.z = side.
__global__ void __launch_bounds__(kBlock) k_select_filter0(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status) return;
    const int s = blockIdx.z;
    const bool values_mode = P.mode == kModeValues;  // no means there: nothing is added up
    if (s == 1 && values_mode) return;
    __shared__ unsigned long long s_bins[2][256];
    __shared__ uint32_t s_nonzero[2][8];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ uint32_t s_base;
    __shared__ RestShared s_rest;
    s_bins[0][threadIdx.x] = 0ull;
    __syncthreads();
    const BandView view = band_view(P, ctl, s);
    const uint32_t cnt = view.count;
    const SelectDigits dg = select_digits(ctl, s);
    const bool all_kept = ctl->sampled_ok != 0u;
    const bool thr_known = ctl->sel_done[s] != 0u;
    const bool only_sums = all_kept || thr_known;
    const unsigned long long thr = all_kept ? 0ull : ctl->thr[s];
    const uint32_t sel = digit_of(ctl->b_prefix[s], 0, dg.top);
    ExactSum sum;
    sum.start(value_bits_of(s, thr_known ? thr : ((unsigned long long)ctl->lo_key[s] << 32)));
    unsigned long long* __restrict__ dst = P.buf[s][0];
    constexpr int kItems = 4;  // loads in flight per thread
    for (uint32_t base = S.bx * (kBlock * kItems); base < cnt && !(only_sums && values_mode); base += S.nb * (kBlock * kItems)) {
        unsigned long long c[kItems];
        unsigned match = 0u;
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const uint32_t i = base + j * kBlock + threadIdx.x;
            c[j] = (i < cnt) ? view.src[i] : 0ull;
        }
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const bool valid = base + j * kBlock + threadIdx.x < cnt;
            bool keep;
            if (only_sums) {
                keep = valid && c[j] >= thr;
            } else {
                const uint32_t d = digit_of(c[j] - dg.sub, 0, dg.top);
                keep = valid && d > sel;
                match |= (valid && d == sel) ? (1u << j) : 0u;
            }
            if (keep && !values_mode) sum.add(value_bits_of(s, c[j]), s_bins[0]);
        }
        if (only_sums) continue;  // uniform
        uint32_t total;
        const uint32_t excl = block_exclusive_scan<uint32_t>((uint32_t)__popc(match), s_scan, &total);
        if (threadIdx.x == 0) s_base = total ? atomicAdd(&ctl->list_cnt[s], total) : 0u;
        __syncthreads();
        uint32_t pos = s_base + excl;
#pragma unroll
        for (int j = 0; j < kItems; ++j)
            if ((match >> j) & 1u) { if (pos < P.cap) dst[pos] = c[j] - dg.sub; ++pos; }
    }
    sum.finish(s_bins[0]);
    __syncthreads();
    {
        const unsigned long long v = s_bins[0][threadIdx.x];
        if (v) atomicAdd(reinterpret_cast<unsigned long long*>(&ctl->bins[s][threadIdx.x]), v);
    }
    if (!last_block_ticket(&ctl->done[ST_FILTER_S0 + s], S.nb)) return;
    if (!only_sums) {
        s_bins[0][threadIdx.x] = 0ull;
        __syncthreads();
        select_rest_side(P, ctl, s, s_rest, s_bins[0]);
    }
    if (!last_block_ticket(&ctl->done[ST_SUM], values_mode ? 1u : 2u)) return;
    sums_decide_finish(P, S, ctl, s_bins, s_nonzero);
}

// The whole selection and the sums of one side by ONE block, for lists of at most kSmallList
// entries: the entries sit in registers, every level is a shared-memory histogram of the entries
// that still match the prefix, and the walk stops as soon as the selected bucket holds a single
// entry.  Same result as k_select_hist0 + k_select_filter0; the host launches this kernel instead of
// those when every list of the launch is that small.  One block per problem, grid.z = side.
__global__ void __launch_bounds__(kBlock) k_select_small(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status) return;
    const int s = blockIdx.z;
    const bool values_mode = P.mode == kModeValues;
    if (s == 1 && values_mode) return;
    constexpr int kPer = (int)(kSmallList / kBlock);
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    __shared__ unsigned long long s_result;
    __shared__ unsigned long long s_bins[2][256];
    __shared__ uint32_t s_nonzero[2][8];
    __shared__ unsigned long long s_top[kBlock / 32];
    s_bins[0][threadIdx.x] = 0ull;
    const BandView view = band_view(P, ctl, s);
    const uint32_t cnt = view.count, rank = view.rank;
    const SelectDigits dg = select_digits(ctl, s);
    if (cnt > kSmallList) {  // cannot happen: cnt <= cap <= kSmallList is what the host checked
        if (threadIdx.x == 0) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    } else {
        unsigned long long c[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
            c[j] = (i < cnt) ? view.src[i] - dg.sub : 0ull;
        }
        unsigned long long thr_rel = 0ull;  // accepted sampled thresholds: every candidate is kept
        bool good = true;
        if (!ctl->sampled_ok) {
            unsigned long long bits = 0ull;
#pragma unroll
            for (int j = 0; j < kPer; ++j) bits |= c[j];
            const int top = min(dg.top, block_top_bit(bits, s_top));
            good = block_select_registers<kPer>(c, cnt, rank, top, 0, 0ull, s_hist, s_scan, &s_pick, &s_result, &thr_rel);
            if (threadIdx.x == 0) {
                if (good) ctl->thr[s] = thr_rel + dg.sub;
                else atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
        }
        __syncthreads();
        if (good && !values_mode) {
            ExactSum sum;
            sum.start(value_bits_of(s, thr_rel + dg.sub));
#pragma unroll
            for (int j = 0; j < kPer; ++j)
                if ((uint32_t)j * kBlock + threadIdx.x < cnt && c[j] >= thr_rel) sum.add(value_bits_of(s, c[j] + dg.sub), s_bins[0]);
            sum.finish(s_bins[0]);
            __syncthreads();
            const unsigned long long v = s_bins[0][threadIdx.x];
            if (v) atomicAdd(reinterpret_cast<unsigned long long*>(&ctl->bins[s][threadIdx.x]), v);
        }
    }
    if (!last_block_ticket(&ctl->done[ST_SUM], values_mode ? 1u : 2u)) return;
    sums_decide_finish(P, S, ctl, s_bins, s_nonzero);
}

}  // namespace sbc
