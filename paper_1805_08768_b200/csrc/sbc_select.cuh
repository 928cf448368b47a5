// Exact k-th largest composite of each side's candidates (Algorithm 2: exactly k
// kept entries, equal values ordered by index), by MSB-first radix selection
// with 11-bit digits over the 64-bit composites.  Each level keeps only the
// entries that fall in the selected bucket, so the lists shrink quickly.
// Then the exact sums, the two means, the side choice and mu (Algorithm 2).
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// Digit schedule.  The entries being ranked agree in every composite bit above `top`, so the
// digits run from bit `top` downwards, 11 bits each (the last one takes what is left).  For the
// whole key range top = 63 (six levels); for the band between the two sample bounds the keys share
// their leading bits and top is around 50 (five levels, and already the first digit tells the
// entries apart).
__device__ __forceinline__ int digit_bits(int level, int top) { return max(0, min(11, top + 1 - 11 * level)); }
__device__ __forceinline__ int digit_shift(int level, int top) { return max(0, top + 1 - 11 * (level + 1)); }
__device__ __forceinline__ int digit_levels(int top) { return (top + 1 + 10) / 11; }
__device__ __forceinline__ uint32_t digit_of(unsigned long long c, int level, int top) {
    return (uint32_t)(c >> digit_shift(level, top)) & ((1u << digit_bits(level, top)) - 1u);
}
// Highest composite bit in which the entries of the selected part of the list can differ, and
// (through *base) the bits above it, which they all share.
__device__ __forceinline__ int select_top(const Prob& P, const Ctl* ctl, int s, unsigned long long* base) {
    *base = 0ull;
    if (ctl->use_fallback) return 63;  // exact route: the whole key range
    const uint32_t lo = ctl->lo_key[s], hi = ctl->up_key[s] - 1u;  // band keys lie in [lo, hi]
    const uint32_t diff = lo ^ hi;
    const int top = 32 + (diff ? 31 - __clz(diff) : -1);
    *base = top == 63 ? 0ull : (((unsigned long long)lo << 32) & (~0ull << (top + 1)));
    return top;
}

// Rank `rank` (1 = largest) among the cnt <= PER * kBlock composites a block holds in registers
// (slot j of thread t = entry j * kBlock + t), which agree in every digit before `first_level`
// (`prefix` holds those digits).  Radix selection, 11-bit digits from bit `top` down, on
// shared-memory histograms; stops at the first bucket with a single entry.  Returns false if the
// histogram walk failed (inconsistent counts).  All threads call; result identical in all.
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

constexpr int kFinishPer = 8;  // entries per thread a selection kernel's last block finishes by itself
constexpr uint32_t kFinishList = kFinishPer * kBlock;

// Histogram of the top digit over a whole candidate list.  grid.z = side.
__global__ void __launch_bounds__(kBlock) k_select_hist0(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status || ctl->sampled_ok) return;  // sampled thresholds: every candidate is kept (thr = 0)
    const int s = blockIdx.z;
    if (s == 1 && P.mode == kModeValues) return;  // magnitude selection has one side only
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) s_hist[i] = 0u;
    __syncthreads();
    const BandView view = band_view(P, ctl, s);
    const uint32_t cnt = view.count, rank = view.rank;
    unsigned long long shared_bits;
    const int top = select_top(P, ctl, s, &shared_bits);
    constexpr int kItems = 4;  // loads in flight per thread
    for (uint32_t base = S.bx * (kBlock * kItems); base < cnt; base += S.nb * (kBlock * kItems)) {
        unsigned long long c[kItems];
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const uint32_t i = base + j * kBlock + threadIdx.x;
            c[j] = (i < cnt) ? view.src[i] : 0ull;
        }
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const bool valid = base + j * kBlock + threadIdx.x < cnt;
            // whole key range: nearly all entries share the first digit, so one atomic per warp and
            // bin; band: the first digit already spreads them, plain atomics collide rarely
            if (top == 63) warp_hist_add(s_hist, digit_of(c[j], 0, top), valid);
            else if (valid) atomicAdd(&s_hist[digit_of(c[j], 0, top)], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&P.hists->b[0][s][i], v);
    }
    if (last_block_ticket(&ctl->done[ST_BH0_S0 + s], S.nb)) {
        if (cnt <= kFinishList) {  // a short range: this block ranks it alone, the filter kernels return at once
            __shared__ unsigned long long s_result;
            unsigned long long c[kFinishPer], thr = 0ull;
#pragma unroll
            for (int j = 0; j < kFinishPer; ++j) {
                const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
                c[j] = (i < cnt) ? view.src[i] : 0ull;
            }
            const bool good = block_select_registers<kFinishPer>(c, cnt, rank, top, 0, shared_bits, s_hist, s_scan, &s_pick,
                                                                 &s_result, &thr);
            if (threadIdx.x == 0) {
                ctl->thr[s] = thr;
                ctl->sel_done[s] = 1u;
                if (!good) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
            return;
        }
        block_pick_desc(P.hists->b[0][s], kHistBins, false, rank, s_scan, &s_pick);
        if (threadIdx.x == 0) {
            // the k-th largest composite, known down to the end of the first digit
            ctl->b_prefix[s] = shared_bits | ((unsigned long long)s_pick.bin << digit_shift(0, top));
            ctl->b_rank[s] = s_pick.rank;
            if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
        }
    }
}

// The whole selection of one side by ONE block, for lists of at most kSmallList entries (every
// tensor of a ResNet-sized layer at p = 0.001): the entries sit in registers, every level is a
// shared-memory histogram of the entries that still match the prefix, and the walk stops as soon as
// the selected bucket holds a single entry.  Same result as k_select_hist0 + k_select_filter<0..4>;
// the host launches this kernel instead of those when every list of the launch is that small.
// One block per problem, grid.z = side.
__global__ void __launch_bounds__(kBlock) k_select_small(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status || ctl->sampled_ok) return;
    const int s = blockIdx.z;
    if (s == 1 && P.mode == kModeValues) return;
    constexpr int kPer = (int)(kSmallList / kBlock);
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    const BandView view = band_view(P, ctl, s);
    const uint32_t cnt = view.count, rank = view.rank;
    unsigned long long prefix;
    const int top = select_top(P, ctl, s, &prefix);
    if (cnt > kSmallList) {  // cannot happen: cnt <= cap <= kSmallList is what the host checked
        if (threadIdx.x == 0) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
        return;
    }
    unsigned long long c[kPer];
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
        c[j] = (i < cnt) ? view.src[i] : 0ull;
    }
    __shared__ unsigned long long s_result;
    unsigned long long thr = 0ull;
    const bool good = block_select_registers<kPer>(c, cnt, rank, top, 0, prefix, s_hist, s_scan, &s_pick, &s_result, &thr);
    if (threadIdx.x == 0) {
        if (good) ctl->thr[s] = thr;
        else atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
}

// Keep the entries whose level-L digit is the selected one, histogram their
// next digit, and let the last block select at level L+1.  grid.z = side.
template <int LEVEL>
__global__ void __launch_bounds__(kBlock) k_select_filter(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status || ctl->sampled_ok) return;
    const int s = blockIdx.z;
    if (s == 1 && P.mode == kModeValues) return;
    if (ctl->sel_done[s]) return;  // an earlier level's last block finished the selection
    constexpr int kItems = 4;
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ uint32_t s_base;
    __shared__ Pick s_pick;
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) s_hist[i] = 0u;
    __syncthreads();
    const BandView view = band_view(P, ctl, s);
    unsigned long long shared_bits;
    const int top = select_top(P, ctl, s, &shared_bits);
    if (LEVEL + 1 >= digit_levels(top)) return;  // the previous level was the last one
    const uint32_t cnt = LEVEL == 0 ? view.count : ctl->list_cnt[s][LEVEL];
    const unsigned long long* __restrict__ src = P.buf[s][(LEVEL + 1) & 1];  // the previous level's output
    unsigned long long* __restrict__ dst = P.buf[s][LEVEL & 1];
    const uint32_t sel = digit_of(ctl->b_prefix[s], LEVEL, top);
    for (uint32_t base = S.bx * (kBlock * kItems); base < cnt; base += S.nb * (kBlock * kItems)) {
        unsigned long long c[kItems];
        unsigned match = 0u;
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const uint32_t i = base + j * kBlock + threadIdx.x;
            c[j] = (i < cnt) ? (LEVEL == 0 ? view.src[i] : src[i]) : 0ull;
            const bool m = (i < cnt) && digit_of(c[j], LEVEL, top) == sel;
            match |= m ? (1u << j) : 0u;
            warp_hist_add(s_hist, digit_of(c[j], LEVEL + 1, top), m);
        }
        uint32_t total;
        const uint32_t excl = block_exclusive_scan<uint32_t>((uint32_t)__popc(match), s_scan, &total);
        if (threadIdx.x == 0) s_base = total ? atomicAdd(&ctl->list_cnt[s][LEVEL + 1], total) : 0u;
        __syncthreads();
        uint32_t pos = s_base + excl;
#pragma unroll
        for (int j = 0; j < kItems; ++j)
            if ((match >> j) & 1u) { if (pos < P.cap) dst[pos] = c[j]; ++pos; }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&P.hists->b[LEVEL + 1][s][i], v);
    }
    if (last_block_ticket(&ctl->done[ST_BF0_S0 + 2 * LEVEL + s], S.nb)) {
        const uint32_t n_next = min(__ldcg(&ctl->list_cnt[s][LEVEL + 1]), P.cap);  // entries that matched this level's digit
        if (n_next <= kFinishList && LEVEL + 2 < digit_levels(top)) {
            // few entries left and more than one digit to go: this block ranks them alone (they
            // agree in every digit up to this level's), and the later levels return at once
            __shared__ unsigned long long s_result;
            unsigned long long c[kFinishPer], thr = 0ull;
#pragma unroll
            for (int j = 0; j < kFinishPer; ++j) {
                const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
                c[j] = (i < n_next) ? __ldcg(dst + i) : 0ull;
            }
            const bool good = block_select_registers<kFinishPer>(c, n_next, ctl->b_rank[s], top, LEVEL + 1, ctl->b_prefix[s],
                                                                 s_hist, s_scan, &s_pick, &s_result, &thr);
            if (threadIdx.x == 0) {
                ctl->thr[s] = thr;
                ctl->sel_done[s] = 1u;
                if (!good) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
            return;
        }
        block_pick_desc(P.hists->b[LEVEL + 1][s], 1 << digit_bits(LEVEL + 1, top), false,
                        ctl->b_rank[s], s_scan, &s_pick);
        if (threadIdx.x == 0) {
            const unsigned long long prefix =
                ctl->b_prefix[s] | ((unsigned long long)s_pick.bin << digit_shift(LEVEL + 1, top));
            ctl->b_prefix[s] = prefix;
            ctl->b_rank[s] = s_pick.rank;
            if (LEVEL + 2 == digit_levels(top)) ctl->thr[s] = prefix;  // last digit: the k-th largest composite itself
            if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
        }
    }
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

// Sum the kept values of both sides exactly: a value is m * 2^(e-150) with an
// integer m of at most 24 bits, so one 64-bit integer per exponent holds the
// sum of up to 2^39 of them and integer addition makes the result independent
// of the order of the atomics.  On the fast route the entries above the sample's upper bound of the
// threshold were summed while the streaming pass flushed them (pre_bins); only the band is read
// here.  grid.z = side.  The last block turns the bins into mu+ and mu- and takes Algorithm 2's
// side decision.
__global__ void __launch_bounds__(kBlock) k_sums_decide(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    if (ctl->status) return;
    const int s = blockIdx.z;
    const bool values_mode = P.mode == kModeValues;
    if (s == 1 && values_mode) return;
    __shared__ unsigned long long s_bins[2][256];
    s_bins[0][threadIdx.x] = 0ull;
    __syncthreads();
    const BandView view = band_view(P, ctl, s);
    const unsigned long long thr = ctl->thr[s];
    const uint32_t thr_bits = ctl->sampled_ok ? __float_as_uint(s ? ctl->hi_f : ctl->lo_f)
                            : values_mode ? (uint32_t)(thr >> 32) : bits_of_key(side_key(s, (uint32_t)(thr >> 32)));
    // Values within eight binades of the threshold's (nearly all of them) are summed in one
    // register, in units of the lowest of those binades; the rest goes to the shared bins.
    const int bin_a = max((int)((thr_bits >> 23) & 0xffu) - 1, 0);
    long long acc_a = 0;
    auto add = [&](unsigned long long c) {
        const uint32_t bits = bits_of_key(side_key(s, (uint32_t)(c >> 32)));
        const uint32_t e = (bits >> 23) & 0xffu;
        int m = (int)(bits & 0x7fffffu) | (e ? 0x800000 : 0);
        if (bits >> 31) m = -m;
        const int bin = e ? (int)e - 1 : 0;
        const uint32_t up = (uint32_t)(bin - bin_a);
        if (up < 8u) acc_a += (long long)m << up;   // |m| < 2^24: at most 2^31 per entry, 2^62 over 2^31 entries
        else atomicAdd(&s_bins[0][bin], (unsigned long long)(long long)m);
    };
    if (!values_mode) {  // the means exist only for the binarised form
        constexpr int kItems = 8;  // loads in flight per thread
        const uint32_t stride = S.nb * kBlock * kItems;
        for (uint32_t base = S.bx * kBlock * kItems + threadIdx.x; base < view.count; base += stride) {
            unsigned long long c[kItems];
#pragma unroll
            for (int j = 0; j < kItems; ++j) c[j] = (base + j * kBlock < view.count) ? view.src[base + j * kBlock] : 0ull;
#pragma unroll
            for (int j = 0; j < kItems; ++j)
                if (base + j * kBlock < view.count && c[j] >= thr) add(c[j]);
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc_a += __shfl_down_sync(0xffffffffu, acc_a, d);
    if (lane_id() == 0 && acc_a) atomicAdd(&s_bins[0][bin_a], (unsigned long long)acc_a);
    __syncthreads();
    {
        const unsigned long long v = s_bins[0][threadIdx.x];
        if (v) atomicAdd(reinterpret_cast<unsigned long long*>(&ctl->bins[s][threadIdx.x]), v);
    }
    if (last_block_ticket(&ctl->done[ST_SUM], values_mode ? S.nb : S.nb * gridDim.z)) {
        __shared__ uint32_t s_nonzero[2][8];
        // fast route: every entry above the upper bound is kept and was summed when it was flushed
        const bool pre = !ctl->use_fallback && !values_mode;
        const long long b0 = __ldcg(&ctl->bins[0][threadIdx.x]) + (pre ? __ldcg(&ctl->pre_bins[0][threadIdx.x]) : 0ll);
        const long long b1 = __ldcg(&ctl->bins[1][threadIdx.x]) + (pre ? __ldcg(&ctl->pre_bins[1][threadIdx.x]) : 0ll);
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
}

}  // namespace sbc
