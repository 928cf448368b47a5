// Front half of sbc_encode: accumulate A = R + dW (Algorithm 1) and gather,
// for each side, a candidate list that is guaranteed to contain the k
// entries Algorithm 2's top_p selects.
//
// Fast route: bound both thresholds from a strided sample, then ONE pass over
// the tensor writes A and appends everything at or beyond the bounds.
// Exact route (taken when the bounds did not bracket k entries, e.g. heavy
// ties or a sample that misrepresents the tensor): three radix-histogram
// passes over A find both k-th keys exactly, a tie-rank pass orders equal
// values by index, and a last pass gathers exactly k entries per side.
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// ---------------------------------------------------------------- sample

// Element behind sample slot i: the sample is made of whole 32-element segments spread evenly over
// the tensor, segment g starting at line floor(g * n_lines / n_segments) (the quotient is a
// fixed-point constant of the problem, at least 1, so the segments are distinct and in range).
__device__ __forceinline__ long long sample_element(const Prob& P, uint32_t i) {
    if ((long long)P.m == P.n) return (long long)i;
    const uint32_t seg = i >> 5, lane = i & 31u;
    return (long long)(((unsigned long long)seg * P.sample_step) >> 20) * 32 + lane;
}

// Level 0: keys of the sampled A values, histogram of their top 11 bits; the
// last block locates the bin of the target rank for each side.
__global__ void __launch_bounds__(kBlock, 4) k_sample0(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick, s_pick_up;
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) s_hist[i] = 0u;
    __syncthreads();
    constexpr int kItems = 8;  // sampled elements per thread and step, all loads issued before any is used
    const float* __restrict__ R = P.residual;
    const float* __restrict__ U = P.update;
    uint32_t* __restrict__ keys = P.sample_keys;
    const uint32_t m = P.m;
    const bool whole = (long long)m == P.n, by_arithmetic = P.sampled == 0;
    const int mode = P.mode;
    const unsigned long long step = P.sample_step;
    for (uint32_t base = S.bx * (kBlock * kItems); base < P.m; base += S.nb * (kBlock * kItems)) {
        if (by_arithmetic && base + kBlock * kItems <= m) {
            // Every slot of the step is a sample slot and its element follows from its number (in
            // range by construction): 32-bit indices, the segment's line by adding up instead of
            // multiplying (slot i + 256 j lies 8 j segments further on), no checks.  This kernel runs
            // at the rate it issues instructions, not at the memory's.
            uint32_t e[kItems];
            const uint32_t i0 = base + threadIdx.x;
            if (whole) {
#pragma unroll
                for (int j = 0; j < kItems; ++j) e[j] = i0 + (uint32_t)j * kBlock;
            } else {
                unsigned long long prod = (unsigned long long)(i0 >> 5) * step;
#pragma unroll
                for (int j = 0; j < kItems; ++j) {
                    e[j] = (uint32_t)(prod >> 20) * 32u + (i0 & 31u);
                    prod += (unsigned long long)(kBlock / 32) * step;
                }
            }
            float r[kItems], u[kItems];
#pragma unroll
            for (int j = 0; j < kItems; ++j) { r[j] = R[e[j]]; u[j] = U[e[j]]; }
#pragma unroll
            for (int j = 0; j < kItems; ++j) {
                const uint32_t key = select_key(mode, __float_as_uint(__fadd_rn(r[j], u[j])));
                keys[i0 + (uint32_t)j * kBlock] = key;
                atomicAdd(&s_hist[key >> 21], 1u);
            }
            continue;
        }
        long long e[kItems];
        float r[kItems], u[kItems];
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const uint32_t i = base + j * kBlock + threadIdx.x;
            e[j] = -1;
            if (i < P.m) {
                e[j] = P.sampled ? (long long)P.sample_idx[i] : sample_element(P, i);
                if (e[j] >= P.n) { e[j] = P.n - 1; atomicOr(&ctl->status, SBC_STATUS_RANGE); }  // bad caller-given position
            }
        }
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            r[j] = e[j] >= 0 ? P.residual[e[j]] : 0.f;
            u[j] = e[j] >= 0 ? P.update[e[j]] : 0.f;
        }
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const bool valid = e[j] >= 0;
            const uint32_t key = select_key(P.mode, __float_as_uint(__fadd_rn(r[j], u[j])));
            if (valid) P.sample_keys[base + j * kBlock + threadIdx.x] = key;
            if (valid) atomicAdd(&s_hist[key >> 21], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&P.hists->s0[i], v);
    }
    if (last_block_ticket(&ctl->done[ST_SAMPLE0], S.nb)) {
        for (int s = 0; s < 2; ++s) {
            // one walk finds the bin of the lower bound's rank and of the upper bound's (if any)
            block_pick_desc(P.hists->s0, kHistBins, s == 1, P.s_target, s_scan, &s_pick, P.s_up, &s_pick_up);
            if (threadIdx.x == 0) {
                ctl->s_bin0[s] = s_pick.bin;
                ctl->s_rank[s] = s_pick.rank;
                if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
                ctl->s_bin0_up[s] = s_pick_up.bin;
                ctl->s_rank_up[s] = s_pick_up.found ? s_pick_up.rank : 0u;  // 0: no upper bound
            }
            __syncthreads();
        }
    }
}

// Level 1: next 11 bits inside the located bins; the last block turns the
// 22-bit prefixes into the two float bounds used by the candidate pass.
__global__ void __launch_bounds__(kBlock, 4) k_sample1(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    __shared__ uint32_t s_hist[2][kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick, s_pick_up;
    const uint32_t bin0[2] = {ctl->s_bin0[0], ctl->s_bin0[1]};
    // the upper bound's top-level bin gets a histogram of its own only where it differs from the
    // lower bound's, in a second walk over the sample keys
    const bool has_up[2] = {ctl->s_rank_up[0] != 0u, ctl->s_rank_up[1] != 0u};
    const uint32_t bin0_up[2] = {ctl->s_bin0_up[0], ctl->s_bin0_up[1]};
    const bool own_up[2] = {has_up[0] && bin0_up[0] != bin0[0], has_up[1] && bin0_up[1] != bin0[1]};
    for (int u = 0; u < ((own_up[0] || own_up[1]) ? 2 : 1); ++u) {
        const uint32_t want0 = u ? bin0_up[0] : bin0[0], want1 = u ? bin0_up[1] : bin0[1];
        const bool on0 = u == 0 || own_up[0], on1 = u == 0 || own_up[1];
        for (int i = threadIdx.x; i < 2 * kHistBins; i += kBlock) (&s_hist[0][0])[i] = 0u;
        __syncthreads();
        constexpr int kItems = 8;  // keys per thread and step, loaded together
        for (uint32_t base = S.bx * (kBlock * kItems); base < P.m; base += S.nb * (kBlock * kItems)) {
            uint32_t keys[kItems];
#pragma unroll
            for (int j = 0; j < kItems; ++j) {
                const uint32_t i = base + j * kBlock + threadIdx.x;
                keys[j] = (i < P.m) ? P.sample_keys[i] : 0u;
            }
#pragma unroll
            for (int j = 0; j < kItems; ++j) {
                const bool valid = base + j * kBlock + threadIdx.x < P.m;
                const uint32_t key = keys[j], sk1 = ~key;
                if (valid && on0 && (key >> 21) == want0) atomicAdd(&s_hist[0][(key >> 10) & 2047u], 1u);
                if (valid && on1 && (sk1 >> 21) == want1) atomicAdd(&s_hist[1][(sk1 >> 10) & 2047u], 1u);
            }
        }
        __syncthreads();
        for (int i = threadIdx.x; i < 2 * kHistBins; i += kBlock) {
            const uint32_t v = (&s_hist[0][0])[i];
            if (v) atomicAdd(&P.hists->s1[i / kHistBins][u][i % kHistBins], v);
        }
        __syncthreads();
    }
    if (last_block_ticket(&ctl->done[ST_SAMPLE1], S.nb)) {
        for (int s = 0; s < 2; ++s) {
            // "sure" = at or above the lower edge of the second-level bin just above the one that
            // holds the upper bound's rank: fewer sample entries than that rank lie there
            const bool want_up = has_up[s] && !P.sampled;
            if (want_up && own_up[s])
                block_pick_desc(P.hists->s1[s][1], kHistBins, false, ctl->s_rank_up[s], s_scan, &s_pick_up);
            // same top-level bin: both ranks come out of one walk
            block_pick_desc(P.hists->s1[s][0], kHistBins, false, ctl->s_rank[s], s_scan, &s_pick,
                            (want_up && !own_up[s]) ? ctl->s_rank_up[s] : 0u, own_up[s] ? nullptr : &s_pick_up);
            if (threadIdx.x == 0) {
                uint32_t up_key = 0xffffffffu;
                if (want_up && s_pick_up.found) {
                    const unsigned long long edge =
                        ((((unsigned long long)bin0_up[s] << 11) | (unsigned long long)s_pick_up.bin) + 1ull) << 10;
                    if (edge <= 0xffffffffull) up_key = (uint32_t)edge;
                }
                ctl->up_key[s] = up_key;
                const uint32_t lower = (bin0[s] << 21) | (s_pick.bin << 10);  // side key, low bits 0
                ctl->lo_key[s] = lower;
                if (P.sampled) {  // one more level follows: the exact order statistic is wanted
                    ctl->s_prefix22[s] = lower >> 10;
                    ctl->s_rank[s] = s_pick.rank;
                } else if (P.mode == kModeValues) {  // the key is the magnitude's bit pattern; no second side
                    if (s == 0) ctl->lo_f = __uint_as_float(lower);
                    else        ctl->hi_f = -INFINITY;
                } else if (s == 0) {
                    ctl->lo_f = __uint_as_float(bits_of_key(lower));
                } else {
                    ctl->hi_f = __uint_as_float(bits_of_key(~lower));
                }
                if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
            __syncthreads();
        }
    }
}

// Level 2 (sampled mode only): the last 10 key bits, which pins the sample's order statistic
// exactly; the two thresholds are then that value itself.
__global__ void __launch_bounds__(kBlock) k_sample2(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    __shared__ uint32_t s_hist[2][1024];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    for (int i = threadIdx.x; i < 2 * 1024; i += kBlock) (&s_hist[0][0])[i] = 0u;
    __syncthreads();
    const uint32_t pre[2] = {ctl->s_prefix22[0], ctl->s_prefix22[1]};
    for (uint32_t base = S.bx * kBlock; base < P.m; base += S.nb * kBlock) {
        const uint32_t i = base + threadIdx.x;
        const bool valid = i < P.m;
        const uint32_t key = valid ? P.sample_keys[i] : 0u;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const uint32_t sk = side_key(s, key);
            warp_hist_add(s_hist[s], sk & 1023u, valid && (sk >> 10) == pre[s]);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * 1024; i += kBlock) {
        const uint32_t v = (&s_hist[0][0])[i];
        if (v) atomicAdd(&P.hists->s2[0][0] + i, v);
    }
    if (last_block_ticket(&ctl->done[ST_SAMPLE2], S.nb)) {
        for (int s = 0; s < 2; ++s) {
            block_pick_desc(P.hists->s2[s], 1024, false, ctl->s_rank[s], s_scan, &s_pick);
            if (threadIdx.x == 0) {
                const uint32_t skey = (pre[s] << 10) | s_pick.bin;
                ctl->lo_key[s] = skey;  // the threshold itself: candidates are exactly the entries at or beyond it
                if (s == 0) ctl->lo_f = __uint_as_float(bits_of_key(skey));
                else        ctl->hi_f = __uint_as_float(bits_of_key(~skey));
                if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------- accumulate + collect

constexpr int kUnroll = 4;                    // float4 loads per array per thread per step
constexpr int kPerThread = 4 * kUnroll;       // elements per thread per step
static_assert(32 * kPerThread == kWarpChunk, "one warp step covers kWarpChunk elements");
constexpr int kStage = 128;                   // staged candidates per warp per side
constexpr int kBandStage = 64;                // staged band entries per warp per side (flushed from 32 on)
constexpr int kCollectBlocksPerSM = 2;        // persistent blocks per SM (16 warps, each with 128 B per thread in flight nearly all the time)

// Shared-memory state of the candidate stages of one block of the streaming pass.
struct StageState {
    // the same for all warps of the block
    uint32_t up_key[2];
    int bin_a[2];                     // lowest of the eight binades the register accumulators cover
    uint32_t cap_w, band_cap, use_runs, pad_;
    unsigned long long* band[2];
    uint32_t* band_cnt[2];
    // per warp and side
    unsigned long long* region[kBlock / 32][2];
    uint32_t fill[kBlock / 32][2];    // candidates already in the region (or dropped, once it overflowed)
    uint32_t bcnt[kBlock / 32][2];    // staged band entries
    uint32_t n_sure[kBlock / 32][2];
    uint32_t flags[kBlock / 32];      // bit 0: a non-finite candidate, bit 1: a region or band list overflowed
    uint2 stage[kBlock / 32][2][kStage];   // staged candidates: x = bit pattern of A_i, y = i
    unsigned long long bstage[kBlock / 32][2][kBandStage];
    unsigned long long bins[2][256];  // exact sums of sure entries outside the accumulators' binades
};

// The `cnt` staged band entries of one side go to the band list (one atomic for all of them).
// All lanes call, with the same `cnt`; the caller sets its count of staged entries back to zero.
__device__ __forceinline__ void flush_band_stage(StageState& st, int warp, int s, uint32_t cnt) {
    if (cnt == 0u) return;  // warp-uniform
    const uint32_t lane = lane_id();
    __syncwarp();
    uint32_t first = 0u;
    if (lane == 0u) first = atomicAdd(st.band_cnt[s], cnt);
    first = __shfl_sync(0xffffffffu, first, 0);
    unsigned long long* const dst = st.band[s];
    if (first <= st.band_cap && cnt <= st.band_cap - first) {
        for (uint32_t i = lane; i < cnt; i += 32u) dst[first + i] = st.bstage[warp][s][i];
    } else if (lane == 0u) {
        st.flags[warp] |= 2u;
    }
    __syncwarp();
}

// The `cnt` staged candidates of side `s` of this warp go to the warp's region, in the order they
// were staged.  A staged candidate is the pair (bit pattern of A_i, i): the key, the composite,
// the non-finite check, the exact sums of the entries at or above the sample's upper bound of the
// threshold ("sure": known to be kept) and the copy of the others ("band") to the band list are
// all done here, by 32 lanes at a time, and not where the candidate is found, by the one lane that
// holds it.  Returns the lane's accumulator of the exact sums, advanced.  One copy of this code
// serves every place that flushes (the streaming kernel is large enough as it is, and its
// instruction fetch showed).  All lanes call.
template <int MODE>
__device__ __noinline__ long long flush_stage(StageState& st, int warp, int s, uint32_t cnt, long long acc) {
    const uint32_t lane = lane_id();
    const unsigned lt = (1u << lane) - 1u;
    __syncwarp();
    const uint32_t up_key = st.up_key[s], cap_w = st.cap_w;
    const int bin_a = st.bin_a[s];
    const bool use_runs = st.use_runs != 0u;
    unsigned long long* const dst = st.region[warp][s];
    const uint32_t fill = st.fill[warp][s];
    const bool room = use_runs && fill <= cap_w && cnt <= cap_w - fill;
    uint32_t bcnt = st.bcnt[warp][s], n_sure = 0u, flags = (use_runs && !room) ? 2u : 0u;
    for (uint32_t i0 = 0u; i0 < cnt; i0 += 32u) {
        const uint32_t i = i0 + lane;
        const bool valid = i < cnt;
        const uint2 e = valid ? st.stage[warp][s][i] : make_uint2(0u, 0u);
        const uint32_t bits = e.x;
        if ((bits & 0x7f800000u) == 0x7f800000u) flags |= 1u;   // padding lanes hold 0
        const uint32_t skey = side_key(s, select_key(MODE, bits));
        const unsigned long long c = make_composite(skey, e.y);
        if (valid && room) dst[fill + i] = c;
        const bool sure = valid && skey >= up_key;
        const unsigned mb = __ballot_sync(0xffffffffu, valid && !sure);
        n_sure += (uint32_t)__popc(__ballot_sync(0xffffffffu, sure));
        if (MODE == kModeBinary && sure) {
            const uint32_t ex = (bits >> 23) & 0xffu;
            int m = (int)(bits & 0x7fffffu) | (ex ? 0x800000 : 0);
            if (bits >> 31) m = -m;
            const int bin = ex ? (int)ex - 1 : 0;
            const uint32_t up = (uint32_t)(bin - bin_a);
            if (up < 8u) acc += (long long)m << up;  // |m| < 2^24: at most 2^31 per entry, 2^62 over 2^31 entries
            else atomicAdd(&st.bins[s][bin], (unsigned long long)(long long)m);
        }
        if (mb) {
            if (valid && !sure) st.bstage[warp][s][bcnt + (uint32_t)__popc(mb & lt)] = c;
            bcnt += (uint32_t)__popc(mb);
            if (bcnt >= 32u) {   // room for another round of 32 is kept at all times
                flush_band_stage(st, warp, s, bcnt);
                bcnt = 0u;
            }
        }
    }
    flags = __reduce_or_sync(0xffffffffu, flags);
    __syncwarp();
    if (lane == 0u) {
        st.fill[warp][s] = fill + cnt;
        st.bcnt[warp][s] = bcnt;
        st.n_sure[warp][s] += n_sure;
        if (flags) st.flags[warp] |= flags;
    }
    __syncwarp();
    return acc;
}

// The streaming pass: A = R + dW written over R (12 bytes per element), two float compares per
// element, and a rare append of (key, index) composites.  Each thread has eight 16-byte loads in
// flight, and the loads of the next step are issued before the step at hand is looked through.
//
// A warp works through whole spans (span_steps consecutive steps of 512 elements), span after
// span in ascending order, and appends each side's candidates, in position order, to a region of
// the ordered list that belongs to this warp alone: no atomics, nothing to wait for.  Where a
// span's entries start in the region and how many they are goes into the span's record, which is
// all a later kernel needs to walk the candidates of the whole tensor in position order.
// Candidates pass through a per-warp shared-memory stage so that the region is written in full
// lines (see flush_stage).
template <int MODE>
__global__ void __launch_bounds__(kBlock, kCollectBlocksPerSM) k_add_collect(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    constexpr int kSides = (MODE == kModeValues) ? 1 : 2;
    __shared__ StageState st;
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const unsigned lt = (1u << lane) - 1u;
    const float lo = ctl->lo_f, hi = ctl->hi_f;
    const long long n = P.n;
    const float* __restrict__ U = P.update;
    float* __restrict__ R = P.residual;
    const bool vec_ok = P.vec_ok != 0;
    const bool use_runs = P.use_runs != 0u;
    const uint32_t cap_w = P.cap_w;
    const uint32_t total_warps = S.nb * (kBlock / 32);
    const uint32_t gw = S.bx * (kBlock / 32) + (uint32_t)warp;   // < P.main_warps: the grid is sized from the same plan
    if (threadIdx.x < 2) {
        const int s = threadIdx.x;
        const uint32_t up_key = ctl->up_key[s];
        st.up_key[s] = up_key;
        // the exact sums of the sure entries: values within eight binades of the upper bound's are added
        // in one register per lane and side (units of the lowest of those binades), the rest in shared bins
        const uint32_t ub = bits_of_key(side_key(s, up_key));
        st.bin_a[s] = max((int)((ub >> 23) & 0xffu) - 1, 0);
        st.band[s] = P.band[s];
        st.band_cnt[s] = &ctl->band_cnt[s];
        if (s == 0) { st.cap_w = cap_w; st.band_cap = P.cap; st.use_runs = P.use_runs; }
    }
    if (lane < 2) {
        st.region[warp][lane] = P.list[lane] + (size_t)gw * cap_w;
        st.fill[warp][lane] = 0u;
        st.bcnt[warp][lane] = 0u;
        st.n_sure[warp][lane] = 0u;
        if (lane == 0) st.flags[warp] = 0u;
    }
    st.bins[0][threadIdx.x] = 0ull;
    st.bins[1][threadIdx.x] = 0ull;
    __syncthreads();
    long long acc[2] = {0, 0};
    uint32_t wcnt[2] = {0u, 0u};   // staged, not yet in the region
    auto flush = [&](int s) {
        if (wcnt[s]) acc[s] = flush_stage<MODE>(st, warp, s, wcnt[s], acc[s]);
        wcnt[s] = 0u;
    };

    const long long n_chunks = (n + kWarpChunk - 1) / kWarpChunk;
    const uint32_t span_steps = P.span_steps, n_spans = P.n_spans;   // span_steps is a power of two
    const uint32_t step_shift = 31u - (uint32_t)__clz((int)span_steps);
    // This warp's spans are gw, gw + total_warps, ...; its steps are numbered through: step t is
    // step t % span_steps of its (t / span_steps)-th span.
    const uint32_t my_spans = gw < n_spans ? (n_spans - gw + total_warps - 1u) / total_warps : 0u;
    const uint32_t my_steps = my_spans << step_shift;
    auto chunk_at = [&](uint32_t t) -> long long {   // chunk of step t; -1 past the end of the tensor
        if (t >= my_steps) return -1ll;
        const long long c = ((long long)gw + (long long)(t >> step_shift) * total_warps) * span_steps + (t & (span_steps - 1u));
        return c < n_chunks ? c : -1ll;
    };
    // The loads of a step are issued while the step before it is still being looked through for
    // candidates (the registers they land in are free by then), so that a warp has loads in flight
    // nearly all the time.  Only whole, aligned chunks are loaded ahead.
    float4 x[kUnroll], r[kUnroll];
    auto load_ahead = [&](long long chunk) -> bool {
        if (chunk < 0 || !vec_ok || (chunk + 1) * kWarpChunk > n) return false;  // warp-uniform
        const float4* __restrict__ u4 = reinterpret_cast<const float4*>(U + chunk * kWarpChunk) + lane;
        const float4* __restrict__ r4 = reinterpret_cast<const float4*>(R + chunk * kWarpChunk) + lane;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) { x[u] = __ldcs(u4 + u * 32); r[u] = __ldcs(r4 + u * 32); }
        return true;
    };
    bool vec_layout = load_ahead(chunk_at(0u));
    uint32_t span_first[2] = {0u, 0u};
    for (uint32_t t = 0u; t < my_steps; ++t) {
        const uint32_t span = gw + (t >> step_shift) * total_warps;
        if ((t & (span_steps - 1u)) == 0u) {
            span_first[0] = st.fill[warp][0] + wcnt[0];
            span_first[1] = st.fill[warp][1] + wcnt[1];
        }
        const long long chunk = chunk_at(t);
        if (chunk >= 0) {
            const long long base = chunk * kWarpChunk;
            float a[kPerThread];
            unsigned inb = 0u;
            if (vec_layout) {
                // thread owns elements base + (u*32 + lane)*4 + {0..3}, u = 0..kUnroll-1
                float4* __restrict__ r4 = reinterpret_cast<float4*>(R + base) + lane;
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    float4 y;
                    y.x = __fadd_rn(r[u].x, x[u].x); y.y = __fadd_rn(r[u].y, x[u].y);
                    y.z = __fadd_rn(r[u].z, x[u].z); y.w = __fadd_rn(r[u].w, x[u].w);
                    __stcs(r4 + u * 32, y);
                    a[4 * u + 0] = y.x; a[4 * u + 1] = y.y; a[4 * u + 2] = y.z; a[4 * u + 3] = y.w;
                }
                inb = (1u << kPerThread) - 1u;
            } else {
                // ragged tail or unaligned pointers: thread owns elements base + j*32 + lane
#pragma unroll
                for (int j = 0; j < kPerThread; ++j) {
                    const long long e = base + j * 32 + lane;
                    a[j] = 0.f;
                    if (e < n) {
                        a[j] = __fadd_rn(R[e], U[e]);
                        R[e] = a[j];
                        inb |= 1u << j;
                    }
                }
            }
            const bool this_vec = vec_layout;
            vec_layout = load_ahead(chunk_at(t + 1u));
            unsigned mask[2] = {0u, 0u};
#pragma unroll
            for (int j = 0; j < kPerThread; ++j) {
                if (MODE == kModeValues) {
                    mask[0] |= (!(fabsf(a[j]) < lo) ? 1u : 0u) << j;   // also true for NaN
                } else {
                    mask[0] |= (!(a[j] < lo) ? 1u : 0u) << j;          // also true for NaN
                    mask[1] |= (!(a[j] > hi) ? 1u : 0u) << j;
                }
            }
            mask[0] &= inb;
            mask[1] &= inb;
            if (__any_sync(0xffffffffu, (mask[0] | mask[1]) != 0u)) {
            if (this_vec && __all_sync(0xffffffffu, ((mask[0] & (mask[0] - 1u)) | (mask[1] & (mask[1] - 1u))) == 0u)) {
                // No lane holds more than one candidate per side (nine steps in ten at p = 0.01):
                // position order (row u, lane) comes from one ballot per row, no scan.
                const uint32_t idx0 = (uint32_t)base + (uint32_t)lane * 4u;
#pragma unroll
                for (int s = 0; s < kSides; ++s) {
                    const uint32_t m = mask[s];
                    const unsigned b_any = __ballot_sync(0xffffffffu, m != 0u);
                    if (b_any == 0u) continue;  // warp-uniform
                    const unsigned b0 = __ballot_sync(0xffffffffu, (m & 0x000fu) != 0u);
                    const unsigned b1 = __ballot_sync(0xffffffffu, (m & 0x00f0u) != 0u);
                    const unsigned b2 = __ballot_sync(0xffffffffu, (m & 0x0f00u) != 0u);
                    const unsigned b3 = b_any & ~(b0 | b1 | b2);
                    const uint32_t tot_s = (uint32_t)__popc(b_any);
                    if (wcnt[s] + tot_s > (uint32_t)kStage) flush(s);
                    const uint32_t j = (uint32_t)__ffs((int)m) - 1u;   // the lane's candidate, if it has one
                    const bool t0 = j & 1u, t1 = j & 2u, t2 = j & 4u, t3 = j & 8u;
                    const float x0 = t0 ? a[1] : a[0], x1 = t0 ? a[3] : a[2], x2 = t0 ? a[5] : a[4], x3 = t0 ? a[7] : a[6];
                    const float x4 = t0 ? a[9] : a[8], x5 = t0 ? a[11] : a[10], x6 = t0 ? a[13] : a[12], x7 = t0 ? a[15] : a[14];
                    const float y0 = t1 ? x1 : x0, y1 = t1 ? x3 : x2, y2 = t1 ? x5 : x4, y3 = t1 ? x7 : x6;
                    const float z0 = t2 ? y1 : y0, z1 = t2 ? y3 : y2;
                    const float v = t3 ? z1 : z0;
                    const unsigned row = t3 ? (t2 ? b3 : b2) : (t2 ? b1 : b0);
                    const uint32_t before = (t3 || t2 ? (uint32_t)__popc(b0) : 0u) + (t3 ? (uint32_t)__popc(b1) : 0u) +
                                            (t3 && t2 ? (uint32_t)__popc(b2) : 0u) + (uint32_t)__popc(row & lt);
                    if (m) st.stage[warp][s][wcnt[s] + before] = make_uint2(__float_as_uint(v), idx0 + (j >> 2) * 128u + (j & 3u));
                    wcnt[s] += tot_s;
                }
            } else if (this_vec) {
                // Position order inside the step is (u, lane, element of the float4).  Per side and u,
                // the number of candidates of every lane goes into one byte of a 64-bit word; one warp
                // scan gives every (side, u, lane) its slot.
                unsigned long long packed = 0ull;
#pragma unroll
                for (int s = 0; s < kSides; ++s) {
                    // bits set per nibble of the 16-bit mask, each count then moved into a byte of its own
                    uint32_t c = mask[s];
                    c = c - ((c >> 1) & 0x5555u);
                    c = (c & 0x3333u) + ((c >> 2) & 0x3333u);
                    c = (c | (c << 8)) & 0x00ff00ffu;
                    c = (c | (c << 4)) & 0x0f0f0f0fu;
                    packed |= (unsigned long long)c << (32 * s);
                }
                const unsigned long long incl = warp_inclusive_scan(packed);   // at most 128 per byte: no carries
                const unsigned long long tot = __shfl_sync(0xffffffffu, incl, 31);
                const unsigned long long excl = incl - packed;
                const uint32_t idx0 = (uint32_t)base + (uint32_t)lane * 4u;
#pragma unroll
                for (int s = 0; s < kSides; ++s) {
                    const uint32_t tot4 = (uint32_t)(tot >> (32 * s)), excl4 = (uint32_t)(excl >> (32 * s));
                    const uint32_t tot_s = __dp4a(tot4, 0x01010101u, 0u);   // the four bytes added up
                    if (tot_s == 0u) continue;  // warp-uniform
                    uint2* const dst = &st.stage[warp][s][0];
                    if (tot_s > (uint32_t)kStage) {
                        // more candidates in one step than the stage holds (dense ties): row by row
                        // (a row is one u, at most 128 candidates), the stage flushed in between
#pragma unroll
                        for (int u = 0; u < kUnroll; ++u) {
                            const uint32_t tu = (tot4 >> (8 * u)) & 0xffu;
                            if (wcnt[s] + tu > (uint32_t)kStage) flush(s);
                            uint32_t slot = wcnt[s] + ((excl4 >> (8 * u)) & 0xffu);
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                if ((mask[s] >> (4 * u + q)) & 1u) dst[slot] = make_uint2(__float_as_uint(a[4 * u + q]), idx0 + (uint32_t)(u * 128 + q));
                                slot += (mask[s] >> (4 * u + q)) & 1u;
                            }
                            wcnt[s] += tu;
                        }
                        continue;
                    }
                    if (wcnt[s] + tot_s > (uint32_t)kStage) flush(s);
                    // rows (one u each) in which no lane holds a candidate are skipped by the whole warp
                    const unsigned any_lane = __reduce_or_sync(0xffffffffu, mask[s]);
                    uint32_t row = wcnt[s];
#pragma unroll
                    for (int u = 0; u < kUnroll; ++u) {
                        if (((any_lane >> (4 * u)) & 0xfu) == 0u) continue;  // warp-uniform
                        const uint32_t nib = (mask[s] >> (4 * u)) & 0xfu;
                        uint32_t slot = row + ((excl4 >> (8 * u)) & 0xffu);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {   // no branches: four predicated stores
                            if ((nib >> q) & 1u) dst[slot] = make_uint2(__float_as_uint(a[4 * u + q]), idx0 + (uint32_t)(u * 128 + q));
                            slot += (nib >> q) & 1u;
                        }
                        row += (tot4 >> (8 * u)) & 0xffu;
                    }
                    wcnt[s] += tot_s;
                }
            } else {
                // position order is (j, lane): one ballot per element slot
#pragma unroll
                for (int s = 0; s < kSides; ++s) {
#pragma unroll 1
                    for (int j = 0; j < kPerThread; ++j) {
                        const bool mine = (mask[s] >> j) & 1u;
                        const unsigned mm = __ballot_sync(0xffffffffu, mine);
                        if (mm == 0u) continue;
                        const uint32_t tj = (uint32_t)__popc(mm);
                        if (wcnt[s] + tj > (uint32_t)kStage) flush(s);
                        if (mine) {
                            float aj = a[0];  // a[j] without indexing the register array dynamically
#pragma unroll
                            for (int jj = 1; jj < kPerThread; ++jj) aj = (jj == j) ? a[jj] : aj;
                            st.stage[warp][s][wcnt[s] + (uint32_t)__popc(mm & lt)] =
                                make_uint2(__float_as_uint(aj), (uint32_t)(base + j * 32 + lane));
                        }
                        wcnt[s] += tj;
                    }
                }
            }
            __syncwarp();
            }
        }
        // end of a span: its record says where its candidates sit (staged entries keep their order
        // and follow the flushed ones)
        if ((t & (span_steps - 1u)) == span_steps - 1u && use_runs && lane < kSides)
            P.span_rec[lane][span] = make_uint2(gw * cap_w + (lane ? span_first[1] : span_first[0]),
                                                st.fill[warp][lane] + (lane ? wcnt[1] - span_first[1] : wcnt[0] - span_first[0]));
    }
#pragma unroll
    for (int s = 0; s < kSides; ++s) {
        flush(s);
        flush_band_stage(st, warp, s, st.bcnt[warp][s]);
    }
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kSides; ++s) {
            if (st.fill[warp][s]) atomicAdd(&ctl->cand_cnt[s], st.fill[warp][s]);
            if (st.n_sure[warp][s]) atomicAdd(&ctl->sure_cnt[s], st.n_sure[warp][s]);
        }
        if (st.flags[warp] & 1u) atomicOr(&ctl->status, SBC_STATUS_NONFINITE);
        if (st.flags[warp] & 2u) atomicOr(&ctl->overflow, 1u);
    }
    if (MODE == kModeBinary) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            long long v = acc[s];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(0xffffffffu, v, d);
            if (lane == 0 && v) atomicAdd(&st.bins[s][st.bin_a[s]], (unsigned long long)v);
        }
        __syncthreads();
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const unsigned long long v = st.bins[s][threadIdx.x];
            if (v) atomicAdd(reinterpret_cast<unsigned long long*>(&ctl->pre_bins[s][threadIdx.x]), v);
        }
    }

    if (last_block_ticket(&ctl->done[ST_COLLECT], S.nb)) {
        if (threadIdx.x == 0) {
            const uint32_t c0 = __ldcg(&ctl->cand_cnt[0]), c1 = __ldcg(&ctl->cand_cnt[1]);
            const uint32_t u0 = __ldcg(&ctl->sure_cnt[0]), u1 = __ldcg(&ctl->sure_cnt[1]);
            const bool spilled = __ldcg(&ctl->overflow) != 0u;
            // exact modes: both lists must hold at least the k wanted entries, of which fewer than
            // k may lie above the upper bound (else the bound was too low and says nothing);
            // sampled mode: the lists ARE the kept sets and only have to be non-empty; either way
            // they must fit
            const uint32_t need = P.sampled ? 1u : (uint32_t)P.k;
            const bool counts_ok = c0 >= need && c0 <= P.cap && (MODE == kModeValues || (c1 >= need && c1 <= P.cap));
            const bool bounds_ok = P.sampled || (u0 < (uint32_t)P.k && (MODE == kModeValues || u1 < (uint32_t)P.k));
            const bool ok = counts_ok && bounds_ok && !spilled;
            ctl->use_fallback = ok ? 0u : 1u;
            if (!ok) {
                atomicOr(B.any_exact, 1u);
                // The exact route rebuilds the lists.  If only the placement failed (a warp's region
                // too small for unevenly spread candidates) the bounds still hold, and so does everything
                // that does not depend on where a candidate was put: the band list (it cannot overflow
                // while the counts fit) and the counts and sums of the sure entries.  Only the ordered
                // lists are gathered again, this time with space reserved tile by tile, and the fast
                // route's kernels go on from there.
                if (counts_ok && bounds_ok) {
                    ctl->x_known = 1u;
                    ctl->x_thr[0] = ctl->lo_key[0];
                    ctl->x_thr[1] = ctl->lo_key[1];
                }
                else {
                    ctl->sure_cnt[0] = 0u;
                    ctl->sure_cnt[1] = 0u;
                }
                ctl->cand_cnt[0] = 0u;   // counted again as the lists are rebuilt
                ctl->cand_cnt[1] = 0u;
            }
            ctl->sampled_ok = (counts_ok && P.sampled) ? 1u : 0u;
        }
    }
}

}  // namespace sbc
