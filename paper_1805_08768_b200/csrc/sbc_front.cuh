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
    for (uint32_t base = S.bx * (kBlock * kItems); base < P.m; base += S.nb * (kBlock * kItems)) {
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
constexpr int kWarpChunk = 32 * kPerThread;   // elements per warp per step
constexpr int kStage = 128;                   // staged candidates per warp per side
constexpr int kCollectBlocksPerSM = 3;        // persistent blocks per SM (24 warps, 128 B in flight per thread)

// The streaming pass: A = R + dW written over R (12 bytes per element), two
// float compares per element, and a rare append of (key, index) composites
// through per-warp shared-memory staging so that the global list counters see
// one atomic per hundred or so candidates.  Each thread has eight 16-byte
// loads in flight before it touches any of them.
template <int MODE>
__global__ void __launch_bounds__(kBlock, 4) k_add_collect(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    __shared__ unsigned long long s_stage[kBlock / 32][2][kStage];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const float lo = ctl->lo_f, hi = ctl->hi_f;
    const long long n = P.n;
    const float* __restrict__ U = P.update;
    float* __restrict__ R = P.residual;
    uint32_t wcnt[2] = {0u, 0u};
    bool bad = false;
    const uint32_t cap = P.cap;
    unsigned long long* const cand0 = P.cand[0];
    unsigned long long* const cand1 = P.cand[1];
    const bool vec_ok = P.vec_ok != 0;

    const uint32_t up_key0 = ctl->up_key[0], up_key1 = ctl->up_key[1];

    // Staged candidates of one side go to the list: sure entries (key at or above the upper bound
    // of the threshold) to its front, the others to its back, with ONE atomic for both ranges.
    auto flush = [&](int s) {
        const uint32_t cnt = wcnt[s];
        if (cnt == 0u) return;  // warp-uniform
        __syncwarp();
        const uint32_t up_key = s ? up_key1 : up_key0;
        unsigned long long* const dst = s ? cand1 : cand0;
        uint32_t n_sure = 0u;
        for (uint32_t i0 = 0u; i0 < cnt; i0 += 32u) {
            const uint32_t i = i0 + lane;
            const bool sure = i < cnt && (uint32_t)(s_stage[warp][s][i] >> 32) >= up_key;
            n_sure += (uint32_t)__popc(__ballot_sync(0xffffffffu, sure));
        }
        const uint32_t n_band = cnt - n_sure;
        unsigned long long old = 0ull;
        if (lane == 0)
            old = atomicAdd(&ctl->cand_cnt2[s], (unsigned long long)n_sure | ((unsigned long long)n_band << 32));
        old = __shfl_sync(0xffffffffu, old, 0);
        uint32_t front = (uint32_t)old, back = (uint32_t)(old >> 32);
        // both ranges must stay clear of each other; a list that does not fit is rebuilt by the exact route
        if ((unsigned long long)front + n_sure + (unsigned long long)back + n_band <= (unsigned long long)cap) {
            const unsigned lt = (1u << lane) - 1u;
            for (uint32_t i0 = 0u; i0 < cnt; i0 += 32u) {
                const uint32_t i = i0 + lane;
                const bool valid = i < cnt;
                const unsigned long long c = valid ? s_stage[warp][s][i] : 0ull;
                const bool sure = valid && (uint32_t)(c >> 32) >= up_key;
                const unsigned ms = __ballot_sync(0xffffffffu, sure);
                const unsigned mb = __ballot_sync(0xffffffffu, valid && !sure);
                if (sure) dst[front + (uint32_t)__popc(ms & lt)] = c;
                else if (valid) dst[cap - 1u - (back + (uint32_t)__popc(mb & lt))] = c;
                front += (uint32_t)__popc(ms);
                back += (uint32_t)__popc(mb);
            }
        }
        __syncwarp();
        wcnt[s] = 0u;
    };

    const long long n_chunks = (n + kWarpChunk - 1) / kWarpChunk;
    const long long total_warps = (long long)S.nb * (kBlock / 32);
    for (long long chunk = (long long)S.bx * (kBlock / 32) + warp; chunk < n_chunks;
         chunk += total_warps) {
        const long long base = chunk * kWarpChunk;
        float a[kPerThread];
        unsigned inb = 0u;
        const bool vec_layout = vec_ok && (base + kWarpChunk <= n);  // warp-uniform
        if (vec_layout) {
            // thread owns elements base + (u*32 + lane)*4 + {0..3}, u = 0..kUnroll-1
            const float4* __restrict__ u4 = reinterpret_cast<const float4*>(U + base) + lane;
            float4* __restrict__ r4 = reinterpret_cast<float4*>(R + base) + lane;
            float4 x[kUnroll], r[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) { x[u] = __ldcs(u4 + u * 32); r[u] = __ldcs(r4 + u * 32); }
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
        unsigned pm = 0u, qm = 0u;
#pragma unroll
        for (int j = 0; j < kPerThread; ++j) {
            if (MODE == kModeValues) {
                pm |= (!(fabsf(a[j]) < lo) ? 1u : 0u) << j;   // also true for NaN
            } else {
                pm |= (!(a[j] < lo) ? 1u : 0u) << j;          // also true for NaN
                qm |= (!(a[j] > hi) ? 1u : 0u) << j;
            }
        }
        pm &= inb;
        qm &= inb;
        if (__any_sync(0xffffffffu, (pm | qm) != 0u)) {
            const uint32_t packed = (uint32_t)__popc(pm) | ((uint32_t)__popc(qm) << 16);
            const uint32_t incl = warp_inclusive_scan(packed);
            const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
            const uint32_t excl = incl - packed;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const uint32_t tot_s = s ? (tot >> 16) : (tot & 0xffffu);
                if (tot_s == 0u) continue;
                if (wcnt[s] + tot_s > (uint32_t)kStage) flush(s);
                const unsigned mask = s ? qm : pm;
                if (tot_s > (uint32_t)kStage) {
                    // more candidates in one step than the stage holds (dense ties): element slot by
                    // element slot, at most 32 at a time, each round flushed at once
#pragma unroll 1
                    for (int j = 0; j < kPerThread; ++j) {
                        const bool mine = (mask >> j) & 1u;
                        const unsigned mm = __ballot_sync(0xffffffffu, mine);
                        if (mm == 0u) continue;
                        if (mine) {
                            float aj = a[0];  // a[j] without indexing the register array dynamically
#pragma unroll
                            for (int jj = 1; jj < kPerThread; ++jj) aj = (jj == j) ? a[jj] : aj;
                            const uint32_t bits = __float_as_uint(aj);
                            if ((bits & 0x7f800000u) == 0x7f800000u) bad = true;
                            const long long e = vec_layout ? base + (long long)(((j >> 2) * 32 + lane) * 4 + (j & 3))
                                                           : base + j * 32 + lane;
                            s_stage[warp][s][__popc(mm & ((1u << lane) - 1u))] =
                                make_composite(side_key(s, select_key(MODE, bits)), (uint32_t)e);
                        }
                        wcnt[s] = (uint32_t)__popc(mm);
                        flush(s);
                    }
                    continue;
                }
                uint32_t off = (s ? (excl >> 16) : (excl & 0xffffu)) + wcnt[s];
                wcnt[s] += tot_s;
#pragma unroll
                for (int j = 0; j < kPerThread; ++j) {
                    if ((mask >> j) & 1u) {
                        const uint32_t bits = __float_as_uint(a[j]);
                        if ((bits & 0x7f800000u) == 0x7f800000u) bad = true;
                        const long long e = vec_layout ? base + (long long)(((j >> 2) * 32 + lane) * 4 + (j & 3))
                                                       : base + j * 32 + lane;
                        s_stage[warp][s][off] = make_composite(side_key(s, select_key(MODE, bits)), (uint32_t)e);
                        ++off;
                    }
                }
            }
            __syncwarp();
        }
    }
    flush(0);
    flush(1);
    if (bad) atomicOr(&ctl->status, SBC_STATUS_NONFINITE);

    if (last_block_ticket(&ctl->done[ST_COLLECT], S.nb)) {
        if (threadIdx.x == 0) {
            const unsigned long long t0 = __ldcg(&ctl->cand_cnt2[0]), t1 = __ldcg(&ctl->cand_cnt2[1]);
            const unsigned long long sum0 = (t0 & 0xffffffffull) + (t0 >> 32), sum1 = (t1 & 0xffffffffull) + (t1 >> 32);
            const uint32_t c0 = (uint32_t)min(sum0, 0xffffffffull), c1 = (uint32_t)min(sum1, 0xffffffffull);
            ctl->cand_cnt[0] = c0;
            ctl->cand_cnt[1] = c1;
            ctl->sure_cnt[0] = (uint32_t)t0;
            ctl->sure_cnt[1] = (uint32_t)t1;
            // exact modes: both lists must hold at least the k wanted entries; sampled mode: the
            // lists ARE the kept sets and only have to be non-empty; either way they must fit
            const uint32_t need = P.sampled ? 1u : (uint32_t)P.k;
            const bool ok = c0 >= need && c0 <= P.cap &&
                            (MODE == kModeValues || (c1 >= need && c1 <= P.cap));
            ctl->use_fallback = ok ? 0u : 1u;
            if (!ok) atomicOr(B.any_exact, 1u);
            ctl->sampled_ok = (ok && P.sampled) ? 1u : 0u;
        }
    }
}

}  // namespace sbc
