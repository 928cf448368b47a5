// Exact-select route over the whole accumulated tensor A (Algorithm 2's top_p
// by radix selection on the fp32 bit patterns).  Runs only when the candidate
// pass could not bracket both thresholds (or could not place its candidates);
// otherwise its one kernel returns at once.  Result: exactly k composites per
// side in the candidate lists (or, when only the gathering is redone, every
// candidate at or beyond the sample's bounds).
//
// The route is six steps with a grid-wide dependency between them (three radix
// levels, tie counts, their scan, the gathering).  As six kernels they cost
// every encode six launches just to find out that they are not needed, so they
// are ONE cooperative kernel: all its blocks are resident at the same time, and
// between two steps they meet at a barrier in global memory (grid_barrier, a
// bounded wait: if it ever gives up, the problems that needed the route get
// SBC_STATUS_TIMEOUT and the kernel returns).
#pragma once
#include "sbc_common.cuh"
#include "../../include/sbc.h"

namespace sbc {

// Whether a problem takes the route.  Decided by the streaming pass and not changed before the
// route's last step (one block per problem, which is then done with it), so that every block of
// the route's kernel sees the same answer in every step that works on the problem.
__device__ __forceinline__ bool exact_route_active(const Ctl* ctl) { return ctl->use_fallback != 0u; }

// Shared memory of the exact route's kernel, used by one step at a time.
struct ExactShared {
    uint32_t hist[2][kHistBins];
    uint32_t scan[kBlock / 32 + 1];
    Pick pick;
    uint32_t warp_ties[2][kBlock / 32];
    uint32_t warp_emit[2][kBlock / 32 + 1];
    uint32_t base[2];
};

// One radix level (0: key bits 31..21, 1: bits 20..10, 2: bits 9..0) for both
// sides; block `bx` of `nb`; the last block to finish extends the two prefixes.
template <int LEVEL>
__device__ __forceinline__ void exact_hist_step(const Prob& P, uint32_t bx, uint32_t nb, ExactShared& sh) {
    Ctl* ctl = P.ctl;
    struct { uint32_t bx, nb; } S = {bx, nb};
    uint32_t (&s_hist)[2][kHistBins] = sh.hist;
    uint32_t* const s_scan = sh.scan;
    Pick& s_pick = sh.pick;
    constexpr int kBins = (LEVEL == 2) ? 1024 : kHistBins;
    __syncthreads();  // the shared buffers may still be in use by the step before
    for (int i = threadIdx.x; i < 2 * kHistBins; i += kBlock) (&s_hist[0][0])[i] = 0u;
    __syncthreads();
    const uint32_t pre[2] = {__ldcg(&ctl->x_prefix[0]), __ldcg(&ctl->x_prefix[1])};  // written by another block of this kernel
    const float* __restrict__ A = P.residual;
    const long long stride = (long long)S.nb * kBlock;
    for (long long base = (long long)S.bx * kBlock; base < P.n; base += stride) {
        const long long i = base + threadIdx.x;
        const bool valid = i < P.n;
        const uint32_t key = valid ? select_key(P.mode, __float_as_uint(A[i])) : 0u;
        if (LEVEL == 0) {
            warp_hist_add(s_hist[0], key >> 21, valid);
        } else {
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const uint32_t sk = side_key(s, key);
                if (LEVEL == 1)
                    warp_hist_add(s_hist[s], (sk >> 10) & 2047u, valid && (sk >> 21) == pre[s]);
                else
                    warp_hist_add(s_hist[s], sk & 1023u, valid && (sk >> 10) == pre[s]);
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistBins; i += kBlock) {
        if (LEVEL == 0) {
            const uint32_t v = s_hist[0][i];
            if (v) {
                atomicAdd(&P.hists->x[0][0][i], v);
                atomicAdd(&P.hists->x[0][1][kHistBins - 1 - i], v);  // same counts, complemented key
            }
        } else {
            for (int s = 0; s < 2; ++s) {
                const uint32_t v = s_hist[s][i];
                if (v) atomicAdd(&P.hists->x[LEVEL][s][i], v);
            }
        }
    }
    if (last_block_ticket(&ctl->done[ST_XH0 + LEVEL], S.nb)) {
        for (int s = 0; s < 2; ++s) {
            const uint32_t rank = (LEVEL == 0) ? (uint32_t)P.k : __ldcg(&ctl->x_rank[s]);
            block_pick_desc(P.hists->x[LEVEL][s], kBins, false, rank, s_scan, &s_pick);
            if (threadIdx.x == 0) {
                const uint32_t prefix =
                    (LEVEL == 0) ? s_pick.bin : ((pre[s] << (LEVEL == 1 ? 11 : 10)) | s_pick.bin);
                ctl->x_prefix[s] = prefix;
                ctl->x_rank[s] = s_pick.rank;
                if (LEVEL == 2) {
                    ctl->x_thr[s] = prefix;             // side key of the k-th entry
                    ctl->x_ties_take[s] = s_pick.rank;  // equal entries to keep (lowest indices)
                    ctl->x_ties_have[s] = s_pick.count;
                    ctl->cand_cnt[s] = 0u;              // the lists are rebuilt from scratch
                }
                if (!s_pick.found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            }
            __syncthreads();
        }
    }
}

__device__ __forceinline__ bool tie_ranks_needed(const Ctl* ctl, int s) {
    return __ldcg(&ctl->x_ties_take[s]) < __ldcg(&ctl->x_ties_have[s]);
}

// Entries equal to the threshold, per tile of kXTile elements.
__device__ __forceinline__ void exact_tiecount_step(const Prob& P, uint32_t bx, uint32_t nb, ExactShared& sh) {
    Ctl* ctl = P.ctl;
    struct { uint32_t bx, nb; } S = {bx, nb};
    if (!tie_ranks_needed(ctl, 0) && !tie_ranks_needed(ctl, 1)) return;
    uint32_t* const s_scan = sh.scan;
    const uint32_t thr[2] = {__ldcg(&ctl->x_thr[0]), __ldcg(&ctl->x_thr[1])};
    const float* __restrict__ A = P.residual;
    for (uint32_t tile = S.bx; tile < P.n_xtiles; tile += S.nb) {
        uint32_t c = 0u;  // side 0 in the low half, side 1 in the high half
        for (int j = 0; j < kXTile / kBlock; ++j) {
            const long long i = (long long)tile * kXTile + j * kBlock + threadIdx.x;
            if (i < P.n) {
                const uint32_t key = select_key(P.mode, __float_as_uint(A[i]));
                c += (key == thr[0]) ? 1u : 0u;
                c += (~key == thr[1]) ? 0x10000u : 0u;
            }
        }
        uint32_t total;
        block_exclusive_scan<uint32_t>(c, s_scan, &total);
        if (threadIdx.x == 0) {
            P.x_tile_cnt[0][tile] = total & 0xffffu;
            P.x_tile_cnt[1][tile] = total >> 16;
        }
    }
}

// In-place exclusive scan of the per-tile tie counts (one block).
__device__ __forceinline__ void exact_tiescan_step(const Prob& P, ExactShared& sh) {
    Ctl* ctl = P.ctl;
    if (!tie_ranks_needed(ctl, 0) && !tie_ranks_needed(ctl, 1)) return;
    uint32_t* const s_scan = sh.scan;
    const uint32_t per = (P.n_xtiles + kBlock - 1) / kBlock;
    for (int s = 0; s < 2; ++s) {
        uint32_t* cnt = P.x_tile_cnt[s];
        const uint32_t lo = threadIdx.x * per;
        const uint32_t hi = min(lo + per, P.n_xtiles);
        uint32_t sum = 0u;
        for (uint32_t t = lo; t < hi; ++t) sum += __ldcg(cnt + t);
        uint32_t run = block_exclusive_scan<uint32_t>(sum, s_scan, nullptr);
        for (uint32_t t = lo; t < hi; ++t) {
            const uint32_t v = __ldcg(cnt + t);
            cnt[t] = run;
            run += v;
        }
        __syncthreads();
    }
}

// Gather the composites of each side: everything strictly beyond the threshold plus the
// lowest-index ties (exactly k when the route found the thresholds itself; everything at or beyond
// the known bounds when only the gathering is redone).  A block takes a tile of kXTile elements,
// its warps 512 consecutive elements each, walked 32 at a time, so the rank of a tie is
// (ties in earlier tiles) + (earlier warps) + (earlier steps) + (lower lanes), and the entries of a
// tile leave in position order: space for them is reserved with one atomic per tile and side, and
// every span of the tile gets its record (offset, count) as in the streaming pass.
__device__ __forceinline__ void exact_collect_step(const Prob& P, uint32_t bx, uint32_t nb, ExactShared& sh) {
    Ctl* ctl = P.ctl;
    struct { uint32_t bx, nb; } S = {bx, nb};
    constexpr int kSteps = kXTile / kBlock;  // 16 steps of 32 lanes per warp
    constexpr int kWarps = kBlock / 32;
    static_assert(kXTile / kWarps == kWarpChunk, "a warp of this kernel covers one step of the streaming pass");
    uint32_t (&s_warp_ties)[2][kWarps] = sh.warp_ties;
    uint32_t (&s_warp_emit)[2][kWarps + 1] = sh.warp_emit;
    uint32_t (&s_base)[2] = sh.base;
    __syncthreads();  // the shared buffers may still be in use by the step before
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const unsigned lt = (1u << lane) - 1u;
    const uint32_t thr[2] = {__ldcg(&ctl->x_thr[0]), __ldcg(&ctl->x_thr[1])};
    const uint32_t take[2] = {__ldcg(&ctl->x_ties_take[0]), __ldcg(&ctl->x_ties_take[1])};
    const bool ranked[2] = {tie_ranks_needed(ctl, 0), tie_ranks_needed(ctl, 1)};
    const bool one_sided = P.mode == kModeValues;  // magnitude selection has no second side
    const float* __restrict__ A = P.residual;
    const uint32_t span_steps = P.span_steps;
    unsigned long long least[2] = {~0ull, ~0ull};  // smallest composite this thread gathered
    for (uint32_t tile = S.bx; tile < P.n_xtiles; tile += S.nb) {
        const long long wbase = (long long)tile * kXTile + (long long)warp * kWarpChunk;
        uint32_t key[kSteps];
        unsigned inb = 0u;
#pragma unroll
        for (int j = 0; j < kSteps; ++j) {
            const long long i = wbase + j * 32 + lane;
            key[j] = 0u;
            if (i < P.n) {
                key[j] = select_key(P.mode, __float_as_uint(A[i]));
                inb |= 1u << j;
            }
        }
        unsigned emit[2] = {0u, 0u};
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (s == 1 && one_sided) continue;
            if (!ranked[s]) {
#pragma unroll
                for (int j = 0; j < kSteps; ++j)
                    emit[s] |= ((inb >> j) & 1u) && (side_key(s, key[j]) >= thr[s]) ? (1u << j) : 0u;
            } else {
                uint32_t wt = 0u;
#pragma unroll
                for (int j = 0; j < kSteps; ++j)
                    wt += __popc(__ballot_sync(0xffffffffu,
                                               ((inb >> j) & 1u) && side_key(s, key[j]) == thr[s]));
                if (lane == 0) s_warp_ties[s][warp] = wt;
            }
        }
        __syncthreads();
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (!ranked[s] || (s == 1 && one_sided)) continue;
            uint32_t run = __ldcg(&P.x_tile_cnt[s][tile]);
            for (int w = 0; w < warp; ++w) run += s_warp_ties[s][w];
#pragma unroll
            for (int j = 0; j < kSteps; ++j) {
                const bool in = (inb >> j) & 1u;
                const uint32_t sk = side_key(s, key[j]);
                const unsigned tb = __ballot_sync(0xffffffffu, in && sk == thr[s]);
                const uint32_t my_rank = run + __popc(tb & lt);
                const bool keep = in && (sk > thr[s] || (sk == thr[s] && my_rank < take[s]));
                emit[s] |= keep ? (1u << j) : 0u;
                run += __popc(tb);
            }
        }
        // entries per warp and side; position order inside a warp is (step, lane)
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            uint32_t wt = 0u;
#pragma unroll
            for (int j = 0; j < kSteps; ++j) wt += __popc(__ballot_sync(0xffffffffu, (emit[s] >> j) & 1u));
            if (lane == 0) s_warp_emit[s][warp] = wt;
        }
        __syncthreads();
        if (threadIdx.x < 2) {  // one thread per side: exclusive scan over the warps, then the tile's reservation
            const int s = threadIdx.x;
            uint32_t run = 0u;
            for (int w = 0; w < kWarps; ++w) { const uint32_t v = s_warp_emit[s][w]; s_warp_emit[s][w] = run; run += v; }
            s_warp_emit[s][kWarps] = run;
            s_base[s] = run ? atomicAdd(&ctl->cand_cnt[s], run) : 0u;
        }
        __syncthreads();
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (s == 1 && one_sided) continue;
            const uint32_t first = s_base[s] + s_warp_emit[s][warp];
            uint32_t pos = first;
#pragma unroll
            for (int j = 0; j < kSteps; ++j) {
                const bool mine = (emit[s] >> j) & 1u;
                const unsigned mm = __ballot_sync(0xffffffffu, mine);
                if (mine) {
                    const uint32_t slot = pos + (uint32_t)__popc(mm & lt);
                    const unsigned long long c = make_composite(side_key(s, key[j]), (uint32_t)(wbase + j * 32 + lane));
                    if (slot < P.list_cap) P.list[s][slot] = c;
                    least[s] = min(least[s], c);
                }
                pos += (uint32_t)__popc(mm);
            }
            // the span that starts with this warp's 512 elements: its warps' entries follow one another
            if (P.use_runs && lane == 0 && (uint32_t)warp % span_steps == 0u) {
                const uint32_t span = (tile * (uint32_t)kWarps + (uint32_t)warp) / span_steps;
                const uint32_t end_warp = min((uint32_t)warp + span_steps, (uint32_t)kWarps);
                if (span < P.n_spans)
                    P.span_rec[s][span] = make_uint2(first, s_base[s] + s_warp_emit[s][end_warp] - first);
            }
        }
        __syncthreads();  // the shared arrays are reused by the next tile
    }
    // the k-th largest composite of a side is the smallest one gathered (when exactly k were)
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        unsigned long long v = ~least[s];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v = max(v, __shfl_down_sync(0xffffffffu, v, d));
        if (lane == 0 && v) atomicMax(&ctl->x_min_inv[s], v);
    }
}

// What the kernels after the route go by.  Thresholds found here: the lists hold exactly the k
// kept entries of each side, so the selection has nothing to do.  Gathering redone: the fast
// route's lists are whole again, its kernels take over.  One thread of one block per problem.
__device__ __forceinline__ void exact_final_step(const Prob& P) {
    Ctl* ctl = P.ctl;
    if (threadIdx.x != 0) return;
    if (__ldcg(&ctl->x_known) != 0u) {
        ctl->regathered = 1u;
        ctl->use_fallback = 0u;
        return;
    }
    const int sides = P.mode == kModeValues ? 1 : 2;
    for (int s = 0; s < sides; ++s) {
        const unsigned long long inv = __ldcg(&ctl->x_min_inv[s]);
        ctl->thr[s] = ~inv;
        ctl->sel_done[s] = 1u;
        if (inv == 0ull || __ldcg(&ctl->cand_cnt[s]) != (uint32_t)P.k) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
}

// ---------------------------------------------------------------- the route as one kernel

constexpr uint32_t kBarrierSpins = 1u << 19;   // polls (each a load from L2 and a short sleep, ~0.7 us) before a barrier gives up: ~0.4 s

struct ExactLaunch {
    const Prob* probs;
    uint32_t n_probs;
    uint32_t* any_exact;   // non-zero once a problem of the launch needs the route (set by the streaming pass)
    uint32_t* barrier;     // arrivals at the barriers of this launch (zeroed with the control blocks)
};

// All blocks of the (cooperative, hence fully resident) grid meet here: the `epoch`-th barrier is
// passed once epoch * n_blocks arrivals have been counted.  The wait is bounded; false (in every
// thread of the block) if it ran out.
__device__ __forceinline__ bool grid_barrier(uint32_t* word, uint32_t n_blocks, uint32_t& epoch) {
    __shared__ uint32_t s_ok;
    __syncthreads();
    ++epoch;
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(word, 1u);
        const uint32_t target = epoch * n_blocks;
        uint32_t ok = 1u;
        for (uint32_t spins = 0u; ; ++spins) {
            if (*reinterpret_cast<volatile uint32_t*>(word) >= target) break;
            if (spins >= kBarrierSpins) { ok = 0u; break; }
            __nanosleep(64);
        }
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0u;
}

// Copies problem `p` of the launch into shared memory (all threads call).
__device__ __forceinline__ void load_problem(const ExactLaunch& L, uint32_t p, Prob* s_prob) {
    __syncthreads();  // s_prob may still be read
    for (int i = threadIdx.x; i < (int)(sizeof(Prob) / 8); i += blockDim.x)
        reinterpret_cast<unsigned long long*>(s_prob)[i] = reinterpret_cast<const unsigned long long*>(L.probs + p)[i];
    __syncthreads();
}

enum ExactStepKind : int { XS_HIST0 = 0, XS_HIST1, XS_HIST2, XS_TIECOUNT, XS_TIESCAN, XS_COLLECT, XS_FINAL };

// One step of the route for every problem of the launch that needs it.  Problems are looked at 256
// at a time (every thread reads one problem's flags); all blocks see the same flags, so they all
// take the same path.
template <int STEP>
__device__ __forceinline__ void exact_step_all(const ExactLaunch& L, Prob* s_prob, ExactShared& sh, uint32_t* s_list,
                                               uint32_t* s_count) {
    for (uint32_t p0 = 0u; p0 < L.n_probs; p0 += kBlock) {
        __syncthreads();
        if (threadIdx.x == 0) *s_count = 0u;
        __syncthreads();
        const uint32_t p = p0 + threadIdx.x;
        if (p < L.n_probs) {
            const Ctl* ctl = L.probs[p].ctl;
            const bool active = exact_route_active(ctl);
            const bool wanted = active && (STEP == XS_COLLECT || STEP == XS_FINAL || ctl->x_known == 0u);
            if (wanted) s_list[atomicAdd(s_count, 1u)] = p;   // any order: the problems are independent
        }
        __syncthreads();
        const uint32_t count = *s_count;
        for (uint32_t j = 0u; j < count; ++j) {
            const uint32_t q = s_list[j];
            if ((STEP == XS_TIESCAN || STEP == XS_FINAL) && q % gridDim.x != blockIdx.x) continue;  // one block per problem (block-uniform)
            load_problem(L, q, s_prob);
            if (STEP == XS_HIST0) exact_hist_step<0>(*s_prob, blockIdx.x, gridDim.x, sh);
            if (STEP == XS_HIST1) exact_hist_step<1>(*s_prob, blockIdx.x, gridDim.x, sh);
            if (STEP == XS_HIST2) exact_hist_step<2>(*s_prob, blockIdx.x, gridDim.x, sh);
            if (STEP == XS_TIECOUNT) exact_tiecount_step(*s_prob, blockIdx.x, gridDim.x, sh);
            if (STEP == XS_TIESCAN) exact_tiescan_step(*s_prob, sh);
            if (STEP == XS_COLLECT) exact_collect_step(*s_prob, blockIdx.x, gridDim.x, sh);
            if (STEP == XS_FINAL) exact_final_step(*s_prob);
        }
    }
}

// Launched cooperatively.  Returns at once unless a problem of the launch needs the route.
__global__ void __launch_bounds__(kBlock) k_exact_route(const ExactLaunch L) {
    cudaTriggerProgrammaticLaunchCompletion();
    cudaGridDependencySynchronize();
    if (__ldcg(L.any_exact) == 0u) return;
    __shared__ Prob s_prob;
    __shared__ ExactShared sh;
    __shared__ uint32_t s_list[kBlock];
    __shared__ uint32_t s_count, s_full;
    // does any problem need the thresholds searched (and not only the gathering redone)?
    if (threadIdx.x == 0) s_full = 0u;
    __syncthreads();
    for (uint32_t p = threadIdx.x; p < L.n_probs; p += kBlock) {
        const Ctl* ctl = L.probs[p].ctl;
        if (exact_route_active(ctl) && ctl->x_known == 0u) s_full = 1u;
    }
    __syncthreads();
    const bool full = s_full != 0u;   // the same in every block: the flags were final before this kernel started
    uint32_t epoch = 0u;
    bool ok = true;
    if (full) {
        exact_step_all<XS_HIST0>(L, &s_prob, sh, s_list, &s_count);
        ok = ok && grid_barrier(L.barrier, gridDim.x, epoch);
        if (ok) exact_step_all<XS_HIST1>(L, &s_prob, sh, s_list, &s_count);
        ok = ok && grid_barrier(L.barrier, gridDim.x, epoch);
        if (ok) exact_step_all<XS_HIST2>(L, &s_prob, sh, s_list, &s_count);
        ok = ok && grid_barrier(L.barrier, gridDim.x, epoch);
        if (ok) exact_step_all<XS_TIECOUNT>(L, &s_prob, sh, s_list, &s_count);
        ok = ok && grid_barrier(L.barrier, gridDim.x, epoch);
        if (ok) exact_step_all<XS_TIESCAN>(L, &s_prob, sh, s_list, &s_count);
        ok = ok && grid_barrier(L.barrier, gridDim.x, epoch);
    }
    if (ok) {
        exact_step_all<XS_COLLECT>(L, &s_prob, sh, s_list, &s_count);
        ok = grid_barrier(L.barrier, gridDim.x, epoch);
        if (ok) {
            exact_step_all<XS_FINAL>(L, &s_prob, sh, s_list, &s_count);
            return;
        }
    }
    // a barrier gave up: whatever needed the route has no lists to go on with
    for (uint32_t p = threadIdx.x; p < L.n_probs; p += kBlock) {
        Ctl* ctl = L.probs[p].ctl;
        if (ctl->use_fallback != 0u) atomicOr(&ctl->status, SBC_STATUS_TIMEOUT);
    }
}

// Test instrument: one barrier that can never be passed (it waits for one block more than the grid
// has).  Shows that the wait of grid_barrier ends by itself and reports it.
__global__ void __launch_bounds__(kBlock) k_debug_barrier_timeout(uint32_t* word, uint32_t* status_out) {
    uint32_t epoch = 0u;
    const bool ok = grid_barrier(word, gridDim.x + 1u, epoch);
    if (threadIdx.x == 0 && !ok) atomicOr(status_out, SBC_STATUS_TIMEOUT);
}

}  // namespace sbc
