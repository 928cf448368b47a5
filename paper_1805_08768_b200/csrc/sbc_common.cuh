// Shared definitions for the SBC CUDA kernels (sm_100a).
//
// Vocabulary (paper notation): A = R + dW is the accumulated update
// (Algorithm 1), k the number of kept positions per side (Algorithm 2),
// b the Golomb parameter b* (Algorithm 3).  "side 0" is the positive side
// (val+), "side 1" the negative side (val-).
//
// Ordering trick used throughout: every fp32 value maps to an unsigned
// 32-bit key whose integer order is the value order (with -0 folded onto
// +0); side 1 uses the complemented key, so both sides are always "take the
// largest".  A candidate is one 64-bit composite, key in the high word and
// the complemented index in the low word, so that a larger composite means
// "larger value, or equal value and lower index" -- exactly the tie rule.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/sbc.h"

namespace sbc {

constexpr int kBlock = 256;           // threads per block for every kernel here
constexpr int kHistBins = 2048;       // 11-bit radix digits
constexpr uint32_t kSampleMax = 1u << 20;  // elements looked at to bound the thresholds
constexpr int kXTile = 4096;          // elements per tile in the exact-select fallback
constexpr int kWarpChunk = 512;       // elements one warp handles per step of the streaming pass
constexpr int kMaxSpanSteps = kXTile / kWarpChunk;  // a span is 1, 2, 4 or 8 steps and never straddles a tile
constexpr int kChunkCodewords = 256;  // most codewords per chunk-table entry (long streams)
constexpr uint32_t kOrderBlocksMax = 148 * 8;  // ordering kernels: most blocks a problem gets (long spans: one span per lane at 2^30 elements)
constexpr uint32_t kOrderBlocksWave = 148 * 5; // ... and what is resident at once on 148 SMs (the walk that writes needs 48 registers): the grid for short spans
constexpr int kSumBins = 254;         // one exact integer bin per fp32 exponent
constexpr uint32_t kSmallList = 8192;  // candidate lists up to this capacity are ranked by one block

// Stages that use the "last block to finish does the serial step" pattern.
enum Stage : int {
    ST_SAMPLE0 = 0, ST_SAMPLE1, ST_SAMPLE2, ST_COLLECT, ST_XH0, ST_XH1, ST_XH2,
    ST_HIST_S0, ST_HIST_S1, ST_FILTER_S0, ST_FILTER_S1, ST_SUM, ST_ORDER, ST_COUNT
};

// Device-side control block of one encode call; zeroed before the first kernel.
struct Ctl {
    uint32_t status;            // SBC_STATUS_* bits
    uint32_t use_fallback;      // 1: the candidate pass did not bracket both thresholds
    uint32_t launch_exact;      // in the launch's first problem: some problem of the launch has use_fallback set
    uint32_t x_barrier;         // in the launch's first problem: arrivals at the exact route's grid barriers
    uint32_t done[ST_COUNT];    // tickets for the last-block pattern
    // threshold bounds from the sample
    uint32_t s_bin0[2], s_rank[2];
    uint32_t s_prefix22[2];     // sampled mode: 22-bit prefix of the sample's order statistic
    uint32_t sampled_ok;        // sampled mode: the estimated thresholds were accepted
    uint32_t k_final;           // positions actually sent (k, or the count the sampled thresholds gave)
    float lo_f, hi_f;           // candidates: !(a < lo_f) for side 0, !(a > hi_f) for side 1
    uint32_t s_bin0_up[2], s_rank_up[2];  // the same search for the upper bound of the threshold
    uint32_t up_key[2];         // side key at and above which a candidate is certainly kept ("sure")
    uint32_t lo_key[2];         // side key of the lower bound: every candidate's key is at least this
    // candidates per side: all of them, those at or above up_key ("sure"), and the cursor of the band list
    uint32_t cand_cnt[2];
    uint32_t sure_cnt[2];
    uint32_t band_cnt[2];
    uint32_t overflow;          // a warp's region of the ordered list, or a band list, did not hold its entries
    uint32_t x_known;           // exact route: the thresholds are already known (x_thr), only the gathering is redone
    uint32_t regathered;        // the gathering was redone (what x_known asked for), and the fast route's kernels go on from there
    long long pre_bins[2][256]; // exact sums of the sure entries, gathered while they were flushed
    // exact select over A (fallback)
    uint32_t x_prefix[2], x_rank[2], x_thr[2], x_ties_take[2], x_ties_have[2];
    unsigned long long x_min_inv[2];  // complement of the smallest composite the exact route gathered (zero: none yet)
    // select over the candidate lists
    unsigned long long b_prefix[2];   // digits of the k-th largest composite found so far (relative to SelectDigits::sub)
    uint32_t b_rank[2];
    uint32_t list_cnt[2];             // entries that share the first digit with the k-th largest
    unsigned long long thr[2];  // kept <=> composite >= thr[side]
    uint32_t sel_done[2];       // thr[side] is final: the remaining selection kernels have nothing to do
    // sums and decision
    long long bins[2][256];
    double mu64[2];
    uint32_t side;
    float mu32;
    // Golomb stage
    unsigned long long nbits;
    uint32_t kept_total;
    uint32_t pad_;
};

// Zeroed scratch that sits right behind Ctl.
struct Hists {
    uint32_t s0[kHistBins];
    uint32_t s1[2][2][kHistBins];  // [side][0: lower bound's bin, 1: upper bound's bin]
    uint32_t s2[2][1024];
    uint32_t x[3][2][kHistBins];
    uint32_t b0[2][kHistBins];     // first digit of the entries the candidate select ranks
};

// Everything a kernel needs to know about one encode problem.  Lives in
// device memory (first bytes of the workspace).
struct Prob {
    const float* update;
    float* residual;
    long long n;
    long long k;
    int b;
    int vec_ok;                 // 1: update and residual are 16-byte aligned
    int mode;                   // kModeBinary (SBC) or kModeValues (top-p by magnitude, values sent)
    int sampled;                // 1: thresholds are the order statistics of a caller-given subsample
    const uint32_t* sample_idx; // sampled mode: m positions (device)
    uint8_t* stream;            // container out
    unsigned long long stream_cap;
    unsigned long long stream_bytes;  // bytes sbc_stream_bytes(n, p) promises to stay within
    float* out_mu;
    Ctl* ctl;
    Hists* hists;
    uint32_t* sample_keys;
    // Candidates in position order: the tensor is cut into spans of span_steps * 512 elements; the
    // entries of a span sit together in list[s], ascending, at span_rec[s][span] = {offset, count}.
    // The streaming pass gives each of its warps a private region of cap_w slots (no atomics, no
    // waits); the exact route reserves space tile by tile.
    unsigned long long* list[2];
    uint2* span_rec[2];
    // Candidates below the sample's upper bound of the threshold ("band"), in any order: the part
    // of the candidates the exact selection has to rank.  Without an upper bound: all of them.
    unsigned long long* band[2];
    unsigned long long* buf[2][2];   // ping-pong lists of the candidate select
    uint32_t* x_tile_cnt[2];
    struct RangeSum* rng_sum;        // per warp range of the ordering kernels: what its kept entries add up to
    struct RangeSum* blk_sum;        // the same per block (eight ranges)
    struct RangeBase* blk_base;      // where each block starts (rank, bit offset, previous position)
    uint32_t cap;               // capacity of each band list
    uint32_t list_cap;          // slots of each ordered list
    uint32_t cap_w;             // slots of one streaming warp's region
    uint32_t main_warps;        // warps of the streaming pass that share this problem
    uint32_t span_steps;        // steps (512 elements each) per span: 1, 2, 4 or 8
    uint32_t n_spans;
    uint32_t use_runs;          // 0: short-list form, only the band lists are needed
    uint32_t chunk_cw;          // codewords per chunk-table entry
    uint32_t m;                 // sample size
    unsigned long long sample_step;  // 128-byte lines between sampled segments, 20 fractional bits
    uint32_t s_target;          // rank looked up in the sample (the same for both sides)
    uint32_t s_up;              // rank in the sample of the upper bound (0: no upper bound)
    uint32_t n_xtiles, n_chunks;
    unsigned long long payload_offset;
};

// A launch serves one problem (prefix == nullptr: the grid is that problem's) or a batch: then
// prefix[i] .. prefix[i+1] are the blocks of problem i for this kernel's kind of work, and a block
// finds its problem by binary search.
struct Batch {
    const Prob* probs;
    const uint32_t* prefix;  // n_probs + 1 entries, or nullptr
    uint32_t n_probs;
    uint32_t* any_exact;     // one word per launch: non-zero once a problem needs the exact route
    // One-block-per-problem kernels of a batch: slot i of the grid works on problem perm[i] (largest
    // problems first: the grid can be larger than what is resident at once, and the blocks that
    // have to wait for a free slot should be the short ones).  nullptr: slot i is problem i.
    const uint32_t* perm;
};
struct Slot {
    const Prob* P;
    Prob* G;      // the descriptor in global memory (patched when the sent count is only known on the device)
    uint32_t bx;  // block index within the problem
    uint32_t nb;  // blocks working on the problem
};
// Finds the block's problem and copies its descriptor into shared memory (all threads call):
// kernels then read the descriptor at shared-memory cost and the compiler knows that their global
// stores cannot change it.
__device__ __forceinline__ Slot resolve(const Batch& B, Prob* s_prob) {
    // Programmatic dependent launch: the encode kernels are launched so that a kernel's blocks may
    // be placed on the SMs while the kernel before it in the stream is still running.  Let the next
    // kernel do the same as soon as every block of this one has got this far, then wait here until
    // the previous kernel has completed and its writes are visible.  Nothing above this line reads
    // memory another kernel writes.
    cudaTriggerProgrammaticLaunchCompletion();
    cudaGridDependencySynchronize();
    Slot s;
    const Prob* src;
    if (B.prefix == nullptr) {
        src = B.probs; s.bx = blockIdx.x; s.nb = gridDim.x;
    } else {
        // The block's problem: largest i with prefix[i] <= blockIdx.x.  The first warp searches
        // 32 ways at a time (two rounds of loads for up to 1024 problems); a binary search by one
        // thread costs a block ten dependent loads before it can start, in every kernel of the chain.
        __shared__ uint32_t s_slot[3];
        if (threadIdx.x < 32u) {
            const uint32_t lane = threadIdx.x;
            uint32_t lo = 0u, hi = B.n_probs;  // invariant: prefix[lo] <= blockIdx.x < prefix[hi]
            while (hi - lo > 1u) {
                const uint32_t step = (hi - lo + 31u) / 32u;
                const uint32_t probe = lo + lane * step;
                const bool le = probe < hi && B.prefix[probe] <= blockIdx.x;  // true on lanes 0..j
                const unsigned m = __ballot_sync(0xffffffffu, le);
                const uint32_t j = 31u - (uint32_t)__clz((int)(m | 1u));
                lo += j * step;
                hi = min(hi, lo + step);
            }
            if (lane < 2u) s_slot[1 + lane] = B.prefix[lo + lane];
            if (lane == 0u) s_slot[0] = B.perm ? B.perm[lo] : lo;
        }
        __syncthreads();
        src = B.probs + s_slot[0]; s.bx = blockIdx.x - s_slot[1]; s.nb = s_slot[2] - s_slot[1];
    }
    static_assert(sizeof(Prob) % 8 == 0, "copied as 8-byte words");
    for (int i = threadIdx.x; i < (int)(sizeof(Prob) / 8); i += blockDim.x)
        reinterpret_cast<unsigned long long*>(s_prob)[i] = reinterpret_cast<const unsigned long long*>(src)[i];
    __syncthreads();
    s.P = s_prob;
    s.G = const_cast<Prob*>(src);
    return s;
}

// Kinds of work a kernel's grid is sized by (one prefix table per kind in a batch).
enum WorkKind : int {
    WK_SAMPLE = 0, WK_MAIN, WK_CAND, WK_ORDER, WK_ONE, WK_STREAM,
    WK_PERM,   // not a kind of work: the row of the tables that holds the order in which one-block kernels take the problems
    WK_COUNT
};

// What the kept entries of one warp range of the ordering kernels add up to (see k_span_count).
struct RangeSum {
    uint32_t cnt;            // kept entries in the range
    uint32_t first, last;    // position of the first and the last of them (cnt > 0)
    uint32_t pad_;
    unsigned long long inner_bits;  // code lengths of all of them but the first (whose gap reaches into an earlier range)
};
struct RangeBase {
    uint32_t rank;           // kept entries before the range
    uint32_t prev_plus1;     // position of the last of those, plus one (0: none)
    unsigned long long bit;  // payload bits before the range
};

// ---------------------------------------------------------------- keys

__device__ __forceinline__ uint32_t key_of_bits(uint32_t bits) {
    if (bits == 0x80000000u) bits = 0u;  // -0 ranks with +0
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
__device__ __forceinline__ uint32_t bits_of_key(uint32_t key) {
    return (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;
}
__device__ __forceinline__ uint32_t side_key(int side, uint32_t key) { return side ? ~key : key; }

// What the selection ranks by.  kModeBinary: the signed value (Algorithm 2 takes the k largest of
// dW and of -dW).  kModeValues: the magnitude (Gradient Dropping keeps the k entries of largest
// |dW|); only side 0 exists then.
constexpr int kModeBinary = 0;
constexpr int kModeValues = 1;
__device__ __forceinline__ uint32_t select_key(int mode, uint32_t bits) {
    return mode == kModeValues ? (bits & 0x7fffffffu) : key_of_bits(bits);
}
__device__ __forceinline__ unsigned long long make_composite(uint32_t skey, uint32_t idx) {
    return ((unsigned long long)skey << 32) | (unsigned long long)(~idx);
}
__device__ __forceinline__ uint32_t composite_index(unsigned long long c) { return ~(uint32_t)c; }

// What the exact selection ranks and the exact sums read.  Fast route: the band list (every
// candidate below the sample's upper bound of the threshold; all `sure` entries above it are kept
// and already summed), with the rank reduced by the sure entries.  Exact route: the rebuilt list
// itself, which then holds nothing else (densely packed from slot 0).
struct BandView {
    const unsigned long long* src;
    uint32_t count;  // entries
    uint32_t rank;   // the k-th largest candidate is the rank-th largest of these
};
__device__ __forceinline__ BandView band_view(const Prob& P, const Ctl* ctl, int s) {
    BandView v;
    if (ctl->use_fallback) {
        v.src = P.list[s];
        v.count = min(ctl->cand_cnt[s], P.list_cap);
        v.rank = (uint32_t)P.k;
    } else {
        v.src = P.band[s];
        v.count = min(ctl->band_cnt[s], P.cap);
        v.rank = (uint32_t)P.k - min(ctl->sure_cnt[s], (uint32_t)P.k - 1u);  // sure < k on this route
    }
    return v;
}

// Digit schedule of the candidate select.  The entries it ranks lie in a known range of composites:
// `sub` is the smallest composite the range can hold and `top` the highest bit in which an entry
// can differ from it once `sub` is taken off.  Digits are 11 bits each, from bit `top` downwards
// (the last one takes what is left).  Fast route: the band between the two sample bounds, a narrow
// range of keys, so that already the first digit tells the entries apart; exact route: the whole
// range of composites (six digits).
struct SelectDigits {
    int top;
    unsigned long long sub;
};
__device__ __forceinline__ SelectDigits band_digits(const Ctl* ctl, int s) {
    const uint32_t lo = ctl->lo_key[s], width = ctl->up_key[s] - 1u - lo;  // band keys lie in [lo, lo + width]
    SelectDigits d;
    d.top = 63 - __clz((int)width);   // 31 for width 0: only the index half differs
    d.sub = (unsigned long long)lo << 32;
    return d;
}
__device__ __forceinline__ SelectDigits select_digits(const Ctl* ctl, int s) {
    if (ctl->use_fallback) { SelectDigits d; d.top = 63; d.sub = 0ull; return d; }
    return band_digits(ctl, s);
}
__device__ __forceinline__ int digit_bits(int level, int top) { return max(0, min(11, top + 1 - 11 * level)); }
__device__ __forceinline__ int digit_shift(int level, int top) { return max(0, top + 1 - 11 * (level + 1)); }
__device__ __forceinline__ int digit_levels(int top) { return (top + 1 + 10) / 11; }
// Digit `level` of a composite from which `sub` has already been taken off.
__device__ __forceinline__ uint32_t digit_of(unsigned long long c, int level, int top) {
    return (uint32_t)(c >> digit_shift(level, top)) & ((1u << digit_bits(level, top)) - 1u);
}

// Exact sum of fp32 values (Algorithm 2's means): a value is m * 2^(e-150) with an integer m of at
// most 24 bits, so one 64-bit integer per exponent holds the sum of up to 2^39 of them and integer
// addition makes the result independent of the order.  Values within eight binades above `bin_a`
// (nearly all of them, when bin_a is the binade below the threshold's) are added in one register,
// in units of the lowest of those binades; the rest goes to the 256 shared bins by atomics.
struct ExactSum {
    int bin_a;
    long long acc;
    __device__ __forceinline__ void start(uint32_t bits_near) {
        bin_a = max((int)((bits_near >> 23) & 0xffu) - 1, 0);
        acc = 0;
    }
    __device__ __forceinline__ void add(uint32_t bits, unsigned long long* s_bins) {
        const uint32_t e = (bits >> 23) & 0xffu;
        int m = (int)(bits & 0x7fffffu) | (e ? 0x800000 : 0);
        if (bits >> 31) m = -m;
        const int bin = e ? (int)e - 1 : 0;
        const uint32_t up = (uint32_t)(bin - bin_a);
        if (up < 8u) acc += (long long)m << up;   // |m| < 2^24: at most 2^31 per entry, 2^62 over 2^31 entries
        else atomicAdd(&s_bins[bin], (unsigned long long)(long long)m);
    }
    // All lanes of every warp of the block call; the bins are complete after the next barrier.
    __device__ __forceinline__ void finish(unsigned long long* s_bins) {
        long long v = acc;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(0xffffffffu, v, d);
        if ((threadIdx.x & 31u) == 0u && v) atomicAdd(&s_bins[bin_a], (unsigned long long)v);
        acc = 0;
    }
};

// Codewords per chunk-table entry of a stream that carries k positions.  The decoder gives every
// chunk to one lane, which parses it codeword after codeword, so short streams get short chunks:
// a stream of 10^5 positions then still occupies a hundred warps.  (A convention of the container;
// the header carries the value.)
__host__ __device__ __forceinline__ uint32_t chunk_codewords_for(unsigned long long k) {
    if (k < (1ull << 17)) return 32u;
    if (k < (1ull << 21)) return 64u;
    return (uint32_t)kChunkCodewords;
}
// Most chunk-table entries a stream of at most k_max positions can have (the chunk size grows with
// the number of positions, so the count is not monotone).
__host__ __device__ __forceinline__ unsigned long long chunks_of(unsigned long long k) {
    const unsigned long long c = chunk_codewords_for(k);
    return (k + c - 1ull) / c;
}
__host__ __device__ __forceinline__ unsigned long long max_chunks_upto(unsigned long long k_max) {
    unsigned long long m = chunks_of(k_max);
    if (k_max >= (1ull << 17) && chunks_of((1ull << 17) - 1ull) > m) m = chunks_of((1ull << 17) - 1ull);
    if (k_max >= (1ull << 21) && chunks_of((1ull << 21) - 1ull) > m) m = chunks_of((1ull << 21) - 1ull);
    return m;
}

// ---------------------------------------------------------------- scans

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T v) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T o = __shfl_up_sync(0xffffffffu, v, d);
        if ((int)lane_id() >= d) v += o;
    }
    return v;
}

// Exclusive scan over the kBlock threads of a block; *total gets the block sum.
// s_warp: shared scratch of kBlock/32 + 1 elements.  All threads must call.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* s_warp, T* total) {
    const int warp = threadIdx.x >> 5;
    T incl = warp_inclusive_scan(v);
    __syncthreads();  // s_warp may still be read from a previous call
    if (lane_id() == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        T w = (lane_id() < kBlock / 32) ? s_warp[lane_id()] : T(0);
        T wi = warp_inclusive_scan(w);
        if (lane_id() < kBlock / 32) s_warp[lane_id()] = wi - w;
        if (lane_id() == kBlock / 32 - 1) s_warp[kBlock / 32] = wi;
    }
    __syncthreads();
    if (total) *total = s_warp[kBlock / 32];
    return s_warp[warp] + incl - v;
}

// ---------------------------------------------------------------- last-block ticket

// True in exactly one block: the one that finishes last among n_blocks.  Every
// thread must have issued its global writes before calling; all threads call.
__device__ __forceinline__ bool last_block_ticket(uint32_t* counter, uint32_t n_blocks) {
    __shared__ uint32_t s_is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = atomicAdd(counter, 1u);
        s_is_last = (t == n_blocks - 1u) ? 1u : 0u;
    }
    __syncthreads();
    bool last = s_is_last != 0u;
    if (last) __threadfence();
    return last;
}

// ---------------------------------------------------------------- histogram pick

struct Pick {
    uint32_t bin;    // bin that holds the rank-th largest entry
    uint32_t rank;   // rank inside that bin (1 = largest in the bin)
    uint32_t count;  // entries in that bin
    uint32_t found;
};

// Walk a histogram from its top bin down and find where the `rank`-th entry
// falls.  `mirror` reads bin i of the view as hist[nbins-1-i] (the same counts
// seen from the complemented key).  All kBlock threads call; result in *out
// (shared) after the trailing barrier.
// `out2` (may be null) receives the same for a second rank `rank2` from the same walk.
// IN_SHARED: the histogram lives in the block's shared memory (plain loads) instead of global
// memory written by other blocks (loads that bypass L1).
template <bool IN_SHARED = false>
__device__ __forceinline__ void block_pick_desc(const uint32_t* hist, int nbins, bool mirror,
                                                uint32_t rank, uint32_t* s_scan, Pick* out,
                                                uint32_t rank2 = 0u, Pick* out2 = nullptr) {
    const int per = (nbins + kBlock - 1) / kBlock;  // bins per thread, walked top-down
    uint32_t h[kHistBins / kBlock];
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < kHistBins / kBlock; ++j) {
        int view = nbins - 1 - ((int)threadIdx.x * per + j);
        uint32_t v = 0;
        if (j < per && view >= 0) {
            const uint32_t* src = hist + (mirror ? nbins - 1 - view : view);
            v = IN_SHARED ? *src : __ldcg(src);
        }
        h[j] = v;
        sum += v;
    }
    if (threadIdx.x == 0) {
        out->found = 0u;
        if (out2) out2->found = 0u;
    }
    uint32_t total;
    uint32_t cum = block_exclusive_scan<uint32_t>(sum, s_scan, &total);
#pragma unroll
    for (int j = 0; j < kHistBins / kBlock; ++j) {
        if (j < per) {
            if (cum < rank && rank <= cum + h[j]) {
                out->bin = (uint32_t)(nbins - 1 - ((int)threadIdx.x * per + j));
                out->rank = rank - cum;
                out->count = h[j];
                out->found = 1u;
            }
            if (out2 && cum < rank2 && rank2 <= cum + h[j]) {
                out2->bin = (uint32_t)(nbins - 1 - ((int)threadIdx.x * per + j));
                out2->rank = rank2 - cum;
                out2->count = h[j];
                out2->found = 1u;
            }
            cum += h[j];
        }
    }
    __syncthreads();
}

// The bucket of the rank-th largest entry's first digit, from the finished histogram of the list
// the candidate select ranks: the start of b_prefix / b_rank.  One block, all threads call.
__device__ __forceinline__ void select_pick0(const Prob& P, Ctl* ctl, int s, uint32_t rank, int top, uint32_t* s_scan,
                                             Pick* s_pick) {
    block_pick_desc(P.hists->b0[s], 1 << digit_bits(0, top), false, rank, s_scan, s_pick);
    if (threadIdx.x == 0) {
        ctl->b_prefix[s] = (unsigned long long)s_pick->bin << digit_shift(0, top);
        ctl->b_rank[s] = s_pick->rank;
        if (!s_pick->found) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
    }
    __syncthreads();
}

// Add `v` to a shared-memory histogram with one atomic per distinct bin per warp.
__device__ __forceinline__ void warp_hist_add(uint32_t* s_hist, uint32_t bin, bool valid) {
    unsigned active = __ballot_sync(0xffffffffu, valid);
    if (!valid) return;
    unsigned peers = __match_any_sync(active, bin);
    if ((int)lane_id() == __ffs(peers) - 1) atomicAdd(&s_hist[bin], (uint32_t)__popc(peers));
}

}  // namespace sbc
