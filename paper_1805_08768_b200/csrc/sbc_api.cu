// Host side of the SBC C ABI: argument checks, workspace layout, kernel launches.
// Declared and documented in include/sbc.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/sbc.h"
#include "../../include/sbc_debug.h"
#include "sbc_common.cuh"
#include "sbc_decode.cuh"
#include "sbc_exact.cuh"
#include "sbc_front.cuh"
#include "sbc_golomb.cuh"
#include "sbc_select.cuh"
#include "sbc_small.cuh"

namespace sbc {
namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr size_t kProbSlotBytes = 512;  // one problem descriptor, padded
// The counting walk with one thread per span pays only where there are spans enough to fill the
// machine with threads (long spans of a small tensor leave most lanes without one).
constexpr unsigned long long kDenseSpansMin = 65536;
static_assert(sizeof(Prob) <= kProbSlotBytes, "descriptor must fit its slot");

// Host-side plan of one encode problem: scalar parameters and the layout of its scratch, which
// comes in two parts so that a batch can keep each part contiguous across problems:
//   zero part  control block + radix histograms (cleared before every call)
//   rest       everything that needs no clearing
struct Plan {
    long long n, k;
    int b, mode, sampled;
    uint32_t cap, m, n_xtiles, n_chunks, chunk_cw;
    uint32_t s_target, s_up;
    uint32_t main_blocks, main_warps, span_steps, n_spans, cap_w, list_cap, use_runs, order_blocks;
    bool dense_spans;   // sixteen kept entries or more per span expected
    unsigned long long payload_offset;
    size_t stream_bytes;
    size_t zero_bytes, off_ctl, off_hists;                 // offsets inside the zero part
    size_t rest_bytes, off_mu, off_sample, off_list[2], off_band[2], off_buf[2][2], off_xtile[2], off_span[2],
        off_rng_sum, off_blk_sum, off_blk_base;            // inside the rest
    size_t total;                                          // single problem: slot + zero + rest
};

// The layout of the ordered candidate lists depends on how many warps the streaming pass runs, so
// the grids that shape it are planned for the B200's 148 SMs whatever device is current (on
// another device the plan is still valid, only not tuned).
constexpr unsigned kPlanSMs = 148;

bool valid_p(double p) { return p > 0.0 && p < 1.0; }

inline unsigned grid_for(unsigned long long work_items, unsigned per_block, unsigned max_blocks);

// coarse_main: elements per streaming block, in units of 4096 (a batch gives its blocks several
// steps each).  force_runs: the launch this problem is part of takes the general chain of kernels
// even if this problem alone would fit the short-list form.
bool make_plan(long long n, double p, Plan* pl, int mode = kModeBinary, long long sampled_m = 0, unsigned coarse_main = 1,
               bool force_runs = false) {
    if (n <= 0 || n >= (1ll << 31) || !valid_p(p)) return false;
    const int b = sbc_golomb_b(p);
    if (b < 0 || b > 30) return false;
    const long long k = sbc_kept_count(n, p);
    pl->n = n;
    pl->k = k;
    pl->b = b;
    pl->cap = (uint32_t)std::min<long long>(n, 2 * k + 1024);
    // Sample size: a sixteenth of the tensor, but at least 128/p elements (so that the rank looked
    // up below is >= 128 and its relative margin stays small) and at most 2^20; whole 32-element
    // segments unless the sample is the whole tensor.
    {
        const long long want = std::max<long long>(n / 16, (long long)std::ceil(128.0 / p));
        long long m = std::min<long long>(std::min<long long>(want, (long long)kSampleMax), n);
        if (m < n) m = std::max<long long>(32, m / 32 * 32);
        if (m >= n || (n >> 5) < (m >> 5)) m = n;
        pl->m = (uint32_t)m;
    }
    // Rank looked up in the sample.  If the sample is the whole tensor the
    // rank is k itself; otherwise the expected rank plus six standard
    // deviations of a binomial count (and a little), so that the bound falls
    // below the true k-th value except with negligible probability -- and if
    // it does not, the exact route takes over.
    // The same sample bounds the threshold from above (four deviations below the expected rank):
    // candidates at or above that bound are certainly kept, so the exact selection only has to
    // look at the band between the two bounds.  A bound that turns out too low costs time, not
    // correctness: the selection then runs over the certain part instead.
    uint32_t target, up = 0;
    if ((long long)pl->m == n) {
        target = (uint32_t)k;
        up = (uint32_t)k;
    } else {
        const double expect = (double)k * (double)pl->m / (double)n;
        const double t = std::ceil(expect + 6.0 * std::sqrt(expect) + 8.0);
        target = (uint32_t)std::min<double>(t, (double)pl->m);
        const double u = std::floor(expect - 4.0 * std::sqrt(expect) - 4.0);
        up = u >= 1.0 ? (uint32_t)u : 0u;
    }
    pl->sampled = sampled_m > 0;
    if (pl->sampled) {  // the caller's subsample; its floor(p*m)-th order statistics ARE the thresholds
        if (sampled_m > (long long)kSampleMax) return false;
        pl->m = (uint32_t)sampled_m;
        target = (uint32_t)std::max<long long>(1, (long long)std::floor(p * (double)sampled_m));
        up = 0;  // every candidate is kept: nothing is selected afterwards
    }
    if (pl->cap <= kSmallList && !force_runs) up = 0;  // a list one block ranks in its registers has no use for the second bound
    pl->s_target = target;
    pl->s_up = up;
    pl->n_xtiles = (uint32_t)((n + kXTile - 1) / kXTile);
    const long long k_max = pl->sampled ? (long long)pl->cap : k;  // most positions a stream can carry
    pl->chunk_cw = chunk_codewords_for((unsigned long long)k);
    // exact modes: the table of a stream of k positions; sampled mode: the largest table a stream
    // of up to k_max positions can have (the device patches count and chunk size once it knows k)
    pl->n_chunks = pl->sampled ? (uint32_t)max_chunks_upto((unsigned long long)k_max)
                               : (uint32_t)((k + pl->chunk_cw - 1) / pl->chunk_cw);
    pl->payload_offset = SBC_HEADER_BYTES + (unsigned long long)pl->n_chunks * SBC_CHUNK_ENTRY_BYTES;
    if (mode == kModeValues) pl->payload_offset += align_up((size_t)k * 4, 16);  // the values sit before the payload
    pl->mode = mode;
    const unsigned long long bits_bound =
        (unsigned long long)k_max * (1ull + b) + ((unsigned long long)(n - std::min<long long>(n, k_max)) >> b) +
        (pl->sampled ? ((unsigned long long)n >> b) : 0ull);
    pl->stream_bytes = (size_t)pl->payload_offset + align_up((size_t)((bits_bound + 7) / 8), 16);

    // Streaming pass: blocks, warps, spans, and each warp's region of the ordered lists.
    pl->main_blocks = grid_for((unsigned long long)n, kBlock * kPerThread * coarse_main, kPlanSMs * kCollectBlocksPerSM);
    pl->main_warps = pl->main_blocks * (kBlock / 32);
    const unsigned long long n_steps = ((unsigned long long)n + kWarpChunk - 1) / kWarpChunk;
    // the longest span (8, 4, 2 or 1 steps) that still leaves every warp at least two spans
    pl->span_steps = 1;
    for (uint32_t steps = kMaxSpanSteps; steps > 1; steps >>= 1)
        if ((n_steps + steps - 1) / steps >= 2ull * pl->main_warps) { pl->span_steps = steps; break; }
    pl->n_spans = (uint32_t)((n_steps + pl->span_steps - 1) / pl->span_steps);
    // the short-list form (one kernel after the candidate pass, which orders the positions itself)
    // needs no ordered lists; everything else walks them
    pl->use_runs = force_runs || !(pl->cap <= kSmallList && k <= (long long)kSmallKept && mode == kModeBinary && !pl->sampled);
    {
        // candidates a warp expects per side: its share of the spans times the density the lower
        // bound lets through (about k/n and a margin); twice that, eight deviations and a floor
        const unsigned long long spans_per_warp = (pl->n_spans + pl->main_warps - 1) / pl->main_warps;
        const double elems = (double)std::min<unsigned long long>((unsigned long long)n, spans_per_warp * pl->span_steps * kWarpChunk);
        const double expect = (double)k_max * elems / (double)n;
        double slots = std::ceil(2.0 * expect + 8.0 * std::sqrt(expect) + 64.0);
        slots = std::min(slots, elems);                 // a warp cannot see more candidates than elements
        pl->cap_w = (uint32_t)((unsigned long long)slots + 15ull) / 16u * 16u;   // whole 128-byte lines
        const unsigned long long regions = pl->use_runs ? (unsigned long long)pl->main_warps * pl->cap_w : 0ull;
        pl->list_cap = (uint32_t)std::min<unsigned long long>(std::max<unsigned long long>(regions, pl->cap), 0xfffffff0ull);
        if (regions > 0xfffffff0ull) return false;      // cannot happen below 2^31 elements
    }
    // a span or more per warp; where spans are long and many (see k_span_count) as many blocks as it takes
    // to give every lane of the counting walk one span, else one resident wave
    pl->dense_spans = (unsigned long long)k >= 16ull * pl->n_spans && pl->n_spans >= kDenseSpansMin;
    pl->order_blocks = grid_for(pl->n_spans, kBlock / 32, pl->dense_spans ? kOrderBlocksMax : kOrderBlocksWave);

    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    pl->off_ctl = take(sizeof(Ctl));
    pl->off_hists = take(sizeof(Hists));
    pl->zero_bytes = off;
    off = 0;
    pl->off_mu = take(sizeof(float));  // where the host-buffer form parks mu
    pl->off_sample = take((size_t)pl->m * 4);
    for (int s = 0; s < 2; ++s) pl->off_list[s] = take((size_t)pl->list_cap * 8);
    for (int s = 0; s < 2; ++s) pl->off_band[s] = take((size_t)pl->cap * 8);
    for (int s = 0; s < 2; ++s)
        for (int j = 0; j < 2; ++j) pl->off_buf[s][j] = take((size_t)pl->cap * 8);
    for (int s = 0; s < 2; ++s) pl->off_xtile[s] = take((size_t)pl->n_xtiles * 4);
    for (int s = 0; s < 2; ++s) pl->off_span[s] = take(pl->use_runs ? (size_t)pl->n_spans * sizeof(uint2) : 0);
    pl->off_rng_sum = take(pl->use_runs ? (size_t)pl->order_blocks * (kBlock / 32) * sizeof(RangeSum) : 0);
    pl->off_blk_sum = take(pl->use_runs ? (size_t)pl->order_blocks * sizeof(RangeSum) : 0);
    pl->off_blk_base = take(pl->use_runs ? (size_t)pl->order_blocks * sizeof(RangeBase) : 0);
    pl->rest_bytes = off;
    pl->total = kProbSlotBytes + pl->zero_bytes + pl->rest_bytes;
    return true;
}

struct TensorArgs {
    const float* update;
    float* residual;
    void* out_stream;
    size_t out_capacity;
    float* out_mu;
};

// Host-visible argument errors of one tensor (nothing is enqueued if any tensor fails).
int check_tensor(const TensorArgs& a, const Plan& pl) {
    if (!a.update || !a.residual || !a.out_stream) return SBC_EINVAL;
    if (((uintptr_t)a.update & 3) || ((uintptr_t)a.residual & 3) || ((uintptr_t)a.out_stream & 15) ||
        (a.out_mu && ((uintptr_t)a.out_mu & 3)))
        return SBC_EINVAL;
    const uintptr_t u0 = (uintptr_t)a.update, r0 = (uintptr_t)a.residual, len = (uintptr_t)pl.n * 4;
    if (u0 < r0 + len && r0 < u0 + len) return SBC_EINVAL;  // update and residual must not overlap
    if (a.out_capacity < pl.stream_bytes) return SBC_ECAPACITY;
    return SBC_OK;
}

Prob make_prob(const TensorArgs& a, const Plan& pl, uint8_t* zero, uint8_t* rest) {
    Prob P;
    std::memset(&P, 0, sizeof(P));
    P.update = a.update;
    P.residual = a.residual;
    P.n = pl.n;
    P.k = pl.k;
    P.b = pl.b;
    P.vec_ok = (((uintptr_t)a.update | (uintptr_t)a.residual) & 15) == 0;
    P.mode = pl.mode;
    P.sampled = pl.sampled;
    P.stream = static_cast<uint8_t*>(a.out_stream);
    P.stream_cap = a.out_capacity;
    P.stream_bytes = pl.stream_bytes;
    P.out_mu = a.out_mu;
    P.ctl = reinterpret_cast<Ctl*>(zero + pl.off_ctl);
    P.hists = reinterpret_cast<Hists*>(zero + pl.off_hists);
    P.sample_keys = reinterpret_cast<uint32_t*>(rest + pl.off_sample);
    for (int s = 0; s < 2; ++s) {
        P.list[s] = reinterpret_cast<unsigned long long*>(rest + pl.off_list[s]);
        P.band[s] = reinterpret_cast<unsigned long long*>(rest + pl.off_band[s]);
        P.span_rec[s] = reinterpret_cast<uint2*>(rest + pl.off_span[s]);
        for (int j = 0; j < 2; ++j) P.buf[s][j] = reinterpret_cast<unsigned long long*>(rest + pl.off_buf[s][j]);
        P.x_tile_cnt[s] = reinterpret_cast<uint32_t*>(rest + pl.off_xtile[s]);
    }
    P.rng_sum = reinterpret_cast<RangeSum*>(rest + pl.off_rng_sum);
    P.blk_sum = reinterpret_cast<RangeSum*>(rest + pl.off_blk_sum);
    P.blk_base = reinterpret_cast<RangeBase*>(rest + pl.off_blk_base);
    P.s_target = pl.s_target;
    P.s_up = pl.s_up;
    P.cap = pl.cap;
    P.list_cap = pl.list_cap;
    P.cap_w = pl.cap_w;
    P.main_warps = pl.main_warps;
    P.span_steps = pl.span_steps;
    P.n_spans = pl.n_spans;
    P.use_runs = pl.use_runs;
    P.chunk_cw = pl.chunk_cw;
    P.m = pl.m;
    P.sample_step = (pl.m >> 5) ? ((unsigned long long)(pl.n >> 5) << 20) / (unsigned long long)(pl.m >> 5) : 0ull;
    P.n_xtiles = pl.n_xtiles;
    P.n_chunks = pl.n_chunks;
    P.payload_offset = pl.payload_offset;
    return P;
}

int sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 148;
    return sms;
}

inline unsigned grid_for(unsigned long long work_items, unsigned per_block, unsigned max_blocks) {
    unsigned long long g = (work_items + per_block - 1) / per_block;
    if (g < 1) g = 1;
    if (g > max_blocks) g = max_blocks;
    return (unsigned)g;
}

// Blocks one problem gets for each kind of work.  The coarsening factor (1 for a single problem)
// makes the blocks of the sample kernels that many times larger: every block of those kernels
// pays for clearing and flushing a shared-memory histogram, and a batch of hundreds of problems
// has parallelism to spare.  The streaming pass and the ordering kernels take their grids from
// the plan (the layout of the ordered lists depends on them).
void block_counts(const Plan& pl, unsigned sms, unsigned coarse_sample, unsigned nb[WK_COUNT]) {
    nb[WK_SAMPLE] = grid_for(pl.m, kBlock * 8 * coarse_sample, sms * 4);
    nb[WK_MAIN] = pl.main_blocks;
    nb[WK_CAND] = grid_for(pl.cap, kBlock * 4, sms * 2);  // x 2 sides: one resident wave at four blocks per SM
    nb[WK_ORDER] = pl.order_blocks;
    nb[WK_ONE] = 1;
    nb[WK_STREAM] = grid_for(pl.stream_bytes, kBlock * 64, sms * 4);
    nb[WK_PERM] = 0;
}

// Set-up of a single encode in one launch instead of two memsets and a descriptor kernel: the
// descriptor (a kernel argument) goes to the head of the workspace, the scratch that must start at zero (control
// block, histograms, tile counters: `zero_words` 16-byte words at `zero`) and the chunk table and
// payload area the packer ORs into (`stream_words` at `stream_zero`) are cleared.
__global__ void __launch_bounds__(kBlock) k_prepare(Prob* dst, const Prob src, uint4* zero, size_t zero_words,
                                                    uint4* stream_zero, size_t stream_words) {
    if (blockIdx.x == 0 && threadIdx.x == 0) *dst = src;
    const size_t tid = (size_t)blockIdx.x * kBlock + threadIdx.x, stride = (size_t)gridDim.x * kBlock;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (size_t i = tid; i < zero_words; i += stride) zero[i] = z;
    for (size_t i = tid; i < stream_words; i += stride) stream_zero[i] = z;
}

// Plain byte copy (16 bytes per thread and step where both sides are 16-byte aligned).
__global__ void __launch_bounds__(kBlock) k_copy_bytes(uint8_t* __restrict__ dst, const uint8_t* __restrict__ src,
                                                       size_t bytes) {
    const size_t tid = (size_t)blockIdx.x * kBlock + threadIdx.x, stride = (size_t)gridDim.x * kBlock;
    if ((((uintptr_t)dst | (uintptr_t)src) & 15) == 0) {
        const size_t vecs = bytes / 16;
        for (size_t i = tid; i < vecs; i += stride)
            reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
        for (size_t i = vecs * 16 + tid; i < bytes; i += stride) dst[i] = src[i];
    } else {
        for (size_t i = tid; i < bytes; i += stride) dst[i] = src[i];
    }
}

// Zero the chunk table and payload area of every problem's output stream (batch form; a single
// encode uses one memset instead).
__global__ void __launch_bounds__(kBlock) k_zero_stream(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    uint4* dst = reinterpret_cast<uint4*>(P.stream + SBC_HEADER_BYTES);
    const unsigned long long count = (P.stream_bytes - SBC_HEADER_BYTES) / 16ull;
    for (unsigned long long i = (unsigned long long)S.bx * kBlock + threadIdx.x; i < count;
         i += (unsigned long long)S.nb * kBlock)
        dst[i] = make_uint4(0u, 0u, 0u, 0u);
}

// Grid of the exact route's cooperative kernel: two blocks per SM (fewer if fewer fit), all of which
// must be resident at once.  Looked up once per device.
unsigned exact_route_blocks() {
    static std::mutex mu;
    static unsigned cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148u;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0u) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_exact_route, kBlock, 0) != cudaSuccess || per_sm < 1)
            per_sm = 1;
        cached[dev] = (unsigned)sm_count() * (unsigned)std::min(per_sm, 2);
    }
    return cached[dev];
}

// Enqueue every kernel of the encode path once; `grid[kind]` blocks and `prefix[kind]` (null for
// a single problem) say how each kind of work is spread over the problems.
void launch_encode(const Prob* d_probs, uint32_t n_probs, uint32_t* any_exact, const unsigned grid[WK_COUNT],
                   const uint32_t* const* prefix, int mode, bool sampled, bool small_lists, bool small_form, bool dense_spans,
                   cudaStream_t st, const sbc_cuda_event_t* marks) {
    // Every stage boundary closes an NVTX range and opens the next one (host-side ranges around the
    // launches of a stage, for a timeline tool; no-ops when none is attached), and records the
    // caller's event for that boundary if it gave one.
    static const char* const kStageNames[SBC_MARK_COUNT] = {"sbc_encode: bounds", "sbc_encode: accumulate + collect",
                                                            "sbc_encode: exact route", "sbc_encode: select + sums",
                                                            "sbc_encode: order + golomb", ""};
    nvtxRangePushA(kStageNames[0]);
    auto mark = [&](int i) {
        if (marks && marks[i]) cudaEventRecord(marks[i], st);
        nvtxRangePop();
        if (i + 1 < SBC_MARK_COUNT) nvtxRangePushA(kStageNames[i]);
    };
    auto B = [&](int kind) {
        return Batch{d_probs, prefix ? prefix[kind] : nullptr, n_probs, any_exact, (prefix && kind == WK_ONE) ? prefix[WK_PERM] : nullptr};
    };
    auto g1 = [&](int kind) { return dim3(grid[kind]); };
    auto g2 = [&](int kind) { return dim3(grid[kind], 1, 2); };  // z = side
    // Every kernel is launched with programmatic stream serialisation: its blocks may be placed
    // while the previous kernel drains; each kernel waits for its predecessor in resolve().
    // The two long kernels (streaming pass, second ordering walk with the residual write-back) are launched the ordinary way:
    // blocks placed early land wherever the draining kernel happens to free a slot, and the uneven
    // spread over the SMs cost the write-back 30 % at 2^30 elements, p = 1e-2.
    auto go = [&](void (*kernel)(Batch), dim3 g, Batch arg, bool early = true) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = g;
        cfg.blockDim = dim3(kBlock);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = early ? 1 : 0;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, kernel, arg);
    };

    // 1. bounds from the sample, then the streaming accumulate + collect pass
    go(k_sample0, g1(WK_SAMPLE), B(WK_SAMPLE));
    go(k_sample1, g1(WK_SAMPLE), B(WK_SAMPLE));
    if (sampled) go(k_sample2, g1(WK_SAMPLE), B(WK_SAMPLE));
    mark(SBC_MARK_BOUNDS);
    // (a batch's streaming pass is made of many short blocks: there early placement helps)
    if (mode == kModeValues) go(k_add_collect<kModeValues>, g1(WK_MAIN), B(WK_MAIN), prefix != nullptr);
    else                     go(k_add_collect<kModeBinary>, g1(WK_MAIN), B(WK_MAIN), prefix != nullptr);
    mark(SBC_MARK_COLLECT);

    // 2. exact route over A: one cooperative kernel (its steps meet at grid barriers), which returns
    // at once unless the candidate pass failed for some problem of the launch
    {
        ExactLaunch xl = {d_probs, n_probs, any_exact, any_exact + 1};   // launch_exact and x_barrier are neighbours
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(exact_route_blocks());
        cfg.blockDim = dim3(kBlock);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, k_exact_route, xl);
    }
    mark(SBC_MARK_EXACT);

    // 3. exact k-th composite of each candidate list, sums, side
    // 4. ordered positions, residual write-back, Golomb payload, chunk table, header
    if (small_form) {  // every problem of the launch is short: all of it by two blocks per problem
        mark(SBC_MARK_SELECT);
        go(k_small_finish, g2(WK_ONE), B(WK_ONE));
        mark(SBC_MARK_END);
        return;
    }
    if (small_lists) {  // every list of this launch fits one block's registers: one kernel ranks them
        go(k_select_small, g2(WK_ONE), B(WK_ONE));
    } else {
        go(k_select_hist0, g2(WK_CAND), B(WK_CAND));
        go(k_select_filter0, g2(WK_CAND), B(WK_CAND));
    }
    mark(SBC_MARK_SELECT);

    if (dense_spans) go(k_span_count<true>, g1(WK_ORDER), B(WK_ORDER));
    else             go(k_span_count<false>, g1(WK_ORDER), B(WK_ORDER));
    go(k_span_emit, g1(WK_ORDER), B(WK_ORDER), false);
    mark(SBC_MARK_END);
}

}  // namespace
}  // namespace sbc

using namespace sbc;

extern "C" {

int64_t sbc_kept_count(int64_t numel, double p) {
    if (numel <= 0 || !valid_p(p)) return 0;
    int64_t k = (int64_t)std::floor(p * (double)numel);
    if (k < 1) k = 1;
    if (k > numel) k = numel;
    return k;
}

int sbc_golomb_b(double p) {
    if (!valid_p(p)) return -1;
    const double golden = (1.0 + std::sqrt(5.0)) * 0.5;
    const double x = std::log(golden - 1.0) / std::log(1.0 - p);
    const int b = 1 + (int)std::floor(std::log2(x));
    return b < 0 ? 0 : b;
}

double sbc_mean_position_bits(double p, int b) {
    return (double)b + 1.0 / (1.0 - std::pow(1.0 - p, std::ldexp(1.0, b)));
}

size_t sbc_stream_bytes(int64_t numel, double p) {
    Plan pl;
    return make_plan(numel, p, &pl) ? pl.stream_bytes : 0;
}

size_t sbc_workspace_bytes(int64_t numel, double p) {
    // the same figure serves sbc_encode and sbc_encode_values: sized for the general chain of
    // kernels, which the short-list form of sbc_encode needs only a part of
    Plan pl;
    return make_plan(numel, p, &pl, kModeBinary, 0, 1, true) ? pl.total : 0;
}

int sbc_encode(const float* update, float* residual, int64_t numel, double p, void* out_stream,
               size_t out_capacity, float* out_mu, void* workspace, size_t workspace_bytes,
               sbc_cuda_stream_t stream) {
    return sbc_encode_ex(update, residual, numel, p, out_stream, out_capacity, out_mu, workspace,
                         workspace_bytes, stream, nullptr);
}

static int encode_impl(int mode, const uint32_t* sample_idx, int64_t sample_m, const float* update,
                       float* residual, int64_t numel, double p, void* out_stream, size_t out_capacity,
                       float* out_mu, void* workspace, size_t workspace_bytes, sbc_cuda_stream_t stream,
                       const sbc_cuda_event_t* marks) {
    Plan pl;
    if (!workspace || ((uintptr_t)workspace & 255)) return SBC_EINVAL;
    if (sample_idx && (sample_m <= 0 || ((uintptr_t)sample_idx & 3))) return SBC_EINVAL;
    if (!make_plan(numel, p, &pl, mode, sample_idx ? sample_m : 0)) return SBC_EINVAL;
    const TensorArgs a = {update, residual, out_stream, out_capacity, out_mu};
    const int rc = check_tensor(a, pl);
    if (rc != SBC_OK) return rc;
    if (workspace_bytes < pl.total) return SBC_ECAPACITY;

    // workspace: [descriptor][zero part][rest]
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* zero = ws + kProbSlotBytes;
    uint8_t* rest = zero + pl.zero_bytes;
    const bool small_lists = pl.cap <= kSmallList, small_form = !pl.use_runs;
    Prob P = make_prob(a, pl, zero, rest);
    P.sample_idx = sample_idx;
    Prob* d_prob = reinterpret_cast<Prob*>(ws);

    cudaStream_t st = stream;
    if (marks && marks[SBC_MARK_BEGIN]) cudaEventRecord(marks[SBC_MARK_BEGIN], st);
    // scratch that must start at zero: control block + histograms,
    // and the chunk table + payload area the packer ORs into
    {
        // both regions are 16-byte aligned and whole multiples of 16 bytes (workspace parts are
        // 256-byte aligned, the stream pointer 16-byte aligned, header and stream size multiples of 16)
        const size_t zero_words = pl.zero_bytes / 16, stream_words = (pl.stream_bytes - SBC_HEADER_BYTES) / 16;
        const unsigned blocks = grid_for(zero_words + stream_words, kBlock * 4, (unsigned)sm_count() * 4u);
        k_prepare<<<blocks, kBlock, 0, st>>>(d_prob, P, reinterpret_cast<uint4*>(zero), zero_words,
                                            reinterpret_cast<uint4*>(P.stream + SBC_HEADER_BYTES), stream_words);
    }

    unsigned grid[WK_COUNT];
    block_counts(pl, (unsigned)sm_count(), 1u, grid);
    launch_encode(d_prob, 1u, &P.ctl->launch_exact, grid, nullptr, mode, pl.sampled != 0, small_lists, small_form,
                  pl.dense_spans, st, marks);
    return cudaGetLastError() == cudaSuccess ? SBC_OK : SBC_ECUDA;
}

int sbc_encode_ex(const float* update, float* residual, int64_t numel, double p, void* out_stream,
                  size_t out_capacity, float* out_mu, void* workspace, size_t workspace_bytes,
                  sbc_cuda_stream_t stream, const sbc_cuda_event_t* marks) {
    return encode_impl(kModeBinary, nullptr, 0, update, residual, numel, p, out_stream, out_capacity, out_mu, workspace,
                       workspace_bytes, stream, marks);
}

size_t sbc_stream_bytes_sampled(int64_t numel, double p) {
    Plan pl;
    return make_plan(numel, p, &pl, kModeBinary, 32) ? pl.stream_bytes : 0;  // the bound does not depend on m
}

size_t sbc_workspace_bytes_sampled(int64_t numel, double p, int64_t sample_count) {
    Plan pl;
    return (sample_count > 0 && make_plan(numel, p, &pl, kModeBinary, sample_count)) ? pl.total : 0;
}

int sbc_encode_sampled(const float* update, float* residual, int64_t numel, double p, const uint32_t* sample_idx,
                       int64_t sample_count, void* out_stream, size_t out_capacity, float* out_mu, void* workspace,
                       size_t workspace_bytes, sbc_cuda_stream_t stream) {
    if (!sample_idx) return SBC_EINVAL;
    return encode_impl(kModeBinary, sample_idx, sample_count, update, residual, numel, p, out_stream, out_capacity,
                       out_mu, workspace, workspace_bytes, stream, nullptr);
}

size_t sbc_stream_bytes_values(int64_t numel, double p) {
    Plan pl;
    return make_plan(numel, p, &pl, kModeValues) ? pl.stream_bytes : 0;
}

int sbc_encode_values(const float* update, float* residual, int64_t numel, double p, void* out_stream,
                      size_t out_capacity, void* workspace, size_t workspace_bytes, sbc_cuda_stream_t stream) {
    return encode_impl(kModeValues, nullptr, 0, update, residual, numel, p, out_stream, out_capacity, nullptr, workspace,
                       workspace_bytes, stream, nullptr);
}

// Plans of all tensors of a batch.  Two things are decided over the whole batch: how many steps a
// streaming block gets (about two waves of resident blocks over the batch, so that a block's
// start-up -- finding its problem, reading the bounds -- and its final flush are paid for by
// several steps of loads), and whether the launch can use the short-list form (only if every
// tensor fits it).
static bool plan_batch(int n_tensors, const sbc_tensor_desc* descs, std::vector<Plan>* plans, bool* all_small) {
    unsigned long long fine_main = 0;
    bool small = true;
    Plan pl;
    for (int t = 0; t < n_tensors; ++t) {
        if (!make_plan(descs[t].numel, descs[t].p, &pl)) return false;
        fine_main += (unsigned long long)(pl.n + kBlock * kPerThread - 1) / (kBlock * kPerThread);
        small = small && !pl.use_runs;
    }
    unsigned coarse_main = (unsigned)std::min<unsigned long long>(
        16, std::max<unsigned long long>(1, fine_main / (kPlanSMs * 2 * kCollectBlocksPerSM)));
    // Whole waves: with every tensor's block count rounded up, the rule above can leave a last wave
    // that is half empty.  Blocks of up to 32 x 4096 elements if the batch then fits one resident
    // wave (a few large tensors: a block's start-up and final flush cost as much as several
    // steps), else the smallest blocks that fit two.
    auto blocks_at = [&](unsigned c) {
        unsigned long long blocks = 0;
        for (int t = 0; t < n_tensors; ++t)
            blocks += ((unsigned long long)descs[t].numel + (unsigned long long)kBlock * kPerThread * c - 1) / ((unsigned long long)kBlock * kPerThread * c);
        return blocks;
    };
    const unsigned long long wave = (unsigned long long)kPlanSMs * kCollectBlocksPerSM;
    if (blocks_at(32) <= wave) {
        while (blocks_at(coarse_main) > wave) ++coarse_main;
    } else if (blocks_at(32) <= 2 * wave) {
        while (blocks_at(coarse_main) > 2 * wave) ++coarse_main;
    }
    plans->resize((size_t)n_tensors);
    for (int t = 0; t < n_tensors; ++t)
        if (!make_plan(descs[t].numel, descs[t].p, &(*plans)[t], kModeBinary, 0, coarse_main, !small)) return false;
    *all_small = small;
    return true;
}

size_t sbc_workspace_bytes_batch(int n_tensors, const sbc_tensor_desc* descs) {
    if (n_tensors <= 0 || n_tensors > (1 << 20) || !descs) return 0;
    std::vector<Plan> plans;
    bool all_small;
    if (!plan_batch(n_tensors, descs, &plans, &all_small)) return 0;
    size_t total = align_up((size_t)n_tensors * sizeof(Prob), 256) +
                   align_up((size_t)WK_COUNT * (size_t)(n_tensors + 1) * 4, 256);
    for (int t = 0; t < n_tensors; ++t) total += plans[t].zero_bytes + plans[t].rest_bytes;
    return total;
}

int sbc_encode_batch(int n_tensors, const sbc_tensor_desc* descs, void* workspace, size_t workspace_bytes,
                     sbc_cuda_stream_t stream) {
    if (n_tensors <= 0 || !descs || !workspace || ((uintptr_t)workspace & 255)) return SBC_EINVAL;
    if (n_tensors > (1 << 20)) return SBC_EINVAL;
    std::vector<Plan> plans;
    bool all_small;
    if (!plan_batch(n_tensors, descs, &plans, &all_small)) return SBC_EINVAL;
    size_t zero_total = 0, rest_total = 0;
    for (int t = 0; t < n_tensors; ++t) {
        const TensorArgs a = {descs[t].update, descs[t].residual, descs[t].out_stream, descs[t].out_capacity,
                              descs[t].out_mu};
        const int rc = check_tensor(a, plans[t]);
        if (rc != SBC_OK) return rc;
        zero_total += plans[t].zero_bytes;
        rest_total += plans[t].rest_bytes;
    }
    const size_t probs_bytes = align_up((size_t)n_tensors * sizeof(Prob), 256);
    const size_t prefix_bytes = align_up((size_t)WK_COUNT * (size_t)(n_tensors + 1) * 4, 256);
    if (workspace_bytes < probs_bytes + prefix_bytes + zero_total + rest_total) return SBC_ECAPACITY;

    // workspace: [descriptors][prefix tables][zero parts][rests]
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    Prob* d_probs = reinterpret_cast<Prob*>(ws);
    uint32_t* d_prefix = reinterpret_cast<uint32_t*>(ws + probs_bytes);
    uint8_t* zero = ws + probs_bytes + prefix_bytes;
    uint8_t* rest = zero + zero_total;

    const unsigned sms = (unsigned)sm_count();
    // Sample kernels: the smallest block size (in units of 2048 sampled elements) with which the
    // blocks of the whole batch are resident at once (four per SM); a second, short wave would cost
    // as much time again as the first.
    unsigned coarse_sample = 1;
    for (; coarse_sample < 256; ++coarse_sample) {
        unsigned long long blocks = 0;
        for (int t = 0; t < n_tensors; ++t)
            blocks += (plans[t].m + (unsigned long long)kBlock * 8 * coarse_sample - 1) / ((unsigned long long)kBlock * 8 * coarse_sample);
        if (blocks <= (unsigned long long)sms * 4) break;
    }
    bool small_lists = true;
    for (int t = 0; t < n_tensors; ++t) small_lists = small_lists && plans[t].cap <= kSmallList;
    const size_t row_len = (size_t)n_tensors + 1;
    std::vector<Prob> probs((size_t)n_tensors);
    std::vector<uint32_t> prefix((size_t)WK_COUNT * row_len, 0u);
    {
        uint8_t *z = zero, *r = rest;
        for (int t = 0; t < n_tensors; ++t) {
            const TensorArgs a = {descs[t].update, descs[t].residual, descs[t].out_stream,
                                  descs[t].out_capacity, descs[t].out_mu};
            probs[t] = make_prob(a, plans[t], z, r);
            z += plans[t].zero_bytes;
            r += plans[t].rest_bytes;
            unsigned nb[WK_COUNT];
            block_counts(plans[t], sms, coarse_sample, nb);
            for (int kind = 0; kind < WK_COUNT; ++kind) {
                uint32_t* row = prefix.data() + (size_t)kind * row_len;
                const unsigned long long next = (unsigned long long)row[t] + nb[kind];
                if (next > 0x7fffffffull) return SBC_EINVAL;  // more blocks than one grid can hold
                row[t + 1] = (uint32_t)next;
            }
        }
    }

    {   // one-block kernels take the problems largest first
        uint32_t* perm = prefix.data() + (size_t)WK_PERM * row_len;
        for (int t = 0; t < n_tensors; ++t) perm[t] = (uint32_t)t;
        std::stable_sort(perm, perm + n_tensors, [&](uint32_t a, uint32_t b) { return plans[a].n > plans[b].n; });
        perm[n_tensors] = 0u;
    }

    cudaStream_t st = stream;
    if (cudaMemsetAsync(zero, 0, zero_total, st) != cudaSuccess) return SBC_ECUDA;
    // Descriptors and tables are adjacent in the workspace: one copy from a host buffer laid out
    // the same way.  The source is ordinary (pageable) memory, which the runtime reads out before
    // cudaMemcpyAsync returns, so the buffer may die with this call.
    {
        std::vector<uint8_t> image(probs_bytes + prefix.size() * 4, 0);
        std::memcpy(image.data(), probs.data(), probs.size() * sizeof(Prob));
        std::memcpy(image.data() + probs_bytes, prefix.data(), prefix.size() * 4);
        if (cudaMemcpyAsync(ws, image.data(), image.size(), cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SBC_ECUDA;
    }
    unsigned grid[WK_COUNT];
    const uint32_t* d_rows[WK_COUNT];
    for (int kind = 0; kind < WK_COUNT; ++kind) {
        d_rows[kind] = d_prefix + (size_t)kind * row_len;
        grid[kind] = prefix[(size_t)kind * row_len + (size_t)n_tensors];
    }
    k_zero_stream<<<grid[WK_STREAM], kBlock, 0, st>>>(Batch{d_probs, d_rows[WK_STREAM], (uint32_t)n_tensors, nullptr});
    unsigned long long k_total = 0, spans_total = 0;
    for (int t = 0; t < n_tensors; ++t) { k_total += (unsigned long long)plans[t].k; spans_total += plans[t].n_spans; }
    launch_encode(d_probs, (uint32_t)n_tensors, &probs[0].ctl->launch_exact, grid, d_rows, kModeBinary, false, small_lists, all_small,
                  k_total >= 16ull * spans_total && spans_total >= kDenseSpansMin, st, nullptr);
    return cudaGetLastError() == cudaSuccess ? SBC_OK : SBC_ECUDA;
}

// ---- sbc_encode_static: scratch that lives in the library image --------------------------
//
// File-scope device array used as the workspace of sbc_encode_static.  In host code this name is
// only a handle for the runtime, not a device address: the address is looked up per device with
// cudaGetSymbolAddress below and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_workspace[SBC_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};  // device address of g_static_workspace, per device ordinal

// Device address of the static workspace on the current device; looked up on first use.
int static_workspace_ptr(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SBC_ECUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) return SBC_ECUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return SBC_OK;
}
}  // namespace

int sbc_encode_static(const float* update, float* residual, int64_t numel, double p, void* out_stream,
                      size_t out_capacity, float* out_mu, sbc_cuda_stream_t stream) {
    const size_t need = sbc_workspace_bytes(numel, p);
    if (need == 0) return SBC_EINVAL;
    if (need > (size_t)SBC_STATIC_WORKSPACE_BYTES) return SBC_ECAPACITY;  // problem too large for the fixed scratch
    void* ws = nullptr;
    const int rc = static_workspace_ptr(&ws);
    if (rc != SBC_OK) return rc;
    // Same launches as sbc_encode; they clear the control block, histograms, tile counters and payload area
    // themselves, so stale contents of the shared array from an earlier call do not matter.
    return sbc_encode(update, residual, numel, p, out_stream, out_capacity, out_mu, ws,
                      (size_t)SBC_STATIC_WORKSPACE_BYTES, stream);
}

int sbc_encode_launches(void) { return 9; }  // set-up, 2 sample, 1 collect, 1 exact route, 2 select + sums, 2 ordering + Golomb

int sbc_decode_launches(int n_clients) {
    return n_clients <= 0 ? 0 : (n_clients + kMaxClientsPerLaunch - 1) / kMaxClientsPerLaunch;
}

int sbc_debug_barrier_timeout(uint32_t* scratch_dev, sbc_cuda_stream_t stream) {
    if (!scratch_dev || ((uintptr_t)scratch_dev & 3)) return SBC_EINVAL;
    if (cudaMemsetAsync(scratch_dev, 0, 8, stream) != cudaSuccess) return SBC_ECUDA;
    k_debug_barrier_timeout<<<2, kBlock, 0, stream>>>(scratch_dev, scratch_dev + 1);
    return cudaGetLastError() == cudaSuccess ? SBC_OK : SBC_ECUDA;
}

int sbc_encode_diag_get(const void* workspace, sbc_encode_diag* host_out, sbc_cuda_stream_t stream) {
    if (!workspace || !host_out) return SBC_EINVAL;
    Plan pl;
    make_plan(1024, 0.5, &pl);  // the control block sits at a fixed offset
    Prob P;
    Ctl c;
    const uint8_t* ws = static_cast<const uint8_t*>(workspace);
    if (cudaMemcpyAsync(&P, ws, sizeof(P), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemcpyAsync(&c, ws + kProbSlotBytes + pl.off_ctl, sizeof(c), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return SBC_ECUDA;
    host_out->status = c.status;
    host_out->exact_route = (c.use_fallback || c.regathered) ? 1u : 0u;
    host_out->candidates[0] = c.cand_cnt[0];
    host_out->candidates[1] = c.cand_cnt[1];
    host_out->capacity = P.cap;
    host_out->bound_lo = c.lo_f;
    host_out->bound_hi = c.hi_f;
    host_out->mu_pos = c.mu64[0];
    host_out->mu_neg = c.mu64[1];
    for (int s = 0; s < 2; ++s) host_out->certain[s] = c.use_fallback ? 0u : c.sure_cnt[s];
    host_out->regathered = c.regathered;
    return SBC_OK;
}

// Page-locked landing pad for the few bytes the host-buffer calls read back (a header, a status
// word), one per host thread, allocated on the thread's first such call and kept.  A device-to-host
// copy into ordinary (pageable) memory makes the driver wait for the stream inside the copy call,
// which kept a second thread's transfers from being enqueued meanwhile; with the pad the calls only
// ever wait in cudaStreamSynchronize.  Null if the allocation failed: the callers then fall back
// to a buffer on their stack.
static uint8_t* landing_pad() {
    thread_local uint8_t* pad = nullptr;
    thread_local bool tried = false;
    if (!tried) {
        tried = true;
        void* q = nullptr;
        if (cudaHostAlloc(&q, 256, cudaHostAllocDefault) == cudaSuccess) pad = static_cast<uint8_t*>(q);
        else (void)cudaGetLastError();
    }
    return pad;
}

// Small transfers between page-locked host memory and the device are done by a kernel, not by
// the copy engines: a copy engine works through its queue in order, so a header or a container of
// a few MB enqueued behind another stream's multi-GB transfer in the same direction would wait for
// all of it, and two host-buffer calls running on two streams would take turns instead of using
// both directions of the link at once.
static bool kernel_visible(const void* p, void** dev_view) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    if (a.type != cudaMemoryTypeHost && a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeManaged) return false;
    if (!a.devicePointer) return false;
    *dev_view = a.devicePointer;
    return true;
}
// dst <- src, `bytes` bytes, either side in device memory or page-locked host memory; falls back
// to the copy engine when a side is ordinary host memory.
static cudaError_t small_copy(void* dst, const void* src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st) {
    if (bytes == 0) return cudaSuccess;
    void *d = nullptr, *s = nullptr;
    if (!kernel_visible(dst, &d) || !kernel_visible(src, &s)) return cudaMemcpyAsync(dst, src, bytes, kind, st);
    const unsigned blocks = (unsigned)std::min<size_t>((bytes + kBlock * 16 - 1) / (kBlock * 16), (size_t)sm_count() * 4);
    k_copy_bytes<<<blocks, kBlock, 0, st>>>(static_cast<uint8_t*>(d), static_cast<const uint8_t*>(s), bytes);
    return cudaGetLastError();
}

int sbc_encode_host(const float* update_host, float* update_dev, float* residual_dev, int64_t numel,
                    double p, void* out_stream_host, void* stream_dev, size_t out_capacity,
                    size_t* out_bytes_host, float* out_mu_host, void* workspace, size_t workspace_bytes,
                    sbc_cuda_stream_t stream) {
    if (!update_host || !update_dev || !out_stream_host || !stream_dev || !out_bytes_host || numel <= 0)
        return SBC_EINVAL;
    // every check the host can make comes before the first copy is enqueued
    if (!workspace || ((uintptr_t)workspace & 255)) return SBC_EINVAL;
    Plan pl;
    if (!make_plan(numel, p, &pl)) return SBC_EINVAL;
    {
        const TensorArgs a = {update_dev, residual_dev, stream_dev, out_capacity, nullptr};
        const int arc = check_tensor(a, pl);
        if (arc != SBC_OK) return arc;
    }
    if (workspace_bytes < pl.total) return SBC_ECAPACITY;
    if (cudaMemcpyAsync(update_dev, update_host, (size_t)numel * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return SBC_ECUDA;
    float* mu_dev = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + kProbSlotBytes + pl.zero_bytes + pl.off_mu);
    const int rc = sbc_encode(update_dev, residual_dev, numel, p, stream_dev, out_capacity, mu_dev,
                              workspace, workspace_bytes, stream);
    if (rc != SBC_OK) return rc;
    sbc_stream_info info;
    const int irc = sbc_stream_info_get(stream_dev, &info, stream);  // synchronises
    if (irc != SBC_OK) return irc;
    if (info.total_bytes > out_capacity) return SBC_ECAPACITY;
    if (small_copy(out_stream_host, stream_dev, info.total_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return SBC_ECUDA;
    *out_bytes_host = info.total_bytes;
    if (out_mu_host) *out_mu_host = info.mu;  // the header carries the value out_mu received
    return SBC_OK;
}

int sbc_stream_info_get(const void* stream_dev, sbc_stream_info* host_out, sbc_cuda_stream_t stream) {
    if (!stream_dev || !host_out) return SBC_EINVAL;
    uint8_t on_stack[SBC_HEADER_BYTES];
    uint8_t* pad = landing_pad();
    uint8_t* h = pad ? pad : on_stack;
    if (small_copy(h, stream_dev, SBC_HEADER_BYTES, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return SBC_ECUDA;
    sbc_stream_info& o = *host_out;
    std::memcpy(&o.magic, h + 0, 4);
    std::memcpy(&o.version, h + 4, 4);
    std::memcpy(&o.numel, h + 8, 8);
    std::memcpy(&o.k, h + 16, 8);
    std::memcpy(&o.nbits, h + 24, 8);
    std::memcpy(&o.payload_offset, h + 32, 8);
    std::memcpy(&o.b, h + 40, 4);
    std::memcpy(&o.side, h + 44, 4);
    std::memcpy(&o.mu, h + 48, 4);
    std::memcpy(&o.chunk_codewords, h + 52, 4);
    std::memcpy(&o.n_chunks, h + 56, 4);
    std::memcpy(&o.status, h + 60, 4);
    o.total_bytes = o.payload_offset + align_up((size_t)((o.nbits + 7) / 8), 16);
    if (o.magic != SBC_MAGIC || o.version != SBC_VERSION) return SBC_ECORRUPT;
    if (o.status & SBC_STATUS_NONFINITE) return SBC_ENONFINITE;
    if (o.status & SBC_STATUS_TIMEOUT) return SBC_ETIMEOUT;
    if (o.status) return SBC_ECORRUPT;
    return SBC_OK;
}

// Common body of the decode entry points.  `stream_bytes` may be null (sizes not stated).
static int decode_impl(const void* const* streams, const size_t* stream_bytes, int n_clients, float scale,
                       float* out_dense, float* momentum, int64_t numel, uint32_t* status_dev,
                       sbc_cuda_stream_t stream) {
    if (!(scale == scale) || std::isinf(scale) || ((uintptr_t)momentum & 3)) return SBC_EINVAL;
    if (n_clients < 0 || numel <= 0 || numel >= (1ll << 31) || !out_dense) return SBC_EINVAL;
    if (n_clients > 0 && !streams) return SBC_EINVAL;
    if (((uintptr_t)out_dense & 3) || ((uintptr_t)status_dev & 3)) return SBC_EINVAL;
    for (int c = 0; c < n_clients; ++c) {
        if (!streams[c] || ((uintptr_t)streams[c] & 15)) return SBC_EINVAL;
        if (stream_bytes && stream_bytes[c] < SBC_HEADER_BYTES) return SBC_EINVAL;  // not even a header
    }
    const unsigned sms = (unsigned)sm_count();
    for (int first = 0; first < n_clients; first += kMaxClientsPerLaunch) {
        DecodeArgs a;
        std::memset(&a, 0, sizeof(a));
        a.n_clients = std::min(kMaxClientsPerLaunch, n_clients - first);
        for (int c = 0; c < a.n_clients; ++c) {
            a.streams[c] = static_cast<const uint8_t*>(streams[first + c]);
            a.bytes[c] = stream_bytes ? (unsigned long long)stream_bytes[first + c] : 0ull;
        }
        a.out = out_dense;
        a.n = numel;
        a.status = status_dev;
        a.scale = scale;
        a.momentum = momentum;
        // at most max_chunks_upto(numel) chunks per client, 32 chunks per warp, two warps per block
        const unsigned long long max_groups =
            (unsigned long long)a.n_clients * ((max_chunks_upto((unsigned long long)numel) + 31ull) / 32ull);
        const unsigned grid = grid_for(max_groups, kDecodeThreads / 32, sms * 5);
        k_decode_accumulate<<<grid, kDecodeThreads, 0, stream>>>(a);
    }
    return cudaGetLastError() == cudaSuccess ? SBC_OK : SBC_ECUDA;
}

int sbc_decode_accumulate(const void* const* streams, int n_clients, float* out_dense, int64_t numel,
                          uint32_t* status_dev, sbc_cuda_stream_t stream) {
    return decode_impl(streams, nullptr, n_clients, 1.0f, out_dense, nullptr, numel, status_dev, stream);
}

int sbc_decode_accumulate_sized(const void* const* streams, const size_t* stream_bytes, int n_clients,
                                float* out_dense, int64_t numel, uint32_t* status_dev, sbc_cuda_stream_t stream) {
    if (n_clients > 0 && !stream_bytes) return SBC_EINVAL;
    return decode_impl(streams, stream_bytes, n_clients, 1.0f, out_dense, nullptr, numel, status_dev, stream);
}

int sbc_decode_apply(const void* const* streams, int n_clients, float scale, float* out_dense, float* momentum,
                     int64_t numel, uint32_t* status_dev, sbc_cuda_stream_t stream) {
    return decode_impl(streams, nullptr, n_clients, scale, out_dense, momentum, numel, status_dev, stream);
}

int sbc_decode_apply_sized(const void* const* streams, const size_t* stream_bytes, int n_clients, float scale,
                           float* out_dense, float* momentum, int64_t numel, uint32_t* status_dev,
                           sbc_cuda_stream_t stream) {
    if (n_clients > 0 && !stream_bytes) return SBC_EINVAL;
    return decode_impl(streams, stream_bytes, n_clients, scale, out_dense, momentum, numel, status_dev, stream);
}

size_t sbc_decode_workspace_bytes_batch(int n_tensors) {
    return n_tensors > 0 ? align_up((size_t)n_tensors * sizeof(DecodeArgs), 256) : 0;
}

int sbc_decode_accumulate_batch(int n_tensors, int n_clients, const sbc_decode_desc* descs, uint32_t* status_dev,
                                void* workspace, size_t workspace_bytes, sbc_cuda_stream_t stream) {
    if (n_tensors <= 0 || n_tensors > 65535 || n_clients <= 0 || n_clients > kMaxClientsPerLaunch || !descs ||
        !workspace || ((uintptr_t)workspace & 255) || ((uintptr_t)status_dev & 3))
        return SBC_EINVAL;
    if (workspace_bytes < sbc_decode_workspace_bytes_batch(n_tensors)) return SBC_ECAPACITY;
    long long max_numel = 0;
    for (int t = 0; t < n_tensors; ++t) {
        const sbc_decode_desc& d = descs[t];
        if (!d.streams || !d.out_dense || ((uintptr_t)d.out_dense & 3) || d.numel <= 0 || d.numel >= (1ll << 31))
            return SBC_EINVAL;
        for (int c = 0; c < n_clients; ++c) {
            if (!d.streams[c] || ((uintptr_t)d.streams[c] & 15)) return SBC_EINVAL;
            if (d.stream_bytes && d.stream_bytes[c] < SBC_HEADER_BYTES) return SBC_EINVAL;
        }
        max_numel = std::max<long long>(max_numel, d.numel);
    }
    // one copy of all argument blocks from an ordinary host buffer (read out before the call returns)
    DecodeArgs* d_args = static_cast<DecodeArgs*>(workspace);
    {
        std::vector<DecodeArgs> args((size_t)n_tensors);
        std::memset(static_cast<void*>(args.data()), 0, args.size() * sizeof(DecodeArgs));
        for (int t = 0; t < n_tensors; ++t) {
            args[t].n_clients = n_clients;
            for (int c = 0; c < n_clients; ++c) {
                args[t].streams[c] = static_cast<const uint8_t*>(descs[t].streams[c]);
                args[t].bytes[c] = descs[t].stream_bytes ? (unsigned long long)descs[t].stream_bytes[c] : 0ull;
            }
            args[t].out = descs[t].out_dense;
            args[t].n = descs[t].numel;
            args[t].status = status_dev;
            args[t].scale = 1.0f;
        }
        if (cudaMemcpyAsync(d_args, args.data(), args.size() * sizeof(DecodeArgs), cudaMemcpyHostToDevice,
                            stream) != cudaSuccess)
            return SBC_ECUDA;
    }
    const unsigned long long max_groups =
        (unsigned long long)n_clients * ((max_chunks_upto((unsigned long long)max_numel) + 31ull) / 32ull);
    const unsigned gx = grid_for(max_groups, kDecodeThreads / 32,
                                 std::max(16u, (unsigned)sm_count() * 5u / (unsigned)n_tensors));
    k_decode_accumulate_batch<<<dim3(gx, (unsigned)n_tensors), kDecodeThreads, 0, stream>>>(d_args);
    return cudaGetLastError() == cudaSuccess ? SBC_OK : SBC_ECUDA;
}

int sbc_decode_accumulate_host(const void* const* streams_host, const size_t* stream_bytes, int n_clients,
                               float* out_dense_host, float* dense_dev, int64_t numel, void* staging_dev,
                               size_t staging_bytes, uint32_t* status_host, sbc_cuda_stream_t stream) {
    if (n_clients < 0 || n_clients > 4096 || numel <= 0 || numel >= (1ll << 31) || !out_dense_host || !dense_dev ||
        !staging_dev)
        return SBC_EINVAL;
    if (n_clients > 0 && (!streams_host || !stream_bytes)) return SBC_EINVAL;
    if (((uintptr_t)staging_dev & 15) || ((uintptr_t)dense_dev & 3)) return SBC_EINVAL;
    // staging layout: one status word (16 bytes), then the containers
    size_t need = 16;
    for (int c = 0; c < n_clients; ++c) {
        if (!streams_host[c] || stream_bytes[c] < SBC_HEADER_BYTES) return SBC_EINVAL;
        need += align_up(stream_bytes[c], 16);
    }
    if (staging_bytes < need) return SBC_ECAPACITY;
    // The containers are in host memory: what their headers claim is compared with the bytes the
    // caller received, here, before anything is enqueued (the device repeats the check on its copy).
    for (int c = 0; c < n_clients; ++c) {
        const uint8_t* h = static_cast<const uint8_t*>(streams_host[c]);
        uint32_t magic, version;
        unsigned long long hdr_numel, nbits, payload_offset;
        std::memcpy(&magic, h + 0, 4);
        std::memcpy(&version, h + 4, 4);
        std::memcpy(&hdr_numel, h + 8, 8);
        std::memcpy(&nbits, h + 24, 8);
        std::memcpy(&payload_offset, h + 32, 8);
        const bool fits = nbits <= (1ull << 40) && payload_offset <= (unsigned long long)stream_bytes[c] &&
                          payload_offset + align_up((size_t)((nbits + 7) / 8), 16) <= (unsigned long long)stream_bytes[c];
        if (magic != SBC_MAGIC || version != SBC_VERSION || hdr_numel != (unsigned long long)numel || !fits) {
            if (status_host) *status_host = SBC_STATUS_CORRUPT;
            return SBC_ECORRUPT;
        }
    }
    uint8_t* base = static_cast<uint8_t*>(staging_dev);
    std::vector<const void*> dev_ptrs((size_t)std::max(n_clients, 1));
    size_t off = 16;
    if (cudaMemsetAsync(base, 0, 16, stream) != cudaSuccess ||
        cudaMemsetAsync(dense_dev, 0, (size_t)numel * 4, stream) != cudaSuccess)
        return SBC_ECUDA;
    for (int c = 0; c < n_clients; ++c) {
        if (small_copy(base + off, streams_host[c], stream_bytes[c], cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return SBC_ECUDA;
        dev_ptrs[c] = base + off;
        off += align_up(stream_bytes[c], 16);
    }
    const int rc = sbc_decode_accumulate_sized(dev_ptrs.data(), stream_bytes, n_clients, dense_dev, numel,
                                               reinterpret_cast<uint32_t*>(base), stream);
    if (rc != SBC_OK) return rc;
    uint32_t on_stack = 0;
    uint8_t* pad = landing_pad();
    uint32_t* landed = pad ? reinterpret_cast<uint32_t*>(pad + 128) : &on_stack;
    if (cudaMemcpyAsync(out_dense_host, dense_dev, (size_t)numel * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        small_copy(landed, base, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return SBC_ECUDA;
    const uint32_t status = *landed;
    if (status_host) *status_host = status;
    return status ? SBC_ECORRUPT : SBC_OK;
}

}  // extern "C"
