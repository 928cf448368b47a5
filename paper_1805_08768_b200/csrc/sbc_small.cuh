// Back half of sbc_encode for problems whose candidate lists hold at most kSmallList entries
// (every tensor of a ResNet-sized layer at p = 0.001): everything after the candidate pass in ONE
// kernel, two blocks per problem (one per side).  Each block finds its side's k-th largest
// composite and the exact sum of the kept values (Algorithm 2); the block that finishes second
// takes the side decision and goes on alone: kept positions in ascending order, residual
// write-back (Algorithm 1), Golomb code, chunk table and header (Algorithm 3).  Same results as the
// general kernels, which a launch uses as soon as one of its lists is longer.
#pragma once
#include "sbc_common.cuh"
#include "sbc_golomb.cuh"
#include "sbc_select.cuh"
#include "../../include/sbc.h"

namespace sbc {

constexpr uint32_t kSmallKept = 16 * kBlock;  // positions one block orders in registers (k <= (kSmallList - 1024) / 2)
static_assert((kSmallList - 1024u) / 2u <= kSmallKept, "a short list keeps at most kSmallKept positions");

// One block per problem and side (grid.z = side).
__global__ void __launch_bounds__(kBlock) k_small_finish(const Batch B) {
    __shared__ Prob s_prob;
    const Slot S = resolve(B, &s_prob);
    const Prob& P = s_prob;
    Ctl* ctl = P.ctl;
    const int s = blockIdx.z;
    constexpr int kPer = (int)(kSmallList / kBlock);
    __shared__ uint32_t s_hist[kHistBins];
    __shared__ uint32_t s_scan[kBlock / 32 + 1];
    __shared__ unsigned long long s_scan64[kBlock / 32 + 1];
    __shared__ Pick s_pick;
    __shared__ unsigned long long s_result;
    __shared__ long long s_bins[256];
    __shared__ uint32_t s_pos[kSmallKept];
    __shared__ uint32_t s_count, s_status;
    __shared__ uint32_t s_nonzero[8];

    // ---- this side: threshold and exact sum (skipped when an earlier kernel reported an error;
    // one thread reads the status word, since the other side's block may set it meanwhile)
    if (threadIdx.x == 0) s_status = __ldcg(&ctl->status);
    __syncthreads();
    if (s_status == 0u) {
        const BandView view = band_view(P, ctl, s);   // short lists have no upper bound: every candidate is in the band
        const uint32_t cnt = view.count, rank = view.rank;
        unsigned long long thr = 0ull;
        const SelectDigits dg = select_digits(ctl, s);
        bool good = cnt <= kSmallList;  // what the host checked through the capacity
        unsigned long long c[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const uint32_t i = (uint32_t)j * kBlock + threadIdx.x;
            c[j] = (good && i < cnt) ? view.src[i] - dg.sub : 0ull;
        }
        unsigned long long bits = 0ull;
#pragma unroll
        for (int j = 0; j < kPer; ++j) bits |= c[j];
        const int top = min(dg.top, block_top_bit(bits, s_scan64));
        good = good && block_select_registers<kPer>(c, cnt, rank, top, 0, 0ull, s_hist, s_scan, &s_pick, &s_result, &thr);
        thr += dg.sub;
        if (!good) {
            if (threadIdx.x == 0) atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
        } else {
            // exact sum of the kept values: 24-bit integers into one 64-bit bin per exponent.  Nearly
            // all kept values lie within eight binades of the threshold's: those are summed in one
            // register per thread, in units of the lowest of these binades (a 64-bit shared-memory
            // atomic is a compare-and-swap loop, and thousands of them on one bin take turns).
            s_bins[threadIdx.x] = 0ll;
            __syncthreads();
            const uint32_t thr_bits = bits_of_key(side_key(s, (uint32_t)(thr >> 32)));
            const int bin_a = max((int)((thr_bits >> 23) & 0xffu) - 1, 0);
            long long acc_a = 0;
            const unsigned long long thr_rel = thr - dg.sub;   // the entries are still in the registers, with dg.sub taken off
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                if ((uint32_t)j * kBlock + threadIdx.x >= cnt || c[j] < thr_rel) continue;
                const uint32_t bits = bits_of_key(side_key(s, (uint32_t)((c[j] + dg.sub) >> 32)));
                const uint32_t ex = (bits >> 23) & 0xffu;
                int m = (int)(bits & 0x7fffffu) | (ex ? 0x800000 : 0);
                if (bits >> 31) m = -m;
                const int bin = ex ? (int)ex - 1 : 0;
                const uint32_t up = (uint32_t)(bin - bin_a);
                if (up < 8u) acc_a += (long long)m << up;  // |m| < 2^24: at most 2^31 per entry
                else atomicAdd(reinterpret_cast<unsigned long long*>(&s_bins[bin]), (unsigned long long)(long long)m);
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) acc_a += __shfl_down_sync(0xffffffffu, acc_a, d);
            if (lane_id() == 0 && acc_a)
                atomicAdd(reinterpret_cast<unsigned long long*>(&s_bins[bin_a]), (unsigned long long)acc_a);
            __syncthreads();
            bins_nonzero_masks(s_bins[threadIdx.x], s_nonzero);
            __syncthreads();
            if (threadIdx.x == 0) {
                const double sum = bins_to_double(s_bins, s_nonzero);
                ctl->thr[s] = thr;
                ctl->mu64[s] = s ? -sum / (double)P.k : sum / (double)P.k;  // val- holds the negated entries
            }
        }
    }
    // ---- the block that gets here second goes on alone
    if (!last_block_ticket(&ctl->done[ST_SUM], 2u)) return;
    if (__ldcg(&ctl->status) != 0u) {
        if (threadIdx.x == 0) write_header(P, ctl, false, 0ull);
        return;
    }
    const double mu_pos = __ldcg(&ctl->mu64[0]), mu_neg = __ldcg(&ctl->mu64[1]);
    const uint32_t side = (mu_pos >= mu_neg) ? 0u : 1u;
    const float mu = side ? (float)(-mu_neg) : (float)mu_pos;
    const uint32_t k = (uint32_t)P.k;
    if (threadIdx.x == 0) {
        ctl->side = side;
        ctl->mu32 = mu;
        ctl->k_final = k;
        if (P.out_mu) *P.out_mu = mu;
        s_count = 0u;
    }
    // ---- kept positions of the chosen side, ascending: gathered into shared memory in any order,
    // padded with 0xffffffff, sorted in registers (thread t ends up with positions 16 t .. 16 t + 15
    // of the ascending list, which are the codewords it writes below)
    for (uint32_t i = threadIdx.x; i < kSmallKept; i += kBlock) s_pos[i] = 0xffffffffu;
    __syncthreads();
    {
        const BandView view = band_view(P, ctl, (int)side);
        const uint32_t total = min(view.count, kSmallList);
        const unsigned long long thr = __ldcg(&ctl->thr[side]);
        constexpr int kLoads = 4;  // list entries in flight per thread
        for (uint32_t base = 0; base < total; base += kBlock * kLoads) {
            unsigned long long e[kLoads];
#pragma unroll
            for (int j = 0; j < kLoads; ++j) {
                const uint32_t i = base + j * kBlock + threadIdx.x;
                e[j] = (i < total) ? view.src[i] : 0ull;
            }
#pragma unroll
            for (int j = 0; j < kLoads; ++j) {  // one slot reservation per warp and step
                const bool kept = base + j * kBlock + threadIdx.x < total && e[j] >= thr;
                const unsigned mask = __ballot_sync(0xffffffffu, kept);
                uint32_t first = 0u;
                if (lane_id() == 0 && mask) first = atomicAdd(&s_count, (uint32_t)__popc(mask));
                first = __shfl_sync(0xffffffffu, first, 0);
                const uint32_t slot = first + (uint32_t)__popc(mask & ((1u << lane_id()) - 1u));
                if (kept && slot < kSmallKept) s_pos[slot] = composite_index(e[j]);
            }
        }
    }
    __syncthreads();
    if (s_count != k) {  // uniform
        if (threadIdx.x == 0) {
            atomicOr(&ctl->status, SBC_STATUS_INTERNAL);
            write_header(P, ctl, false, 0ull);
        }
        return;
    }
    constexpr int kCw = 16;  // codewords per thread, consecutive
    uint32_t pos[kCw];
#pragma unroll
    for (int r = 0; r < kCw; ++r) pos[r] = s_pos[r * kBlock + threadIdx.x];
    __syncthreads();
    block_sort<16>(pos, s_pos);
    const uint32_t i0 = threadIdx.x * kCw;
#pragma unroll
    for (int j = 0; j < kCw; ++j) s_pos[i0 + j] = pos[j];  // the ascending list, for the neighbours and the chunk table
    __syncthreads();
    // ---- residual write-back, code lengths, bit offsets, payload, chunk table, header
    const int b = P.b;
    uint32_t gap[kCw];
    float r[kCw];
    unsigned long long len_sum = 0ull;
#pragma unroll
    for (int j = 0; j < kCw; ++j) r[j] = (i0 + j < k) ? P.residual[pos[j]] : 0.f;  // all loads in flight together
    long long prev = i0 ? (long long)s_pos[i0 - 1] : -1ll;
#pragma unroll
    for (int j = 0; j < kCw; ++j) {
        const uint32_t i = i0 + j;
        gap[j] = 0u;
        if (i < k) {
            P.residual[pos[j]] = __fsub_rn(r[j], mu);
            gap[j] = (uint32_t)((long long)pos[j] - prev - 1);
            prev = (long long)pos[j];
            len_sum += (unsigned long long)(gap[j] >> b) + 1ull + (unsigned long long)b;
        }
    }
    unsigned long long nbits;
    unsigned long long off = block_exclusive_scan<unsigned long long>(len_sum, s_scan64, &nbits);
    uint32_t* words = reinterpret_cast<uint32_t*>(P.stream + P.payload_offset);
    uint8_t* table = P.stream + SBC_HEADER_BYTES;
    // A payload of at most 2048 words is put together in shared memory (the histogram's, free by
    // now) and stored once: thousands of atomics from one block on global memory take longer
    // than everything else here.  Longer payloads are ORed into the zeroed stream directly.
    const bool in_shared = nbits <= 32ull * kHistBins;  // uniform
    if (in_shared) {
        for (int w = threadIdx.x; w < kHistBins; w += kBlock) s_hist[w] = 0u;
        __syncthreads();
    }
    uint32_t* target = in_shared ? s_hist : words;
#pragma unroll
    for (int j = 0; j < kCw; ++j) {
        const uint32_t i = i0 + j;
        if (i < k) {
            pack_codeword(target, table, P.chunk_cw, i, off, gap[j], b, i ? s_pos[i - 1] + 1u : 0u);
            off += (unsigned long long)(gap[j] >> b) + 1ull + (unsigned long long)b;
        }
    }
    if (in_shared) {
        __syncthreads();
        const uint32_t n_words = (uint32_t)((nbits + 31ull) >> 5);
        for (uint32_t w = threadIdx.x; w < n_words; w += kBlock) words[w] = s_hist[w];
    }
    if (threadIdx.x == 0) {
        ctl->kept_total = k;
        write_header(P, ctl, true, nbits);
    }
}

}  // namespace sbc
