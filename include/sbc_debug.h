/*
 * sbc_debug.h -- instruments of the SBC library: what a call did, how many
 * kernels it launched.  Not part of the method (the paper has no counterpart);
 * used by the tests to see which route an encode took and by the benchmark to
 * count launches.  Exported by the same shared library as sbc.h.
 */
#ifndef SBC_DEBUG_H
#define SBC_DEBUG_H

#include "sbc.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernels one sbc_encode call launches for a tensor whose candidate
 * lists are longer than one thread block handles (memsets not counted; a tensor
 * with 2*k + 1024 <= 8192 and k <= 4096 takes a shorter chain of 11), and
 * one sbc_decode_accumulate call for n_clients streams. */
int sbc_encode_launches(void);
int sbc_decode_launches(int n_clients);

/* What the last sbc_encode that used `workspace` did; synchronises `stream`.
 * workspace: the device pointer that call was given (read only here). */
typedef struct sbc_encode_diag {
    uint32_t status;        /* SBC_STATUS_* bits */
    uint32_t exact_route;   /* 1 if the candidate lists were rebuilt by the exact route */
    uint32_t candidates[2]; /* entries gathered per side (>= k) */
    uint32_t capacity;      /* most candidates a side may have */
    float bound_lo, bound_hi; /* candidates were: value >= bound_lo, value <= bound_hi */
    double mu_pos, mu_neg;  /* the two means of Algorithm 2 */
    uint32_t certain[2];    /* of the candidates, those at or above the sample's upper bound of the
                               threshold (kept, and summed, without being looked at by the exact
                               selection); 0 after the exact route */
    uint32_t regathered;    /* exact route only: 1 if the sample's bounds held and only the gathering
                               was redone (candidates too unevenly spread for the streaming pass's
                               per-warp regions), 0 if the thresholds were searched over the whole tensor */
} sbc_encode_diag;
int sbc_encode_diag_get(const void *workspace, sbc_encode_diag *host_out, sbc_cuda_stream_t stream);

/* The one device-side wait of the library is the barrier between the steps of
 * the exact route's kernel; it gives up after a bounded number of polls (about a
 * quarter of a second) and the affected streams then carry SBC_STATUS_TIMEOUT.
 * This call shows the bound at work without damaging anything: it enqueues a
 * two-block kernel whose barrier waits for a third block that does not exist.
 * scratch_dev: device, two uint32 (zeroed by the call); when the stream has run,
 * scratch_dev[1] holds SBC_STATUS_TIMEOUT.  Asynchronous. */
int sbc_debug_barrier_timeout(uint32_t *scratch_dev, sbc_cuda_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* SBC_DEBUG_H */
