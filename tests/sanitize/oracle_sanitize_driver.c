/* Runs the CPU oracle over a few seeded tensors under AddressSanitizer and
 * UndefinedBehaviorSanitizer (built by tests/test_oracle_sanitizers.py from
 * this file and oracle/sbc_oracle.c).  It checks only what a memory or
 * arithmetic fault would break: that every call returns success and that the
 * decoded tensor is the binarised update.  Exit code 0 = clean run. */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "../../oracle/sbc_oracle.h"

static uint64_t state = 0x9E3779B97F4A7C15ull;
static double uniform01(void) {
    state ^= state << 13; state ^= state >> 7; state ^= state << 17;
    return (double)(state >> 11) / 9007199254740992.0;
}
static float normal(void) {
    double u = uniform01(), v = uniform01();
    if (u < 1e-300) u = 1e-300;
    return (float)(sqrt(-2.0 * log(u)) * cos(6.283185307179586 * v));
}

static int run_case(int64_t n, double p, int kind) {
    float *upd = malloc((size_t)n * sizeof(float)), *res = malloc((size_t)n * sizeof(float));
    float *dense = calloc((size_t)n, sizeof(float)), *a = malloc((size_t)n * sizeof(float));
    size_t cap = sbc_oracle_stream_bytes(n, p);
    uint8_t *out = malloc(cap);
    if (!upd || !res || !dense || !a || !out) return 10;
    for (int64_t i = 0; i < n; ++i) {
        upd[i] = kind == 1 ? 0.0f : kind == 2 ? (float)((i * 7) % 5) - 2.0f : normal() * 1e-3f;
        res[i] = kind == 3 ? normal() * 1e-3f : 0.0f;
        a[i] = res[i] + upd[i];
    }
    size_t len = 0;
    float mu = 0.0f;
    int rc = sbc_oracle_encode(upd, res, n, p, out, cap, &len, &mu);
    if (rc != 0 || len == 0 || len > cap) return 11;
    const uint8_t *streams[2] = {out, out};
    if (sbc_oracle_decode_accumulate(streams, 2, dense, n) != 0) return 12;
    int64_t k = sbc_oracle_kept_count(n, p), seen = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (dense[i] != 0.0f || (mu == 0.0f && res[i] != a[i])) ++seen;
        if (dense[i] != 0.0f && dense[i] != mu + mu) return 13;           /* two clients, same message */
        if (dense[i] == 0.0f && mu != 0.0f && res[i] != a[i]) return 14;  /* residual untouched off the kept set */
    }
    if (mu != 0.0f && seen != k) return 15;
    /* the two variants and the apply step, for their own buffers' sake */
    size_t vcap = sbc_oracle_stream_bytes_values(n, p), vlen = 0;
    uint8_t *vout = malloc(vcap);
    if (!vout || sbc_oracle_encode_values(upd, res, n, p, vout, vcap, &vlen) != 0 || vlen > vcap) return 16;
    float *w = calloc((size_t)n, sizeof(float)), *m = calloc((size_t)n, sizeof(float));
    const uint8_t *one[1] = {out};
    if (!w || !m || sbc_oracle_decode_apply(one, 1, 0.25f, w, m, n) != 0) return 17;
    free(upd); free(res); free(dense); free(a); free(out); free(vout); free(w); free(m);
    return 0;
}

int main(void) {
    const int64_t sizes[] = {1, 2, 31, 257, 4097, 70001, 300000};
    const double ps[] = {0.5, 0.1, 0.01, 0.001};
    for (size_t s = 0; s < sizeof(sizes) / sizeof(sizes[0]); ++s)
        for (size_t q = 0; q < sizeof(ps) / sizeof(ps[0]); ++q)
            for (int kind = 0; kind < 4; ++kind) {
                int rc = run_case(sizes[s], ps[q], kind);
                if (rc != 0) {
                    fprintf(stderr, "case n=%lld p=%g kind=%d failed with %d\n", (long long)sizes[s], ps[q], kind, rc);
                    return rc;
                }
            }
    puts("oracle clean under ASan/UBSan");
    return 0;
}
