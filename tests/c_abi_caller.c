/*
 * A caller of the C ABI written in plain C: no Python, no C++ and no torch in
 * the process.  It allocates g and d with the CUDA runtime, runs gac_init /
 * gac_stats / gac_project / gac_free on hand-derived cases (small integer
 * vectors pushed by hand through the App. A.1 cosine, the Algorithm 1 branches,
 * Eq. 5 and the rank-one form of App. A.2; the same cases as
 * tests/golden/worked_examples.txt) and compares every output.  Exits 0 and
 * prints "ok" when everything matches.
 */
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "gac.h"

#define CHECK(cond, msg)                                         \
    do {                                                         \
        if (!(cond)) {                                           \
            fprintf(stderr, "FAILED %s: %s\n", name, msg);       \
            return 1;                                            \
        }                                                        \
    } while (0)

static int run_case(const char *name, double c_low, double c_high, const float d0[4], const float g0[4],
                    double dot, double gg, double dd, double cosine, int regime, double alpha, double coef,
                    const double g_out[4], int exchange) {
    float *g = NULL, *d = NULL;
    if (cudaMalloc((void **)&g, 4 * sizeof(float)) != cudaSuccess) return 2;
    if (cudaMalloc((void **)&d, 4 * sizeof(float)) != cudaSuccess) return 2;
    cudaMemcpy(g, g0, 4 * sizeof(float), cudaMemcpyHostToDevice);
    cudaMemcpy(d, d0, 4 * sizeof(float), cudaMemcpyHostToDevice);

    gac_hparams hp;
    gac_default_hparams(&hp);
    hp.c_low = c_low;
    hp.c_high = c_high;
    hp.eps = 0.0;
    hp.state_mode = exchange ? GAC_STATE_EXCHANGE : GAC_STATE_RAW;
    gac_tensor t;
    t.g = g;
    t.d = d;
    t.numel = 4;
    gac_ctx *ctx = NULL;
    int rc = gac_init(&ctx, &t, 1, GAC_F32, GAC_F32, &hp, 0);
    if (rc != GAC_OK) fprintf(stderr, "gac_init: %s\n", gac_last_error(NULL));
    CHECK(rc == GAC_OK, "gac_init");

    gac_result r, after;
    rc = gac_stats(ctx, 2, 0, NULL, &r);
    CHECK(rc == GAC_OK, gac_last_error(ctx));
    CHECK(r.dot == dot && r.gg == gg && r.dd == dd, "sums (exact small integers)");
    CHECK(fabs(r.cos - cosine) <= 1e-15 * fabs(cosine), "cosine");
    CHECK(r.regime == regime, "regime");
    CHECK(fabs(r.alpha - alpha) <= 1e-15 * alpha, "alpha");
    CHECK(fabs(r.coef64 - coef) <= 1e-15 * fabs(coef), "coefficient");
    rc = gac_project(ctx, NULL, NULL, &after);
    CHECK(rc == GAC_OK, gac_last_error(ctx));

    float g_host[4], d_host[4];
    cudaMemcpy(g_host, g, sizeof(g_host), cudaMemcpyDeviceToHost);
    cudaMemcpy(d_host, d, sizeof(d_host), cudaMemcpyDeviceToHost);
    const float *out = g_host, *state = d_host;   /* in place: g' in g, d' = g copied into d */
    if (exchange) {                               /* exchange: g untouched is the state, g' (if any) in d */
        state = g_host;
        out = (after.out_set == GAC_SET_D) ? d_host : g_host;
        CHECK((after.out_set == GAC_SET_D) == (regime == GAC_REGIME_PROJECT), "out_set");
        int next = -1;
        CHECK(gac_next_gradient_set(ctx, &next) == GAC_OK && next == GAC_SET_D, "roles swap after a step");
    }
    for (int i = 0; i < 4; ++i) {
        /* the coefficient is rounded once to binary32 before it multiplies d */
        const double tol = 6e-8 * fabs(g_out[i]) + ldexp(fabs(coef) * fabs((double)d0[i]), -24);
        CHECK(fabs((double)out[i] - g_out[i]) <= tol, "projected gradient");
        CHECK(state[i] == g0[i], "stored direction is the raw gradient");
    }
    CHECK(gac_free(ctx) == GAC_OK, "gac_free");
    cudaFree(g);
    cudaFree(d);
    return 0;
}

int main(void) {
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
        fprintf(stderr, "no CUDA device\n");
        return 3;
    }
    const float axis_d[4] = {1, 0, 0, 0}, axis_g[4] = {3, 4, 0, 0}, neg_g[4] = {-3, 4, 0, 0};
    const float diag_d[4] = {2, 2, 2, 2}, diag_g[4] = {5, 1, 1, 1};
    const double axis_out[4] = {1.5, 4, 0, 0}, axis_same[4] = {3, 4, 0, 0}, neg_out[4] = {-1.5, 4, 0, 0};
    const double diag_alpha = 0.33071891388307382;
    const double diag_out[4] = {3.6614378277661477, -0.33856217223385235, -0.33856217223385235,
                                -0.33856217223385235};
    int bad = 0;
    for (int exchange = 0; exchange < 2; ++exchange) {
        bad |= run_case("axis_project", 0.3, 0.9, axis_d, axis_g, 3, 25, 1, 0.6, GAC_REGIME_PROJECT, 0.5, -1.5,
                        axis_out, exchange);
        bad |= run_case("axis_violation", 0.3, 0.6, axis_d, axis_g, 3, 25, 1, 0.6, GAC_REGIME_VIOLATION, 1.0, 0.0,
                        axis_same, exchange);
        bad |= run_case("axis_safe", 0.6, 0.9, axis_d, axis_g, 3, 25, 1, 0.6, GAC_REGIME_SAFE, 1.0, 0.0, axis_same,
                        exchange);
        bad |= run_case("axis_negative", 0.3, 0.9, axis_d, neg_g, -3, 25, 1, -0.6, GAC_REGIME_PROJECT, 0.5, 1.5,
                        neg_out, exchange);
        bad |= run_case("diag_project", 0.25, 0.9, diag_d, diag_g, 16, 28, 16, 0.7559289460184544,
                        GAC_REGIME_PROJECT, diag_alpha, diag_alpha - 1.0, diag_out, exchange);
    }
    if (bad) return 1;
    printf("ok\n");
    return 0;
}
