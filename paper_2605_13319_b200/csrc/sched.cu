// Host side of the method the verify pass serves: PipeSD's token-batch pipeline model, the optimal batching of a
// speculative round's draft tokens, and the dual-threshold verification trigger.  Plain host code behind the same
// C ABI as the kernels (no device work here).
#include <math.h>

#include <vector>

#include "../../include/pipesd.h"

extern "C" {

int32_t pipesd_sched_round_time(int32_t N, double alpha, double beta, double gamma, const int32_t* boundaries, int32_t K,
                                double* T) {
    if (N < 1 || K < 1 || K > N || !boundaries || !T || boundaries[0] != 1) return PIPESD_E_INVALID;
    for (int k = 1; k < K; ++k)
        if (boundaries[k] <= boundaries[k - 1]) return PIPESD_E_INVALID;
    if (boundaries[K - 1] > N) return PIPESD_E_INVALID;
    // gen_end: when the batch's last token has been generated; tx_end: when its transmission has finished
    double gen_end = 0.0, tx_end = 0.0;
    for (int k = 0; k < K; ++k) {
        const int n = (k + 1 < K ? boundaries[k + 1] : N + 1) - boundaries[k];
        gen_end += gamma * n;
        const double tx_start = k == 0 ? gen_end : fmax(tx_end, gen_end);
        tx_end = tx_start + (alpha + beta * n);
    }
    *T = tx_end;
    return PIPESD_OK;
}

int32_t pipesd_sched_optimal_batching(int32_t N, double alpha, double beta, double gamma, int32_t* boundaries, int32_t* K,
                                      double* T) {
    if (N < 1 || N > 65536 || !boundaries || !K) return PIPESD_E_INVALID;
    // best[j]: earliest time at which the first j tokens can have been generated and sent; from[j]: tokens sent
    // before the batch that ends at token j.  A batch i+1..j can be sent once tokens up to j exist (gamma * j) and the
    // batches before it are through (best[i]).
    std::vector<double> best(N + 1, INFINITY);
    std::vector<int32_t> from(N + 1, -1);
    best[0] = 0.0;
    for (int j = 1; j <= N; ++j) {
        const double ready = gamma * j;
        for (int i = 0; i < j; ++i) {
            const double t = fmax(best[i], ready) + (alpha + beta * (j - i));
            if (t < best[j]) { best[j] = t; from[j] = i; }
        }
    }
    int n = 0;
    for (int p = N; p > 0; p = from[p]) ++n;
    *K = n;
    for (int p = N, k = n - 1; p > 0; p = from[p], --k) boundaries[k] = from[p] + 1;
    if (T) *T = best[N];
    return PIPESD_OK;
}

int32_t pipesd_sched_trigger_step(double* c1, double R1, double R2, double p, int32_t* fire) {
    if (!c1 || !fire || !(p >= 0.0 && p <= 1.0) || !(*c1 >= 0.0)) return PIPESD_E_INVALID;
    const double tentative = *c1 * p;
    const bool f = tentative <= R1 || p <= R2;
    *fire = f ? 1 : 0;
    *c1 = f ? 1.0 : tentative;
    return PIPESD_OK;
}

}  // extern "C"
