// gbs_search_clip_ratio: the bracket search of Algorithm 1 ("Gradual Binary Search", inner loop for one
// projection) driven by the library's own objective, the quantization error gbs_clip_error computes.
//
// Algorithm 1 evaluates one clip ratio per iteration and decides from the comparison f_x < f_m how the
// bracket [a, b] and the kept point m move.  Each evaluation here is a pass over the whole activation
// tensor, so the driver does not run them one by one: from the current state it unrolls the next
// iterations' decision tree (both outcomes of every comparison, five levels, at most 31 distinct
// probes), scores all of them in ONE gbs_clip_error launch, reads the K sums back and then walks the
// tree along the outcomes that actually occurred.  The sequence of states visited is exactly the one
// the algorithm as printed would visit; only the grouping of evaluations into launches differs.
#include <math.h>
#include <string.h>

#include "gbs_internal.h"

namespace {

struct State {
    double a, b, m;
    int iteration;
};

// One step of Algorithm 1's loop body: the probe for this state.
double probe_of(const State& s) { return (s.iteration % 2 == 0) ? 0.5 * (s.a + s.m) : 0.5 * (s.b + s.m); }

// The two successor states: improved (f_x < f_m) or not.
State next_state(const State& s, double x, bool improved)
{
    State n = s;
    if (improved) {
        if (x < s.m) n.b = s.m; else n.a = s.m;
        n.m = x;
    } else {
        if (x < s.m) n.a = x; else n.b = x;
    }
    n.iteration = s.iteration + 1;
    return n;
}

constexpr int DEPTH = 5;

// Collect the probes of the decision tree rooted at `s` (depth levels) into alphas[0..K), without repeats.
void collect(const State& s, double eps, int depth, float* alphas, int* K)
{
    if (depth == 0 || !(s.b - s.a > eps)) return;
    const double x = probe_of(s);
    const float xf = (float)x;
    bool seen = false;
    for (int i = 0; i < *K; ++i) seen = seen || alphas[i] == xf;
    if (!seen && *K < GBS_MAX_CANDIDATES) alphas[(*K)++] = xf;
    collect(next_state(s, x, true), eps, depth - 1, alphas, K);
    collect(next_state(s, x, false), eps, depth - 1, alphas, K);
}

int find(const float* alphas, int K, float v)
{
    for (int i = 0; i < K; ++i)
        if (alphas[i] == v) return i;
    return -1;
}

}  // namespace

extern "C" int gbs_search_clip_ratio(const gbs_plan_t* plan, const void* x, int x_dtype, int64_t n_rows,
                                     int64_t x_row_stride, float eps, double* work_dev,
                                     gbs_search_result_t* out_host, void* cuda_stream)
{
    if (!plan || !out_host || !work_dev) return GBS_ERR_INVALID_ARG;
    if (!(eps > 0.f) || !(eps < 1.f)) return GBS_ERR_INVALID_ARG;
    if (n_rows <= 0) return GBS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(work_dev) & 7u) return GBS_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    gbs_device_guard guard;                       // the copies below belong to the plan's device, like its launches
    if (guard.enter(plan->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }

    State s = {0.0, 1.0, 0.5, 0};
    double f_m = 0.0;
    bool have_fm = false;
    int evaluations = 0, rounds = 0;
    float alphas[GBS_MAX_CANDIDATES];
    double sums[GBS_MAX_CANDIDATES];
    while (s.b - s.a > (double)eps) {
        int K = 0;
        if (!have_fm) alphas[K++] = (float)s.m;
        collect(s, (double)eps, DEPTH, alphas, &K);
        if (cudaMemsetAsync(work_dev, 0, sizeof(double) * K, stream) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
        const int rc = gbs_clip_error(plan, x, x_dtype, n_rows, x_row_stride, alphas, K, work_dev, nullptr, cuda_stream);
        if (rc != GBS_OK) return rc;
        if (cudaMemcpyAsync(sums, work_dev, sizeof(double) * K, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) {
            cudaGetLastError();
            return GBS_ERR_CUDA;
        }
        ++rounds;
        if (!have_fm) { f_m = sums[0]; have_fm = true; ++evaluations; }
        // walk the tree along the outcomes that occurred
        for (int level = 0; level < DEPTH && s.b - s.a > (double)eps; ++level) {
            const double xp = probe_of(s);
            const int i = find(alphas, K, (float)xp);
            if (i < 0) break;                         // not scored in this round (cannot happen below 64 probes)
            const double f_x = sums[i];
            ++evaluations;
            const bool improved = f_x < f_m;
            s = next_state(s, xp, improved);
            if (improved) f_m = f_x;
        }
    }
    out_host->alpha = (float)s.m;
    out_host->a = (float)s.a;
    out_host->b = (float)s.b;
    out_host->err = f_m;
    out_host->iterations = s.iteration;
    out_host->evaluations = evaluations;
    out_host->rounds = rounds;
    return GBS_OK;
}
