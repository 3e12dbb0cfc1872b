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

#include <new>

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

// Algorithm 1's start: a = 0, b = 1, m = 1/2, nothing evaluated yet.
void reset(gbs_search_state_t* st)
{
    st->a = 0.0; st->b = 1.0; st->m = 0.5; st->f_m = 0.0;
    st->iteration = 0; st->evaluations = 0; st->have_fm = 0; st->done = 0;
}

State load(const gbs_search_state_t& st) { return State{st.a, st.b, st.m, st.iteration}; }

bool state_valid(const gbs_search_state_t& st)
{
    return st.a >= 0.0 && st.b <= 1.0 && st.a <= st.m && st.m <= st.b && st.iteration >= 0 && st.evaluations >= 0;
}

// One pass through the loop body with the objective value f_x of this state's probe.
void advance(gbs_search_state_t* st, double x, double f_x)
{
    const State s = load(*st);
    const bool improved = f_x < st->f_m;
    const State n = next_state(s, x, improved);
    st->a = n.a; st->b = n.b; st->m = n.m; st->iteration = n.iteration;
    if (improved) st->f_m = f_x;
    st->evaluations += 1;
}

}  // namespace

extern "C" int gbs_search_state_init(gbs_search_state_t* state)
{
    if (!state) return GBS_ERR_INVALID_ARG;
    reset(state);
    return GBS_OK;
}

// Algorithm 1's loop for one projection with the caller's objective (the paper's is perplexity): one evaluation
// per pass, exactly in the printed order; stops at b - a <= eps or after max_iterations passes (> 0), leaving the
// state resumable.
extern "C" int gbs_search_clip_ratio_fn(gbs_objective_fn f, void* ctx, float eps, gbs_search_state_t* st,
                                        int max_iterations)
{
    if (!f || !st) return GBS_ERR_INVALID_ARG;
    if (!(eps > 0.f) || !(eps < 1.f) || max_iterations < 0) return GBS_ERR_INVALID_ARG;
    if (!state_valid(*st)) return GBS_ERR_INVALID_ARG;
    if (!st->have_fm) {
        st->f_m = f((float)st->m, ctx);
        st->have_fm = 1;
        st->evaluations += 1;
    }
    int passes = 0;
    while (st->b - st->a > (double)eps && (max_iterations == 0 || passes < max_iterations)) {
        const double x = probe_of(load(*st));
        advance(st, x, f((float)x, ctx));
        ++passes;
    }
    st->done = !(st->b - st->a > (double)eps);
    return GBS_OK;
}

// Algorithm 1's loop for P projections at once, with the quantization error as the objective.  With that
// objective the projections do not depend on one another (the paper's perplexity couples them, which is why it
// walks them one after the other), so every round scores, for EVERY unfinished projection, the probes of its next
// five iterations' decision tree -- one gbs_clip_error launch per projection, enqueued back to back -- and the
// host waits ONCE per round for all the sums.
extern "C" int gbs_search_clip_ratio_batch(const gbs_search_task_t* tasks, int n_tasks, float eps,
                                           gbs_search_state_t* states, int max_rounds, double* work_dev,
                                           float* alphas_out, int* rounds_out, void* cuda_stream)
{
    if (!tasks || !states || !work_dev || n_tasks < 1 || n_tasks > GBS_MAX_SEARCH_TASKS) return GBS_ERR_INVALID_ARG;
    if (!(eps > 0.f) || !(eps < 1.f) || max_rounds < 0) return GBS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(work_dev) & 7u) return GBS_ERR_ALIGNMENT;
    int device = -1;
    for (int i = 0; i < n_tasks; ++i) {
        if (!tasks[i].plan || tasks[i].n_rows <= 0 || !state_valid(states[i])) return GBS_ERR_INVALID_ARG;
        if (i == 0) device = tasks[i].plan->device;
        else if (tasks[i].plan->device != device) return GBS_ERR_INVALID_ARG;     // one stream, one device
        states[i].done = !(states[i].b - states[i].a > (double)eps);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    gbs_device_guard guard;
    if (guard.enter(device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }

    float* alphas = new (std::nothrow) float[(size_t)n_tasks * GBS_MAX_CANDIDATES];
    double* sums = new (std::nothrow) double[(size_t)n_tasks * GBS_MAX_CANDIDATES];
    int* K = new (std::nothrow) int[n_tasks];
    int rc = (alphas && sums && K) ? GBS_OK : GBS_ERR_ALLOC;
    int rounds = 0;
    while (rc == GBS_OK && (max_rounds == 0 || rounds < max_rounds)) {
        int pending = 0;
        for (int i = 0; i < n_tasks; ++i) pending += states[i].done ? 0 : 1;
        if (!pending) break;
        if (cudaMemsetAsync(work_dev, 0, sizeof(double) * GBS_MAX_CANDIDATES * (size_t)n_tasks, stream) != cudaSuccess) {
            cudaGetLastError();
            rc = GBS_ERR_CUDA;
            break;
        }
        for (int i = 0; i < n_tasks && rc == GBS_OK; ++i) {
            K[i] = 0;
            if (states[i].done) continue;
            float* al = alphas + (size_t)i * GBS_MAX_CANDIDATES;
            if (!states[i].have_fm) al[K[i]++] = (float)states[i].m;
            collect(load(states[i]), (double)eps, DEPTH, al, &K[i]);
            rc = gbs_clip_error(tasks[i].plan, tasks[i].x, tasks[i].x_dtype, tasks[i].n_rows, tasks[i].x_row_stride, al,
                                K[i], work_dev + (size_t)i * GBS_MAX_CANDIDATES, nullptr, cuda_stream);
        }
        if (rc != GBS_OK) break;
        if (cudaMemcpyAsync(sums, work_dev, sizeof(double) * GBS_MAX_CANDIDATES * (size_t)n_tasks, cudaMemcpyDeviceToHost,
                            stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess) {
            cudaGetLastError();
            rc = GBS_ERR_CUDA;
            break;
        }
        ++rounds;
        for (int i = 0; i < n_tasks; ++i) {
            if (states[i].done) continue;
            const float* al = alphas + (size_t)i * GBS_MAX_CANDIDATES;
            const double* sm = sums + (size_t)i * GBS_MAX_CANDIDATES;
            gbs_search_state_t* st = &states[i];
            if (!st->have_fm) { st->f_m = sm[0]; st->have_fm = 1; st->evaluations += 1; }
            // walk the tree along the outcomes that occurred
            for (int level = 0; level < DEPTH && st->b - st->a > (double)eps; ++level) {
                const double xp = probe_of(load(*st));
                const int j = find(al, K[i], (float)xp);
                if (j < 0) break;
                advance(st, xp, sm[j]);
            }
            st->done = !(st->b - st->a > (double)eps);
        }
    }
    delete[] alphas;
    delete[] sums;
    delete[] K;
    if (rc != GBS_OK) return rc;
    if (alphas_out)
        for (int i = 0; i < n_tasks; ++i) alphas_out[i] = (float)states[i].m;     // the list L of Algorithm 1
    if (rounds_out) *rounds_out = rounds;
    return GBS_OK;
}

extern "C" int gbs_search_clip_ratio(const gbs_plan_t* plan, const void* x, int x_dtype, int64_t n_rows,
                                     int64_t x_row_stride, float eps, double* work_dev,
                                     gbs_search_result_t* out_host, void* cuda_stream)
{
    if (!plan || !out_host || !work_dev) return GBS_ERR_INVALID_ARG;
    if (n_rows <= 0) return GBS_ERR_INVALID_ARG;
    gbs_search_task_t task = {plan, x, x_dtype, n_rows, x_row_stride};
    gbs_search_state_t st;
    reset(&st);
    int rounds = 0;
    const int rc = gbs_search_clip_ratio_batch(&task, 1, eps, &st, 0, work_dev, nullptr, &rounds, cuda_stream);
    if (rc != GBS_OK) return rc;
    out_host->alpha = (float)st.m;
    out_host->a = (float)st.a;
    out_host->b = (float)st.b;
    out_host->err = st.f_m;
    out_host->iterations = st.iteration;
    out_host->evaluations = st.evaluations;
    out_host->rounds = rounds;
    return GBS_OK;
}
