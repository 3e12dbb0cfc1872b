/*
 * gbs.h -- C ABI of the B200 (sm_100a) rotate-and-quantize library.
 *
 * The library implements the online activation / KV path of "Gradual Binary Search and
 * Dimension Expansion" (arXiv 2504.13989): every token row of width d is zero-padded to
 * d' = m * 2^k (Section 4.2, Eq. (2)), rotated by the normalised Hadamard matrix
 * H_{d'} = H_m (x) H_{2^k} / sqrt(d')  (Sylvester recursion of Eq. (1) for the power of two,
 * Paley's Algorithm 2 for the factor m, 1/sqrt(n) normalisation of Appendix A), quantized per
 * token or per group with the symmetric uniform quantizer of Section 2.1 under the clip ratio
 * alpha of Section 3.1, and bit-packed.  A companion call scores K candidate clip ratios by
 * quantization error, the quantity a clip-ratio search such as Algorithm 1 queries.
 *
 * Conventions
 *   - Every function returns an int status: GBS_OK (0) or a negative GBS_ERR_* code.
 *     Nothing throws, prints, or synchronises the device.  Argument errors are detected on
 *     the host before any kernel is launched; no call can fault the device through a bad
 *     size (pointers themselves cannot be validated and are the caller's responsibility).
 *   - "device pointer" = memory of the CUDA device that was current when the plan was
 *     created.  The caller owns all buffers; the library never allocates per call.
 *   - Work is enqueued on the CUDA stream passed as `cuda_stream` (a cudaStream_t cast to
 *     void*; NULL = the legacy default stream) and the call returns without waiting.
 *   - Rotated coordinate i of a row is i = a * 2^k + c with a in [0,m), c in [0,2^k):
 *     y[i] = (1/sqrt(d')) * sum_{a',c'} H_m[a,a'] * (-1)^popcount(c & c') * x_pad[a'*2^k + c'].
 *   - Quantizer: per token (group = 0) or per run of `group` consecutive rotated coordinates,
 *     M = max|y|, Delta = alpha * M / D with D = 2^(bits-1) - 1, code q = clamp(rint(y/Delta),
 *     -D, D) (round half to even); M = 0 gives codes 0 and Delta 0.  (Read with `bits` as the
 *     number of magnitude bits, this is the printed formula Delta = max|X| / (2^b - 1): the
 *     printed formula at b equals this one at bits = b + 1.)
 *   - Packed codes: element j of a row occupies bits [j*bits, (j+1)*bits) of the row's
 *     little-endian bit stream and holds the low `bits` bits of the two's-complement code
 *     (bits = 4: even index in the low nibble).  Row r starts at byte r * d' * bits / 8.
 *   - Scales: fp32 Delta, layout [n_rows, scales_per_row], scales_per_row = group ? d'/group : 1.
 */
#ifndef GBS_H_
#define GBS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define GBS_OK 0
#define GBS_ERR_INVALID_ARG (-1) /* a size, pointer or parameter is out of its documented range */
#define GBS_ERR_UNSUPPORTED (-2) /* no Hadamard construction for this m, or d' too large */
#define GBS_ERR_ALIGNMENT (-3)   /* a pointer or stride violates the stated alignment */
#define GBS_ERR_CUDA (-4)        /* a CUDA runtime call failed (e.g. no device, launch error) */
#define GBS_ERR_ALLOC (-5)       /* host or device allocation for the plan failed */

/* element types of activation inputs / dequantized outputs */
#define GBS_DTYPE_F32 0
#define GBS_DTYPE_BF16 1

/* gbs_plan_create_ex flags */
#define GBS_PLAN_ASYMMETRIC 1    /* asymmetric quantizer (KV entries, Section 5.1): see gbs_plan_create_ex */

/* gbs_dequantize flags */
#define GBS_INVERSE_ROTATE 1

/* largest padded width and largest number of clip-ratio candidates per call */
#define GBS_MAX_D_PAD 32768
#define GBS_MAX_CANDIDATES 64
/* largest padded width gbs_rotate_quantize_static serves from its fixed device array */
#define GBS_STATIC_MAX_D_PAD 4096

typedef struct gbs_plan gbs_plan_t;

typedef struct gbs_plan_info {
    int d, d_pad, m, k;            /* d' = m * 2^k                                   */
    int bits, group;               /* group = 0: one scale per token                  */
    float alpha;
    int levels;                    /* D = 2^(bits-1) - 1; codes lie in [-D, D]        */
    int q_lo, q_hi;                /* -D, +D                                          */
    int64_t code_bytes_per_row;    /* d' * bits / 8                                   */
    int scales_per_row;            /* group ? d'/group : 1                            */
    int asymmetric;                /* 1 for a GBS_PLAN_ASYMMETRIC plan                */
    int scale_floats_per_row;      /* scales_per_row, or 2 * scales_per_row when asymmetric */
    int variant;                   /* kernel family chosen for bf16 rows: 0 = generic shared-memory path,
                                      1 = tensor-core path for d' = 32 * U with U = m * 2^j <= 128, U % 16 == 0,
                                      d % 32 == 0 and group in {0, 32 .. 1024}, 2 = tensor-core path for
                                      d' = 128 rows (m = 1, group in {0, 32, 64, 128}), 3 = tensor-core path for
                                      4096 < d' = 32 * G * U <= 32768 (G in {2, 4, 8}, U as above, per-token
                                      scales, d a multiple of 32 * G), 4 = dense tensor-core contraction with the full
                                      Paley matrix (d' = m), 5 = as 3 where also d' = 128 * U with 80 <= U <= 256,
                                      d % 128 == 0 and group <= 4096: rotate-quantize keeps the rest of the transform
                                      in registers, clip scoring runs as in 3 (GBS_NO_UVR=1 forces 3) (set GBS_FORCE_GENERIC=1 in the
                                      environment before gbs_plan_create to force 0; GBS_NO_PDL=1 launches it
                                      without programmatic stream serialization) */
} gbs_plan_info_t;

/*
 * Create a plan (Section 4.2 for d -> d'; Eq. (1) and Algorithm 2 for the rotation;
 * Section 2.1 / 3.1 for bits and alpha).
 *   d       row width, 1 <= d <= d_pad
 *   d_pad   d' = m * 2^k with 2^k >= 8 and d' <= GBS_MAX_D_PAD
 *   m       1 (pure Sylvester); 12, 20, 24, 44, 48, 60, 68, 72, 80, 84, 104 or 108 (Algorithm 2 with the
 *           prime p = m-1 = 3 mod 4); or 28 (Algorithm 2 over GF(27) = GF(3)[x]/(x^3+2x+1), elements
 *           indexed c0 + 3 c1 + 9 c2).  Other orders return GBS_ERR_UNSUPPORTED.
 *           Full orders: d_pad = m (2^k = 1) is accepted when m - 1 is a prime = 3 mod 4, m a multiple of 8 and
 *           128 <= m <= 4096 -- the rotation is then the Paley matrix H_m itself, e.g. d = 1536, d_pad = m = 1544
 *           (Section 5.2.2).  Such plans take bf16 rows with d a multiple of 8 and group = 0, run as a dense
 *           tensor-core contraction, and support gbs_rotate_quantize and gbs_dequantize (both forms; the inverse
 *           rotation is a dense contraction too); gbs_clip_error and the searches return GBS_ERR_UNSUPPORTED
 *           for them.
 *   bits    3 or 4
 *   group   0, or a power of two >= 8 dividing 2^k (so a group never straddles a block of H_m)
 *   alpha   0 < alpha <= 1
 * The plan owns small device tables (the signs of H_m) on the current device, is immutable
 * and may be used from several threads / streams at once.  *out is written only on success.
 */
int gbs_plan_create(gbs_plan_t** out, int d, int d_pad, int m, int bits, int group, float alpha);

/*
 * gbs_plan_create with flags.  flags = 0 is gbs_plan_create.
 * GBS_PLAN_ASYMMETRIC selects the asymmetric uniform quantizer the paper uses for KV entries
 * (Section 5.1 names it, with "a group size of 128", but prints no formula; this is the textbook one,
 * with the clip ratio of Section 3.1 shrinking both ends of the range).  Per token or group:
 *     lo = alpha * min y,  hi = alpha * max y,  Delta = (hi - lo) / (2^bits - 1),
 *     code = clamp(rint((y - lo) / Delta), 0, 2^bits - 1)  (round half to even),  yhat = code * Delta + lo;
 * a constant group gives codes 0 and Delta 0.  Codes are UNSIGNED `bits`-bit fields, packed as usual;
 * `scales` holds the pair (Delta, lo) per group: layout [n_rows, scales_per_row, 2].
 * Limits: d' = 128 rows (m = 1), group 0, 32, 64 or 128, bf16 input; other shapes return
 * GBS_ERR_UNSUPPORTED.  gbs_clip_error and gbs_search_clip_ratio return GBS_ERR_UNSUPPORTED for such a
 * plan; gbs_dequantize (both forms) honours it.
 */
int gbs_plan_create_ex(gbs_plan_t** out, int d, int d_pad, int m, int bits, int group, float alpha, int flags);

/* Free a plan.  NULL is accepted.  Work already enqueued with the plan must have finished. */
int gbs_plan_destroy(gbs_plan_t* plan);

/* Report the derived sizes of a plan. */
int gbs_plan_info(const gbs_plan_t* plan, gbs_plan_info_t* out);

/*
 * Read and clear the plan's device-side status word.  The tensor-core kernels bound every wait on a
 * barrier; if one ever expires the kernel records a non-zero code here, frees what it holds and
 * returns instead of hanging (the results of that launch are then invalid).  0 = no such event.
 * This call copies 4 bytes from the device and therefore WAITS for the device's pending work.
 * (Not an operation of the paper: a diagnostic of this implementation.)
 */
int gbs_plan_device_status(const gbs_plan_t* plan, int* out);

/*
 * Self-test of the bounded waits (a diagnostic of this implementation, not an operation of the paper): one
 * thread of a one-block kernel on the current device waits, for at most `limit_us` microseconds (1 .. 1 000 000),
 * on a barrier that nothing arrives at.  The wait must run out: the call then returns GBS_OK with *code_out = 7
 * (the code that wait records in its status word), *abort_out = 1 (the flag it raises for the other roles of a
 * kernel) and *waited_us_out = how long it waited (limit_us plus at most a few polling periods).  Nothing
 * faults or hangs; the context stays usable.  Runs on the default stream and WAITS for the device.
 */
int gbs_selftest_wait_expiry(int limit_us, int* code_out, int* abort_out, int* waited_us_out);

/*
 * Fused pad -> rotate -> per-token/group absmax -> scale -> round/clip -> pack
 * (Section 4.2, Eq. (1), Algorithm 2, Section 2.1, Section 3.1), one pass over x.
 *   x            device, n_rows rows of d elements of x_dtype; row r starts at element
 *                r * x_row_stride.  Must be 16-byte aligned with x_row_stride * sizeof(elem)
 *                a multiple of 16, x_row_stride >= d.
 *   codes        device, n_rows * d' * bits / 8 bytes, 16-byte aligned
 *   scales       device, n_rows * scale_floats_per_row floats (scales_per_row Deltas per row; (Delta, lo)
 *                pairs for an asymmetric plan)
 *   y_opt        NULL, or device n_rows * d' floats receiving the rotated normalised values
 *                (16-byte aligned)
 * n_rows = 0 is a successful no-op.
 */
int gbs_rotate_quantize(const gbs_plan_t* plan, const void* x, int x_dtype, int64_t n_rows,
                        int64_t x_row_stride, void* codes, float* scales, float* y_opt,
                        void* cuda_stream);

/*
 * gbs_rotate_quantize for callers that must not allocate device memory.  (The paper has no counterpart
 * of this call; it exists for the deployment reasons below.)
 *
 * A plan owns a little device memory that gbs_plan_create obtains from cudaMalloc: the tensor-core
 * kernel reads a 32 KB table (the +-1 matrix H_m (x) H_{2^j} laid out for the MMA unit) and has a
 * status word.  Some callers cannot go through that: a serving process whose memory pool has already
 * claimed all of the GPU, so that a later cudaMalloc fails; a real-time loop that may not take the
 * device-wide synchronisation cudaMalloc and cudaFree imply; code that is handed a device it may use
 * but not grow on.  For them this call takes the plan's parameters directly and keeps the table and
 * the status word in one fixed array inside the library's device image (about 32 KB on every GPU
 * that loads the library, held until the process exits).  It calls no cudaMalloc, cudaFree or other
 * allocating routine, and the caller still passes the input and both outputs.
 *
 *   d, d_pad, m, bits, group, alpha   as for gbs_plan_create, with these extra limits: bf16 rows only;
 *                d_pad <= GBS_STATIC_MAX_D_PAD; m one of 1, 12, 20, 24, 28 (the array's writer keeps one
 *                32-bit sign word per row of H_m); d_pad and d multiples of 32; d_pad / 32 a multiple of
 *                16; group 0 or 32 .. 1024.  Anything else in gbs_plan_create's range returns
 *                GBS_ERR_UNSUPPORTED ("larger than the fixed array serves, or outside its kernel"):
 *                use a plan for those.
 *   x, n_rows, x_row_stride, codes, scales, cuda_stream   as for gbs_rotate_quantize with
 *                x_dtype = GBS_DTYPE_BF16; results are identical to the plan-based call.
 *
 * The array is shared by every call on a device and keeps what the last call left in it:
 *   - The first call on a device looks up the array's device address (with that device current).  Make
 *     that first call before any stream capture begins.  The status word starts at zero (the array is
 *     zero-initialised when the library's device code is loaded).
 *   - A call reuses the table as it stands only if the previous call on that device used the same
 *     (d_pad, m) on the same stream; every other call first rewrites the table with a small kernel on
 *     `cuda_stream`, so its own kernel is ordered behind the write.  A call made while `cuda_stream` is
 *     being captured always includes the rewrite, and after the first captured call on a device every
 *     call rewrites (a replay changes the array without passing through this function).
 *   - Calls that can overlap on the GPU (different streams, or different host threads without
 *     ordering between their streams) are safe when they all use the same (d_pad, m): they rewrite the
 *     same bytes.  Overlapping calls with DIFFERENT (d_pad, m) race on the array: serialise them, or
 *     give the concurrent users plans.
 */
int gbs_rotate_quantize_static(int d, int d_pad, int m, int bits, int group, float alpha, const void* x,
                               int64_t n_rows, int64_t x_row_stride, void* codes, float* scales,
                               void* cuda_stream);

/*
 * Read and clear the status word of gbs_rotate_quantize_static on the current device (the counterpart of
 * gbs_plan_device_status for the plan-free call: 0 = no bounded wait has expired since the last read).
 * Copies 4 bytes from the fixed array, so it WAITS for the device's pending work; allocates nothing.
 * (The paper has no counterpart of this call: a diagnostic of this implementation.)
 */
int gbs_static_device_status(int* out);

/*
 * Inverse of the quantizer: yhat = q * Delta (Section 2.1) in the rotated domain, width d';
 * with GBS_INVERSE_ROTATE also xhat = (H_{d'}^T yhat / sqrt(d'))[0:d] (rotations are undone by
 * the transpose, Section 2.3.1), width d.
 *   codes, scales  device, layouts as written by gbs_rotate_quantize
 *   out            device, n_rows * (d' or d) elements of out_dtype, rows contiguous,
 *                  16-byte aligned
 * The inverse rotation of plans with one symmetric scale per token in the tensor-core family
 * (widths d' = 32 U, 16 <= U <= 128, d a multiple of 32), and of d' = 128 rows with one scale or
 * (Delta, lo) pair per row, runs on the tensor cores: the integer codes are rotated exactly and
 * multiplied by Delta / sqrt(d') once at the end.
 */
int gbs_dequantize(const gbs_plan_t* plan, const void* codes, const float* scales, int64_t n_rows,
                   void* out, int out_dtype, int flags, void* cuda_stream);

/*
 * Score K clip ratios: for each alpha_k, err_sum[k] += sum over rows and rotated coordinates of
 * (y - yhat_k)^2, yhat_k being the quantizer output (Section 2.1) under clip ratio alpha_k
 * (Section 3.1).  The plan's own alpha is ignored; bits and group are honoured.
 *   x, x_dtype, n_rows, x_row_stride   as for gbs_rotate_quantize
 *   alphas_host   HOST pointer to K floats, each in (0, 1]; copied at call time
 *   K             1 .. GBS_MAX_CANDIDATES
 *   err_sum       device, K doubles, ACCUMULATED into (the caller zeroes them)
 *   err_rows_opt  NULL, or device n_rows * K floats receiving the per-row sums
 */
int gbs_clip_error(const gbs_plan_t* plan, const void* x, int x_dtype, int64_t n_rows,
                   int64_t x_row_stride, const float* alphas_host, int K, double* err_sum,
                   float* err_rows_opt, void* cuda_stream);

/*
 * Result of gbs_search_clip_ratio (host memory).
 */
typedef struct gbs_search_result {
    float alpha;        /* the clip ratio kept at the end (m of Algorithm 1)                       */
    float a, b;         /* the final bracket, b - a <= eps                                          */
    double err;         /* the objective at alpha: sum over rows and coordinates of (y - yhat)^2   */
    int iterations;     /* passes through the loop body of Algorithm 1                              */
    int evaluations;    /* objective values the algorithm consumed: iterations + 1                  */
    int rounds;         /* gbs_clip_error launches used to obtain them                              */
} gbs_search_result_t;

/*
 * The bracket search of Algorithm 1 (Gradual Binary Search, the loop for one projection) for the clip
 * ratio of the rows in x, with the quantization error of gbs_clip_error as the objective (the paper
 * minimises perplexity; this library has no model to evaluate, Sections 3.1 and 4.1).
 * Start a = 0, b = 1, m = 1/2; on even iterations probe (a+m)/2, on odd ones (b+m)/2; a probe that
 * lowers the objective becomes the new m and halves the bracket towards it, otherwise the bracket end
 * on the probe's side moves to the probe; stop when b - a <= eps.  The states visited are those of the
 * algorithm as printed; evaluations are grouped: each round scores the probes of the next five
 * iterations' decision tree (at most 31 clip ratios) in one gbs_clip_error launch.
 *   x, x_dtype, n_rows, x_row_stride   as for gbs_clip_error (n_rows >= 1)
 *   eps        0 < eps < 1 (1/64 gives 9 to 13 iterations)
 *   work_dev   device, GBS_MAX_CANDIDATES doubles, 8-byte aligned, overwritten
 *   out_host   host, written on success
 * BLOCKS: after every round the call waits for `cuda_stream` to read the K sums back.
 */
int gbs_search_clip_ratio(const gbs_plan_t* plan, const void* x, int x_dtype, int64_t n_rows,
                          int64_t x_row_stride, float eps, double* work_dev, gbs_search_result_t* out_host,
                          void* cuda_stream);

/*
 * Weight side of the expansion (Section 4.2, Eq. (2)): the rows of W (one per output channel, width d) are
 * zero-padded to d', rotated by the same H_{d'} / sqrt(d') as the activations and quantized round-to-nearest with
 * the plan's bits, group and alpha -- exactly gbs_rotate_quantize applied to the rows of W, which is what makes
 * (H x_pad)^T (H w_pad) / d' = x^T w hold code for code.  With group = 0 there is one scale per output channel, the
 * form gbs_quantized_matmul consumes.  Done once, offline.
 *   w, w_dtype, n_out, w_row_stride   the weight matrix [n_out, d] (device), as x / x_dtype / n_rows / x_row_stride
 *   codes, scales                     as for gbs_rotate_quantize
 */
int gbs_weight_rotate_quantize(const gbs_plan_t* plan, const void* w, int w_dtype, int64_t n_out, int64_t w_row_stride,
                               void* codes, float* scales, void* cuda_stream);

/*
 * The layer's output straight from the packed codes of both sides (Eq. (2); Section 2.3.1 on keeping the inverse
 * rotation out of the online path): out[t][o] = Delta_x[t] * Delta_w[o] * sum_j q_x[t][j] * q_w[o][j], j over the
 * d' rotated coordinates -- the product of the dequantized rotated activation and the dequantized rotated weight,
 * which equals x^T w up to the two quantization errors.  The sum is an int8 x int8 -> int32 contraction on the
 * tensor cores (exact); the rotated activation is never materialised as floats.
 *   plan_x, codes_x, scales_x, n_tokens   activations as written by gbs_rotate_quantize
 *   plan_w, codes_w, scales_w, n_out      weights as written by gbs_weight_rotate_quantize
 *   out, out_dtype, out_row_stride        device, [n_tokens, n_out] fp32 or bf16, row stride in elements (>= n_out);
 *                                         rows that start on 16-byte boundaries get vector stores
 * Limits: both plans on one device with the same d, d' and m, symmetric, group 0 (one scale per token and per
 * output channel, so the scales leave the sum), d' a multiple of 128; bits may differ (3 or 4 each).  Other plans
 * return GBS_ERR_UNSUPPORTED.
 */
int gbs_quantized_matmul(const gbs_plan_t* plan_x, const void* codes_x, const float* scales_x, int64_t n_tokens,
                         const gbs_plan_t* plan_w, const void* codes_w, const float* scales_w, int64_t n_out,
                         void* out, int out_dtype, int64_t out_row_stride, void* cuda_stream);

/*
 * State of one projection's search (Algorithm 1), a handful of numbers: plain data that may be copied, stored
 * and handed back later to resume the search where it stopped (gbs_search_state_init gives the algorithm's
 * start a = 0, b = 1, m = 1/2).
 */
typedef struct gbs_search_state {
    double a, b, m;     /* the bracket and the kept point                                        */
    double f_m;         /* the objective at m (valid once have_fm is set)                       */
    int iteration;      /* passes through the loop body so far                                   */
    int evaluations;    /* objective values consumed so far                                      */
    int have_fm;        /* f(m) of the start point has been evaluated                            */
    int done;           /* b - a <= eps was reached (set by the search calls)                    */
} gbs_search_state_t;

int gbs_search_state_init(gbs_search_state_t* state);

/*
 * Algorithm 1's loop for one projection with the CALLER's objective, e.g. the perplexity the paper minimises
 * (Sections 3.1, 4.1): f(alpha, ctx) is called once per pass, in the order of the algorithm as printed, plus
 * once for the start point.  Runs until b - a <= eps, or for at most max_iterations passes when that is > 0;
 * `state` (in/out) then resumes.  Host only: touches no device.
 */
typedef double (*gbs_objective_fn)(float alpha, void* ctx);
int gbs_search_clip_ratio_fn(gbs_objective_fn f, void* ctx, float eps, gbs_search_state_t* state,
                             int max_iterations);

/*
 * Algorithm 1's loop for n_tasks projections at once with the quantization error as objective.  The paper walks
 * the projections one after the other because its objective, the model's perplexity, couples them; the
 * quantization error of one projection's input does not depend on the others, so here every round scores the
 * pending probes (the next five iterations' decision tree, at most 31 clip ratios, as in gbs_search_clip_ratio)
 * of EVERY unfinished projection, one gbs_clip_error launch per projection enqueued back to back, and waits once
 * per round.  Each projection visits exactly the states its own gbs_search_clip_ratio call would visit.
 *   tasks       host array: plan, rows (device), dtype, n_rows >= 1 and row stride of each projection; all plans on
 *               one device; n_tasks 1 .. GBS_MAX_SEARCH_TASKS
 *   eps         0 < eps < 1
 *   states      host array, in/out: start from gbs_search_state_init, or resume earlier states
 *   max_rounds  0 = run until every projection is done; otherwise stop after that many rounds (resumable)
 *   work_dev    device, n_tasks * GBS_MAX_CANDIDATES doubles, 8-byte aligned, overwritten
 *   alphas_out  NULL, or host array of n_tasks floats: the list L of Algorithm 1 (the kept point of each projection)
 *   rounds_out  NULL, or the number of rounds this call ran
 * BLOCKS: once per round the call waits for `cuda_stream`.
 */
#define GBS_MAX_SEARCH_TASKS 4096
typedef struct gbs_search_task {
    const gbs_plan_t* plan;
    const void* x;
    int x_dtype;
    int64_t n_rows;
    int64_t x_row_stride;
} gbs_search_task_t;
int gbs_search_clip_ratio_batch(const gbs_search_task_t* tasks, int n_tasks, float eps, gbs_search_state_t* states,
                                int max_rounds, double* work_dev, float* alphas_out, int* rounds_out,
                                void* cuda_stream);

/*
 * Host-only helper: write the m x m sign matrix H_m (row-major, +1 / -1) the plans use
 * (Algorithm 2).  `out_host` must hold m*m bytes.  Needs no device.
 */
int gbs_hadamard_m(int m, int8_t* out_host);

/* Human-readable name of a status code (static string). */
const char* gbs_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GBS_H_ */
