// Tensor-core family "UV": bf16 rows of padded width d' = U * 32 with U = m * 2^j <= 128.
//
// A padded row is viewed as a U x 32 matrix X[u][v] (flat index u*32 + v, u = a*2^j + c_hi, v = c_lo).
// With 2^k = 2^j * 32 the rotation H_m (x) H_{2^k} factors as (H_m (x) H_{2^j}) (x) H_32 (Eq. (1) applied
// to the high and the low bits of the Sylvester index; Algorithm 2 for H_m), so
//
//        Y = A * X * H_32,      A = H_m (x) H_{2^j}   (U x U, entries +-1).
//
//   * A * X runs on the 5th-generation tensor cores (tcgen05.mma, kind::f16, bf16 operands, fp32
//     accumulators in TMEM).  Products (+-1) * bf16 are exact, so this half of the transform loses
//     nothing beyond fp32 summation.  A arrives as one bulk copy of a plan-owned, pre-swizzled 32 KB
//     image (K-major, 128-byte swizzle); B is the raw row tile exactly as TMA drops it (N-major,
//     64-byte swizzle),
//     four tokens per MMA (N = 128).  Rows of A beyond U are zero; columns of X beyond d are filled
//     with zeros by TMA, which is the zero-pad expansion of Section 4.2.
//   * TMEM lane u' then holds (A X)[u'][0..31] of a token: one thread owns 32 CONSECUTIVE output
//     coordinates, and the remaining H_32 is five butterfly stages in its registers.
//   * max|.| (Section 2.1): per token = warp shuffle + a 4-warp exchange; per group of 32*g
//     coordinates (g <= 32 lanes) = warp shuffle only.  Delta, rounding, clipping (Section 3.1) and
//     the 3/4-bit packing follow from registers; each thread stores 12 or 16 contiguous bytes.
//
// One persistent CTA per SM.  Warp 0 = TMA producer, warp 1 = MMA issuer / TMEM owner (warp 18 issues the
// MMAs of every other tile), warps 2..17 =
// epilogue: warp (q, t) serves TMEM lane quadrant q and token t of EVERY stage, so all sixteen work on
// each 4-token tile and a tile's accumulators are released as soon as they are in registers.
// The first loads are issued before the rest of the set-up.  Waiting threads sleep in the barrier
// hardware (try_wait with a suspend-time hint) instead of spinning.  Every wait is bounded; on expiry
// the kernel records a code in the plan's status word, all roles leave their loops, TMEM is freed and
// the kernel returns.
#include <math.h>
#include <string.h>

#include <mutex>
#include <type_traits>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int V = 32;                  // in-register factor (low index bits)
constexpr int TOK = 4;                 // tokens per pipeline stage (MMA N = TOK * V = 128)
constexpr int STAGES = 4;              // shared-memory stages = TMEM stages
constexpr int UMAX = 128;              // largest tensor-core factor
constexpr int STAGE_BYTES_MAX = TOK * UMAX * V * 2;   // 32 KB of bf16
constexpr int A_BYTES = UMAX * UMAX * 2;              // 32 KB: A as bf16, two K blocks of 64
constexpr int EPI_WARPS = 4 * TOK;
// Two threads issue the MMAs, on alternate tiles: in the running kernel a tcgen05.mma takes about three times
// as long as alone on the SM and one issuing thread is busy for most of a tile's period; the second one (on
// another scheduler) takes 1 - 3 % off the steady state.  Every stage must belong to one issuer, so that the
// phase parities it waits for cannot alias: the count divides STAGES.
constexpr int N_ISSUERS = 2;
static_assert(STAGES % N_ISSUERS == 0, "a stage is served by one MMA issuer");
constexpr int THREADS = 32 * (1 + N_ISSUERS + EPI_WARPS);   // producer, issuers (warp 1 and the last ones), epilogue
constexpr int TMEM_COLS = 512;
constexpr int STAGE_COLS = TOK * V;               // 128 fp32 columns per stage

struct __align__(1024) Smem {
    unsigned char a[A_BYTES];
    unsigned char b[STAGES][STAGE_BYTES_MAX];
    unsigned long long full[STAGES], empty[STAGES], tfull[STAGES], tempty[STAGES];
    unsigned long long abar;               // the image of A has landed
    int gabort[TOK][2];                    // [token slot][iteration parity]: a warp of the slot gave up waiting
    __align__(16) float red[TOK][2][4];    // [token slot][iteration parity][quadrant]
    float part[TOK][2][4][GBS_MAX_CANDIDATES];   // clip scoring: per-quadrant error sums of a token
    unsigned tmem_base;
    volatile int abort_flag;
};

struct UvParams {
    long long n_rows;
    int n_groups;                 // ceil(n_rows / TOK)
    int U;                        // m * 2^j, 16 <= U <= 128
    int Upad;                     // U rounded up to a multiple of 16: rows of a token in shared memory
    int j;                        // log2 of the Sylvester part of A
    int ksteps;                   // Upad / 16
    int code_row_bytes;           // d' * bits / 8
    int d_pad;
    int glog;                     // lane-group mode: log2(lanes per quantization group)
    int spr;                      // scales per row
    float c_scale;                // alpha / (D sqrt(d'))
    float c_half;                 // 1 / (2 alpha):  y / (2 D Delta) = Y * c_half / max|Y|
    float norm;                   // 1 / sqrt(d')
    const unsigned char* a_img;   // pre-swizzled shared-memory image of A (bf16), 32 KB, plan-owned
    unsigned char* codes;
    float* scales;
    float* y_opt;
    int* status;
    // clip-ratio scoring (the CLIP instantiation only)
    int K;                        // candidates
    int levels;                   // D
    float norm2;                  // 1 / d'
    float clip_half[GBS_MAX_CANDIDATES];    // 1 / (2 alpha_k), zero beyond K
    float clip_scale[GBS_MAX_CANDIDATES];   // alpha_k / D,     zero beyond K
    double* err_sum;
    float* err_rows;
};

// Squared quantization error of this thread's 32 rotated values under every candidate clip ratio
// (Sections 2.1, 3.1), in units of the unnormalised rotation; the sums over the warp's 32 lanes are left in
// part_q[0 .. K).  Per value and candidate: clamp to the clipped range (fma.sat), round half-even (magic
// add), residual, square-accumulate: five fp32 operations.  Candidates go eight at a time so the 32
// values stay in registers; the eight partial sums are folded across the warp by a halving exchange.
__device__ __forceinline__ void clip_score32(const unsigned r[32], float M, const UvParams& P, float* part_q, int lane)
{
    const float rM = (M > 0.f) ? (1.f / M) : 0.f;
    const float twoD = (float)(2 * P.levels);
    const float MAGIC = 8388608.f;                       // 2^23: w * 2D + MAGIC has rint(w * 2D) in its low bits
    const float mD = MAGIC + (float)P.levels;
    for (int k0 = 0; k0 < P.K; k0 += 8) {
        float a1[8], dl[8], acc[8];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            a1[kk] = P.clip_half[k0 + kk] * rM;
            dl[kk] = -P.clip_scale[k0 + kk] * M;         // -Delta_k
            acc[kk] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const float y = __uint_as_float(r[e]);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const float w = __saturatef(fmaf(y, a1[kk], 0.5f));
                const float qv = fmaf(w, twoD, MAGIC) - mD;            // the code, as a float
                const float err = fmaf(qv, dl[kk], y);
                acc[kk] = fmaf(err, err, acc[kk]);
            }
        }
        const float h1 = warp_fold8(acc, lane);
        const int kk = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
        if ((lane & 3) == 0 && k0 + kk < P.K) part_q[k0 + kk] = h1;
    }
}

// ---------------------------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------------------------
// GROUPED = false: one scale per token.  GROUPED = true: one scale per 2^glog adjacent lanes (32 * 2^glog
// consecutive coordinates), 2^glog <= 32.  CLIP = true: instead of quantizing, score K clip ratios.
// WANT_Y = true: also write the rotated normalised values (the parity output of gbs_rotate_quantize).
template <int BITS, bool GROUPED, bool CLIP, bool WANT_Y>
__global__ void __launch_bounds__(THREADS, 1) k_tc_uv_rq(const __grid_constant__ CUtensorMap tmap,
                                                         const __grid_constant__ UvParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned stage_bytes = (unsigned)(TOK * P.Upad * V * 2);

    // ---- set-up.  Thread 0 arms the load barriers and starts the first loads at once; one thread of
    // warp 2 arms the remaining barriers; warp 1 allocates TMEM.  One block barrier joins the three.
    int it_p = 0;                                  // producer iterations already issued
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&S->full[s], 1);
        mbar_init(&S->abar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->abar, A_BYTES);
        bulk_load(S->a, P.a_img, A_BYTES, &S->abar);          // plan-owned, immutable: needs no ordering
        // programmatic dependent launch: until the wait below returns, an earlier kernel of the stream may
        // still be writing the rows.  Nothing of the caller's memory reaches this SM before it; the first
        // tile is only pulled from DRAM into L2 meanwhile, so that the load that follows the wait hits there
        // (one tile, not all four stages: more prefetches queue ahead of the other CTAs' first loads).
        if ((int)blockIdx.x < P.n_groups) tma_prefetch_3d(&tmap, 0, 0, blockIdx.x * TOK);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int g = blockIdx.x; it_p < STAGES && g < P.n_groups; g += gridDim.x, ++it_p) {
            mbar_arrive_expect_tx(&S->full[it_p], stage_bytes);
            tma_load_3d(S->b[it_p], &tmap, &S->full[it_p], 0, 0, g * TOK);
        }
    }
    if (threadIdx.x == 64) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->empty[s], 1);
            mbar_init(&S->tfull[s], 1);
            mbar_init(&S->tempty[s], EPI_WARPS);
        }
        for (int t = 0; t < TOK; ++t) S->gabort[t][0] = S->gabort[t][1] = 0;
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&S->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned tmem_base = S->tmem_base;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int it = it_p;
            for (int g = blockIdx.x + it * (int)gridDim.x; g < P.n_groups; g += gridDim.x, ++it) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                if (!mbar_wait(&S->abort_flag, &S->empty[s], ph ^ 1, P.status, 1)) break;
                mbar_arrive_expect_tx(&S->full[s], stage_bytes);
                tma_load_3d(S->b[s], &tmap, &S->full[s], 0, 0, g * TOK);
            }
            if (S->abort_flag) drain_copies(S->full, STAGES, it);
        }
    } else if (warp == 1 || warp >= 2 + EPI_WARPS) {
        // ------------------------------ MMA issuers ------------------------------
        const int issuer = warp == 1 ? 0 : warp - (2 + EPI_WARPS) + 1;        // takes tiles issuer, issuer + N_ISSUERS, ..
        if (lane == 0) {
            constexpr unsigned IDESC = instr_desc(UMAX, STAGE_COLS);
            const unsigned a_base = smem_u32(S->a);
            const unsigned tok_bytes = (unsigned)(P.Upad * V * 2);
            const unsigned long long ad0 = smem_desc(a_base, 16, 1024, 2);
            const unsigned long long bd0 = smem_desc(smem_u32(S->b[0]), tok_bytes, 512, 4);
            const unsigned ad_lo0 = (unsigned)ad0, ad_hi = (unsigned)(ad0 >> 32);
            const unsigned bd_lo0 = (unsigned)bd0, bd_hi = (unsigned)(bd0 >> 32);
            bool ok = mbar_wait(&S->abort_flag, &S->abar, 0, P.status, 6);
            int it = issuer;
            for (int g = blockIdx.x + issuer * (int)gridDim.x; ok && g < P.n_groups; g += N_ISSUERS * (int)gridDim.x, it += N_ISSUERS) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                if (!mbar_wait(&S->abort_flag, &S->full[s], ph, P.status, 2)) break;
                if (!mbar_wait(&S->abort_flag, &S->tempty[s], ph ^ 1, P.status, 3)) break;
                tc_fence_after();
                // A: k-step ks = 32 bytes inside the 128-byte swizzled row of block ks/4 (blocks UMAX*128 B apart);
                // 8-row groups 1024 B apart.  B: 16 u-rows of 64 bytes per k-step (1024 B); 8-row groups 512 B
                // apart; next token (N atom) Upad*64 B away.  Only the address fields (bytes >> 4, in the low
                // words) change from one k-step to the next.
                unsigned a_lo = ad_lo0, b_lo = bd_lo0 + (unsigned)s * (STAGE_BYTES_MAX >> 4);
                const unsigned d_tmem = tmem_base + s * STAGE_COLS;
                umma_f16_words<false>(d_tmem, a_lo, ad_hi, b_lo, bd_hi, IDESC);
                for (int ks = 1; ks < P.ksteps; ++ks) {
                    a_lo += (ks & 3) ? 2u : (unsigned)((UMAX * 128 - 96) >> 4);
                    b_lo += 1024u >> 4;
                    umma_f16_words<true>(d_tmem, a_lo, ad_hi, b_lo, bd_hi, IDESC);
                }
                umma_commit(&S->empty[s]);
                umma_commit(&S->tfull[s]);
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int t = (warp - 2) >> 2;            // token slot inside every stage
        const int q = warp & 3;                   // TMEM lane quadrant this warp may access
        const int up = q * 32 + lane;             // u' : this thread owns outputs [up*32, up*32+32)
        const unsigned taddr0 = tmem_base + ((unsigned)(q * 32) << 16) + t * V;
        if (!CLIP) {
            // ---- rotate-quantize.  The loop body is kept to the arithmetic: the kernel is bound by instruction
            // issue in these sixteen warps, so per-iteration bookkeeping is precomputed (iteration counts instead of
            // row comparisons, one lane mask for the group maximum) or folded into the data that is exchanged anyway
            // (a warp whose wait expired hands its token's other warps a poisoned maximum instead of a flag).
            const int n_it = (P.n_groups - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // tiles of this CTA
            const long long row_step = (long long)gridDim.x * TOK;
            const long long row0 = (long long)blockIdx.x * TOK + t;
            int n_store = 0;                      // iterations in which this thread has a row (and a live lane) to store
            if (up < P.U && row0 < P.n_rows) n_store = (int)((P.n_rows - row0 + row_step - 1) / row_step);
            unsigned char* cptr = P.codes + row0 * P.code_row_bytes + up * (V * BITS / 8);
            const long long cstep = row_step * P.code_row_bytes;
            float* sptr = P.scales + row0 * P.spr + (GROUPED ? (up >> P.glog) : 0);
            const long long sstep = row_step * P.spr;
            float* yptr = WANT_Y ? P.y_opt + row0 * (long long)P.d_pad + up * V : nullptr;
            const long long ystep = row_step * P.d_pad;
            const unsigned gl = 1u << P.glog;     // lanes per quantization group (GROUPED)
            const bool scale_writer = GROUPED ? ((lane & (gl - 1u)) == 0) : (up == 0);
            const bool arriver = lane == 0;
            // one iteration on pipeline stage s (a compile-time constant: the loop below is unrolled over the
            // stages so that barrier addresses, TMEM columns and the exchange slot are immediates); false = leave
            auto tile = [&](auto stage, int it, unsigned ph) -> bool {
                constexpr int s = decltype(stage)::value;
                if (!mbar_wait(&S->abort_flag, &S->tfull[s], ph, P.status, 4, false)) {
                    // this warp's wait expired.  With per-token scales the token's other three warps are (or will
                    // be) waiting at the named barrier: come there once more, with a pattern no maximum of absolute
                    // values can have (sign bit set); whoever sees it leaves too, so the four leave together.
                    if (!GROUPED) {
                        if (arriver) reinterpret_cast<unsigned*>(&S->red[t][s & 1][0])[q] = 0xffffffffu;
                        asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
                    }
                    return false;
                }
                unsigned r[32];
                tc_fence_after();
                tmem_ld32_issue(taddr0 + s * STAGE_COLS, r);
                tmem_ld_wait(r);
                // the accumulators are in registers: hand the TMEM stage back to the MMA issuer
                tc_fence_before();
                __syncwarp();
                if (arriver) mbar_arrive(&S->tempty[s]);
                float M = fwht32_absmax(r);
                if (GROUPED) {
                    // fold over the 2^glog lanes of this thread's group (a redux with one mask per group would be
                    // issued once per distinct mask, which is slower for small groups)
                    switch (P.glog) {
                        case 5: M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 16));   // fall through
                        case 4: M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 8));    // fall through
                        case 3: M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 4));    // fall through
                        case 2: M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));    // fall through
                        case 1: M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 1));    // fall through
                        default: break;
                    }
                } else {
                    // per-token max: a warp-wide integer max (the values are non-negative floats), then the four
                    // quadrant warps of the token meet at a 128-thread named barrier
                    const unsigned mw = __reduce_max_sync(0xffffffffu, __float_as_uint(M));
                    unsigned* slot = reinterpret_cast<unsigned*>(&S->red[t][s & 1][0]);
                    if (arriver) slot[q] = mw;
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
                    const uint4 m4 = *reinterpret_cast<const uint4*>(slot);
                    const unsigned mb = max(max(m4.x, m4.y), max(m4.z, m4.w));
                    if ((int)mb < 0) return false;
                    M = __uint_as_float(mb);
                }
                // an all-zero token or group has every value at zero: any finite factor gives code 0.  Rows past
                // the end (last tile only) and dead lanes are quantized like the rest; only the stores are guarded.
                const float a1 = __fdividef(P.c_half, fmaxf(M, 1e-30f));
                unsigned out[BITS];
                quantize_pack32<BITS>(r, a1, out);
                const bool st = it < n_store;
                unsigned* dst = reinterpret_cast<unsigned*>(cptr);
                if (BITS == 4) {
                    if (st) *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
                } else {
                    if (st) { dst[0] = out[0]; dst[1] = out[1]; dst[2] = out[2]; }
                }
                if (st && scale_writer) *sptr = P.c_scale * M;
                if (WANT_Y) {
                    if (st) {
                        float4* yo = reinterpret_cast<float4*>(yptr);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            yo[i] = make_float4(__uint_as_float(r[4 * i]) * P.norm, __uint_as_float(r[4 * i + 1]) * P.norm,
                                                __uint_as_float(r[4 * i + 2]) * P.norm, __uint_as_float(r[4 * i + 3]) * P.norm);
                    }
                    yptr += ystep;
                }
                cptr += cstep;
                sptr += sstep;
                return true;
            };
            static_assert(STAGES == 4, "the epilogue loop is unrolled over four stages");
            unsigned ph = 0;
            for (int it = 0;; ph ^= 1u) {
                if (it >= n_it || !tile(std::integral_constant<int, 0>{}, it, ph)) break;
                ++it;
                if (it >= n_it || !tile(std::integral_constant<int, 1>{}, it, ph)) break;
                ++it;
                if (it >= n_it || !tile(std::integral_constant<int, 2>{}, it, ph)) break;
                ++it;
                if (it >= n_it || !tile(std::integral_constant<int, 3>{}, it, ph)) break;
                ++it;
            }
        } else {
            // ---- clip-ratio scoring
            double dacc0 = 0.0, dacc1 = 0.0;      // quadrant-0 warps: totals of candidates lane, lane + 32
            long long row = (long long)blockIdx.x * TOK + t;
            const long long row_step = (long long)gridDim.x * TOK;
            int it = 0;
            for (long long g = blockIdx.x; g < P.n_groups; g += gridDim.x, ++it, row += row_step) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                const bool ok = mbar_wait(&S->abort_flag, &S->tfull[s], ph, P.status, 4, false);
                unsigned r[32];
                float M = 0.f;
                if (ok) {
                    tc_fence_after();
                    tmem_ld32_issue(taddr0 + s * STAGE_COLS, r);
                    tmem_ld_wait(r);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&S->tempty[s]);
                    M = fwht32_absmax(r);
                }
                const unsigned gp = it & 1;
                if (GROUPED) {
                    for (int o = (1 << P.glog) >> 1; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
                } else {
                    // per-token max: warp-wide integer max, then the token's four quadrant warps meet at a named
                    // barrier; a warp whose wait expired still comes and raises the slot's flag first
                    const unsigned mw = __reduce_max_sync(0xffffffffu, __float_as_uint(M));
                    if (lane == 0) {
                        S->red[t][gp][q] = __uint_as_float(mw);
                        if (!ok) S->gabort[t][gp] = 1;
                    }
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
                    const float4 m4 = *reinterpret_cast<const float4*>(&S->red[t][gp][0]);
                    M = fmaxf(fmaxf(m4.x, m4.y), fmaxf(m4.z, m4.w));
                }
                // each quadrant warp leaves its 32-lane sums in shared memory; the four meet at the token's
                // named barrier (a warp whose wait expired comes too, flag raised), then the quadrant-0 warp
                // adds the four parts in a fixed order: per-row output and fp64 running totals
                if (GROUPED && !ok && lane == 0) S->gabort[t][gp] = 1;
                if (ok) clip_score32(r, M, P, S->part[t][gp][q], lane);
                asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
                if (S->gabort[t][gp]) break;
                if (q == 0) {
                    for (int k = lane; k < P.K; k += 32) {
                        const float rk = (S->part[t][gp][0][k] + S->part[t][gp][1][k]) +
                                         (S->part[t][gp][2][k] + S->part[t][gp][3][k]);
                        if (P.err_rows && row < P.n_rows) P.err_rows[row * P.K + k] = rk * P.norm2;
                        if (k < 32) dacc0 += (double)rk; else dacc1 += (double)rk;
                    }
                }
            }
            if (q == 0) {
                if (lane < P.K) atomicAdd(&P.err_sum[lane], dacc0 * (double)P.norm2);
                if (lane + 32 < P.K) atomicAdd(&P.err_sum[lane + 32], dacc1 * (double)P.norm2);
            }
        }
    }

    // ---- teardown: every role leaves its loop (normally or through the abort flag), then TMEM is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
// host
// ---------------------------------------------------------------------------------------------
int ilog2(int v)
{
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
}

template <typename KernelT>
cudaError_t launch(KernelT kernel, int grid, int smem, cudaStream_t stream, bool pdl, const CUtensorMap& tmap,
                   const UvParams& P)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, tmap, P);
}

}  // namespace

// Shared-memory image of A = H_m (x) H_{2^j} as bf16 (+-1; zero outside U x U): two blocks of 64
// k-columns, 128 rows of 128 bytes each, 16-byte chunks XOR-swizzled with the row index (the 128-byte
// swizzle the MMA descriptor names).  Row = output index u', column = input index u (y = H x).
// transpose: the image of A^T instead (row = input index, column = output index: for x = H^T y).
void gbs_tc_sign_image(const int8_t* hm, int m, int j, int U, unsigned char* img, bool transpose)
{
    const int jm = (1 << j) - 1;
    unsigned short* h = reinterpret_cast<unsigned short*>(img);
    for (int kb = 0; kb < 2; ++kb)
        for (int r = 0; r < UMAX; ++r)
            for (int c = 0; c < 8; ++c)
                for (int e = 0; e < 8; ++e) {
                    const int k = kb * 64 + c * 8 + e;
                    unsigned short v = 0;
                    if (r < U && k < U) {
                        int sign = transpose ? hm[(k >> j) * m + (r >> j)] : hm[(r >> j) * m + (k >> j)];
                        if (__builtin_popcount((unsigned)(r & k & jm)) & 1) sign = -sign;
                        v = sign < 0 ? 0xBF80 : 0x3F80;
                    }
                    const size_t off = (size_t)kb * (UMAX * 128) + (size_t)r * 128 + (size_t)((c ^ (r & 7)) << 4) + e * 2;
                    h[off / 2] = v;
                }
}

void gbs_tc_uv_a_image(const gbs_plan* p, unsigned char* img)
{
    gbs_tc_sign_image(p->h_hm, p->m, p->k - 5, p->d_pad / V, img);
}

bool gbs_tc_uv_supported(const gbs_plan* p)
{
    if (p->d_pad % V != 0 || p->d % V != 0 || p->k < 5) return false;
    const int U = p->d_pad / V;
    if (U > UMAX || U < 16) return false;          // U = m 2^j is a multiple of 4; the contraction is padded to 16
    if (p->group != 0 && (p->group < V || p->group / V > 32)) return false;
    return get_encode() != nullptr && p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

namespace {

// Tensor map of the rows and the parameters common to both uses of the kernel.
int uv_prepare(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, CUtensorMap* tmap, UvParams* P)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - TOK) return (int)cudaErrorInvalidValue;      // TMA coordinates are 32-bit
    const int U = p->d_pad / V;
    const cuuint64_t gdim[3] = {(cuuint64_t)V, (cuuint64_t)(p->d / V), (cuuint64_t)n_rows};
    const cuuint64_t gstr[2] = {(cuuint64_t)(V * 2), (cuuint64_t)(stride * 2)};
    // rows u of the box beyond d / 32 (the zero-pad expansion, and the padding of U to a multiple of the
    // MMA's K = 16) are filled with zeros by TMA
    const int Upad = (U + 15) & ~15;
    const cuuint32_t box[3] = {V, (cuuint32_t)Upad, TOK};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;
    memset(P, 0, sizeof(*P));
    P->n_rows = n_rows;
    P->n_groups = (int)((n_rows + TOK - 1) / TOK);
    P->U = U;
    P->j = p->k - 5;
    P->Upad = Upad;
    P->ksteps = Upad / 16;
    P->code_row_bytes = p->d_pad * p->bits / 8;
    P->d_pad = p->d_pad;
    P->glog = p->group ? ilog2(p->group / V) : 0;
    P->spr = p->group ? p->d_pad / p->group : 1;
    P->c_scale = p->c_scale;
    P->c_half = (float)(1.0 / (2.0 * (double)p->alpha));
    P->norm = p->norm;
    P->a_img = p->d_aimg;
    P->status = p->d_status;
    P->levels = p->levels;
    P->norm2 = (float)(1.0 / (double)p->d_pad);
    return 0;
}

// every instantiation, indexed [bits - 3][grouped][want_y] and [grouped] for the scoring form
typedef void (*UvKernel)(const CUtensorMap, const UvParams);
UvKernel uv_rq_kernel(int bits, bool grouped, bool want_y)
{
    static const UvKernel table[2][2][2] = {
        {{k_tc_uv_rq<3, false, false, false>, k_tc_uv_rq<3, false, false, true>},
         {k_tc_uv_rq<3, true, false, false>, k_tc_uv_rq<3, true, false, true>}},
        {{k_tc_uv_rq<4, false, false, false>, k_tc_uv_rq<4, false, false, true>},
         {k_tc_uv_rq<4, true, false, false>, k_tc_uv_rq<4, true, false, true>}}};
    return table[bits - 3][grouped ? 1 : 0][want_y ? 1 : 0];
}
UvKernel uv_clip_kernel(bool grouped) { return grouped ? k_tc_uv_rq<4, true, true, false> : k_tc_uv_rq<4, false, true, false>; }

// opt in to the large dynamic shared memory once per device (not a stream operation); callable from several
// host threads at once
cudaError_t uv_opt_in(const gbs_plan* p, int smem)
{
    static std::mutex mu;
    static bool attr_done[64] = {false};
    std::lock_guard<std::mutex> lock(mu);
    if (p->device >= 0 && p->device < 64 && attr_done[p->device]) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    for (int bits = 3; bits <= 4 && e == cudaSuccess; ++bits)
        for (int g = 0; g < 2 && e == cudaSuccess; ++g)
            for (int y = 0; y < 2 && e == cudaSuccess; ++y)
                e = cudaFuncSetAttribute(uv_rq_kernel(bits, g != 0, y != 0), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    for (int g = 0; g < 2 && e == cudaSuccess; ++g)
        e = cudaFuncSetAttribute(uv_clip_kernel(g != 0), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && p->device >= 0 && p->device < 64) attr_done[p->device] = true;
    return e;
}

}  // namespace

int gbs_tc_uv_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                              float* scales, float* y_opt, cudaStream_t stream)
{
    CUtensorMap tmap;
    UvParams P;
    int rc = uv_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    P.codes = (unsigned char*)codes;
    P.scales = scales;
    P.y_opt = y_opt;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = P.n_groups < p->sm_count ? P.n_groups : p->sm_count;
    cudaError_t e = uv_opt_in(p, smem);
    if (e != cudaSuccess) return (int)e;
    const bool pdl = p->pdl != 0;
    e = launch(uv_rq_kernel(p->bits, p->group != 0, y_opt != nullptr), grid, smem, stream, pdl, tmap, P);
    return (int)e;
}

// Clip-ratio scoring on the same front end: rotate on the tensor cores, keep the rotated values in
// registers, score all K candidates from there.
int gbs_tc_uv_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                         double* err_sum, float* err_rows, cudaStream_t stream)
{
    CUtensorMap tmap;
    UvParams P;
    int rc = uv_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    P.K = K;
    for (int i = 0; i < K; ++i) {
        P.clip_half[i] = (float)(1.0 / (2.0 * (double)alphas[i]));
        P.clip_scale[i] = (float)((double)alphas[i] / (double)p->levels);
    }
    P.err_sum = err_sum;
    P.err_rows = err_rows;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = P.n_groups < p->sm_count ? P.n_groups : p->sm_count;
    cudaError_t e = uv_opt_in(p, smem);
    if (e != cudaSuccess) return (int)e;
    const bool pdl = p->pdl != 0;
    e = launch(uv_clip_kernel(p->group != 0), grid, smem, stream, pdl, tmap, P);
    return (int)e;
}

// ---------------------------------------------------------------------------------------------
// gbs_rotate_quantize_static: the same fused kernel for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------------
// The kernel above needs 32 KB of device memory besides its inputs and outputs (the image of A) and
// a status word.  A plan gets them from cudaMalloc; here they live in a file-scope device array that
// every GPU loading this library carries until the process exits (zero-initialised when the module is
// loaded, so the status word needs no clearing before its first use).
namespace {

constexpr int STATIC_IMAGE_BYTES = A_BYTES;
constexpr int STATIC_SCRATCH_BYTES = STATIC_IMAGE_BYTES + 256;        // image, then the status word
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// Fills the image of A = H_m (x) H_{2^j} (same layout as gbs_tc_uv_a_image) straight into the array.
struct StaticFillParams {
    int U, j;
    unsigned hm_neg[32];          // bit a of word a': H_m[a'][a] == -1   (m <= 28 < 32)
};
__global__ void __launch_bounds__(256) k_static_fill_a(const __grid_constant__ StaticFillParams F)
{
    const unsigned jm = (1u << F.j) - 1u;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < 2 * UMAX * 8; c += gridDim.x * blockDim.x) {
        const int kb = c >> 10, r = (c >> 3) & (UMAX - 1), ch = c & 7;
        const unsigned rowbits = (r < F.U) ? F.hm_neg[r >> F.j] : 0u;
        unsigned w[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
            unsigned h2 = 0;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int k = kb * 64 + ch * 8 + e + t;
                unsigned h = 0u;
                if (r < F.U && k < F.U) {          // k < U keeps the shift below m <= 28
                    const unsigned neg = ((rowbits >> (k >> F.j)) ^ (unsigned)__popc((unsigned)r & (unsigned)k & jm)) & 1u;
                    h = neg ? 0xBF80u : 0x3F80u;
                }
                h2 |= h << (16 * t);
            }
            w[e >> 1] = h2;
        }
        *reinterpret_cast<uint4*>(g_static_scratch + (size_t)kb * (UMAX * 128) + (size_t)r * 128 +
                                  (size_t)((ch ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

struct StaticDeviceState {
    unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
    int sm_count = 0, smem_optin = 0;
    // which A the array holds, and the stream whose work wrote it: a later call may skip the rewrite only if it
    // is ordered behind that write, i.e. on the same stream (0 = nothing written yet)
    int image_m = 0, image_k = 0;
    cudaStream_t image_stream = nullptr;
    bool seen_capture = false;          // a call was captured on this device: replays rewrite the array unseen
};
StaticDeviceState g_static_state[64];
std::mutex g_static_mutex;

// Set-up, once per device, with that device current: the array's name is only a host-side handle, the kernels
// need its device address.  Caller holds g_static_mutex.
int static_state(StaticDeviceState** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return GBS_ERR_CUDA; }
    StaticDeviceState& st = g_static_state[dev];
    if (!st.scratch) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return GBS_ERR_CUDA; }
        if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&st.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            cudaGetLastError();
            return GBS_ERR_CUDA;
        }
        st.scratch = static_cast<unsigned char*>(ptr);
    }
    *out = &st;
    return dev;
}

}  // namespace

extern "C" int gbs_rotate_quantize_static(int d, int d_pad, int m, int bits, int group, float alpha, const void* x,
                                          int64_t n_rows, int64_t x_row_stride, void* codes, float* scales,
                                          void* cuda_stream)
{
    // ---- arguments: the ranges of gbs_plan_create and gbs_rotate_quantize, then this entry point's own limits
    if (d < 1 || d_pad < d || m < 1) return GBS_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4) return GBS_ERR_INVALID_ARG;
    if (!(alpha > 0.f) || !(alpha <= 1.f)) return GBS_ERR_INVALID_ARG;
    if (d_pad % m != 0) return GBS_ERR_INVALID_ARG;
    int k = -1;
    for (int l = 0; l < 31; ++l)
        if ((d_pad / m) == (1 << l)) k = l;
    if (k < 3) return GBS_ERR_INVALID_ARG;
    if (group != 0 && (group < 8 || (group & (group - 1)) != 0 || (1 << k) % group != 0)) return GBS_ERR_INVALID_ARG;
    if (n_rows < 0) return GBS_ERR_INVALID_ARG;
    if (d_pad > GBS_STATIC_MAX_D_PAD) return GBS_ERR_UNSUPPORTED;          // beyond what the fixed array serves
    if (!(m == 1 || m == 12 || m == 20 || m == 24 || m == 28)) return GBS_ERR_UNSUPPORTED;   // m <= 28: one sign word per row
    gbs_plan p;
    memset(&p, 0, sizeof(p));
    if (gbs_build_hadamard_m(m, p.h_hm) != GBS_OK) return GBS_ERR_UNSUPPORTED;
    p.d = d; p.d_pad = d_pad; p.m = m; p.k = k; p.bits = bits; p.group = group; p.alpha = alpha;
    {
        const int U = d_pad / V;
        if (d_pad % V != 0 || d % V != 0 || k < 5 || U % 16 != 0 || (group != 0 && (group < V || group / V > 32)))
            return GBS_ERR_UNSUPPORTED;                                      // outside this kernel family
    }
    if (n_rows == 0) return GBS_OK;
    if (!x || !codes || !scales || x_row_stride < d) return GBS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) || ((x_row_stride * 2) & 15) || (reinterpret_cast<uintptr_t>(codes) & 15u) ||
        (reinterpret_cast<uintptr_t>(scales) & 3u))
        return GBS_ERR_ALIGNMENT;

    p.levels = (1 << (bits - 1)) - 1;
    const double rootn = sqrt((double)d_pad);
    p.norm = (float)(1.0 / rootn);
    p.c_scale = (float)((double)alpha / ((double)p.levels * rootn));
    p.c_inv = (float)((double)p.levels / (double)alpha);
    p.variant = GBS_VARIANT_TC_UV;
    p.pdl = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState* stp = nullptr;
    const int dev = static_state(&stp);
    if (dev < 0) return dev;
    StaticDeviceState& st = *stp;
    if (st.smem_optin < (int)(sizeof(Smem) + 1024) || get_encode() == nullptr) return GBS_ERR_UNSUPPORTED;
    p.device = dev;
    p.sm_count = st.sm_count;
    p.smem_optin = st.smem_optin;
    p.d_aimg = st.scratch;
    p.d_status = reinterpret_cast<int*>(st.scratch + STATIC_IMAGE_BYTES);
    // The array may be reused as it stands only by a call that is ordered behind the work that wrote it: same
    // table and same stream.  Every other call rewrites the table on its own stream first; two streams
    // rewriting the same table write the same bytes.  A captured call always carries its rewrite (it runs at
    // replay, not now), and once a call has been captured on this device the record kept here can no longer
    // be trusted (a replay rewrites the array without passing through this function), so from then on every
    // call rewrites.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    if (capturing) st.seen_capture = true;
    if (st.seen_capture || st.image_m != m || st.image_k != k || st.image_stream != stream) {
        StaticFillParams F;
        F.U = d_pad / V;
        F.j = k - 5;
        for (int a = 0; a < 32; ++a) {
            unsigned neg = 0;
            if (a < m)
                for (int b = 0; b < m; ++b)
                    if (p.h_hm[a * m + b] < 0) neg |= 1u << b;
            F.hm_neg[a] = neg;
        }
        k_static_fill_a<<<8, 256, 0, stream>>>(F);
        if (cudaGetLastError() != cudaSuccess) return GBS_ERR_CUDA;
        st.image_m = m;
        st.image_k = k;
        st.image_stream = stream;
    }
    const int e = gbs_tc_uv_rotate_quantize(&p, x, n_rows, x_row_stride, codes, scales, nullptr, stream);
    if (e != 0) cudaGetLastError();
    return e == 0 ? GBS_OK : GBS_ERR_CUDA;
}

extern "C" int gbs_static_device_status(int* out)
{
    if (!out) return GBS_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState* st = nullptr;
    const int dev = static_state(&st);
    if (dev < 0) return dev;
    int v = 0;
    int* word = reinterpret_cast<int*>(st->scratch + STATIC_IMAGE_BYTES);
    if (cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(word, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return GBS_ERR_CUDA;
    }
    *out = v;
    return GBS_OK;
}
