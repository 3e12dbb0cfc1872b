// Tensor-core family "ROW": bf16 rows of padded width d' = 128 (KV-cache entries: one row per
// (token, head), Section 5.1), rotated by H_128 (Eq. (1)) and quantized per row or per group of 32, 64
// or 128 rotated coordinates (Sections 2.1, 3.1).
//
// 128 rows form one tile.  Y = X * H_128 is ONE tensor-core contraction per tile: A = the raw tile as
// TMA drops it (128 rows x K = 128, K-major, 128-byte swizzle; columns beyond d are zero-filled, which
// is the zero-pad expansion of Section 4.2), B = a plan-owned image of H_128 (+-1, exact in bf16),
// fp32 accumulators in TMEM.  TMEM lane r then holds all 128 rotated coordinates of row r, so ONE
// THREAD OWNS ONE ROW: max|.| is thread-local, there are no butterflies, no shuffles and no exchange
// between threads.  The thread sweeps its lane twice (32 columns at a time): first for the maxima, then
// to scale, round, clip and pack, and stores 48 or 64 contiguous bytes.
//
// One persistent CTA per SM.  Warp 0 = TMA producer, warp 1 = MMA issuer / TMEM owner, warps 2..17 =
// four epilogue groups of four warps (one TMEM lane quadrant each); group e owns TMEM stage e and every
// fourth tile.  Every mbarrier wait is time-bounded; on expiry the kernel records a code in the plan's
// status word, all roles leave their loops, TMEM is freed and the kernel returns.
#include <math.h>
#include <string.h>

#include <mutex>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int DP = 128;                // padded row width
constexpr int TILE = 128;              // rows per tile (MMA M)
constexpr int STAGES = 4;              // shared-memory stages = TMEM stages = epilogue groups
constexpr int TILE_BYTES = TILE * DP * 2;          // 32 KB of bf16
constexpr int H_BYTES = DP * DP * 2;               // 32 KB: H_128 as bf16
constexpr int EPI_WARPS = 4 * STAGES;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int TMEM_COLS = 512;

struct __align__(1024) Smem {
    unsigned char h[H_BYTES];
    unsigned char x[STAGES][TILE_BYTES];
    unsigned long long full[STAGES], empty[STAGES], tfull[STAGES], tempty[STAGES];
    unsigned long long hbar;               // the image of H_128 has landed
    double csum[GBS_MAX_CANDIDATES];       // clip scoring: this CTA's error totals per candidate
    unsigned tmem_base;
    volatile int abort_flag;
};

struct RowParams {
    long long n_rows;
    int n_tiles;                  // ceil(n_rows / TILE)
    int code_row_bytes;           // 128 * bits / 8
    int chunks_per_group;         // 1, 2 or 4 chunks of 32 coordinates share one scale
    int spr;                      // scales per row
    float c_scale;                // alpha / (D sqrt(d'))
    float c_half;                 // 1 / (2 alpha)
    float norm;                   // 1 / sqrt(d')
    float alpha;                  // asymmetric plans: clip ratio
    float a_delta;                // asymmetric plans: alpha / (sqrt(d') (2^bits - 1))
    float a_zero;                 // asymmetric plans: alpha / sqrt(d')
    const unsigned char* h_img;   // pre-swizzled shared-memory image of H_128 (bf16), plan-owned
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

// ASYM = true: the asymmetric quantizer (range [alpha*min, alpha*max], unsigned codes, scales = (Delta, lo)).
// CLIP = true: instead of quantizing, score K clip ratios (symmetric quantizer) from the thread's own row.
template <int BITS, bool ASYM, bool CLIP>
__global__ void __launch_bounds__(THREADS, 1) k_tc_row_rq(const __grid_constant__ CUtensorMap tmap,
                                                          const __grid_constant__ RowParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- set-up: thread 0 arms the load barriers and starts the first loads at once; one thread of
    // warp 2 arms the remaining barriers; warp 1 allocates TMEM.  One block barrier joins the three.
    int it_p = 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&S->full[s], 1);
        mbar_init(&S->hbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->hbar, H_BYTES);
        bulk_load(S->h, P.h_img, H_BYTES, &S->hbar);          // plan-owned, immutable: needs no ordering
        // programmatic dependent launch: nothing of the caller's memory is touched before this point
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int t = blockIdx.x; it_p < STAGES && t < P.n_tiles; t += gridDim.x, ++it_p) {
            mbar_arrive_expect_tx(&S->full[it_p], TILE_BYTES);
            tma_load_2d(S->x[it_p], &tmap, &S->full[it_p], 0, t * TILE);
            tma_load_2d(S->x[it_p] + TILE_BYTES / 2, &tmap, &S->full[it_p], 64, t * TILE);
        }
    }
    if (threadIdx.x == 64) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->empty[s], 1);
            mbar_init(&S->tfull[s], 1);
            mbar_init(&S->tempty[s], 4);
        }
        S->abort_flag = 0;
        for (int k = 0; k < GBS_MAX_CANDIDATES; ++k) S->csum[k] = 0.0;
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
            for (int t = blockIdx.x + it * (int)gridDim.x; t < P.n_tiles; t += gridDim.x, ++it) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                if (!mbar_wait(&S->abort_flag, &S->empty[s], ph ^ 1, P.status, 1)) break;
                mbar_arrive_expect_tx(&S->full[s], TILE_BYTES);
                tma_load_2d(S->x[s], &tmap, &S->full[s], 0, t * TILE);
                tma_load_2d(S->x[s] + TILE_BYTES / 2, &tmap, &S->full[s], 64, t * TILE);
            }
            if (S->abort_flag) drain_copies(S->full, STAGES, it);
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr unsigned IDESC = instr_desc(TILE, DP, false);
            const unsigned h_base = smem_u32(S->h);
            const unsigned long long xd0 = smem_desc(smem_u32(S->x[0]), 16, 1024, 2);
            const unsigned long long hd0 = smem_desc(h_base, 16, 1024, 2);
            const unsigned xd_lo0 = (unsigned)xd0, xd_hi = (unsigned)(xd0 >> 32);
            const unsigned hd_lo0 = (unsigned)hd0, hd_hi = (unsigned)(hd0 >> 32);
            bool ok = mbar_wait(&S->abort_flag, &S->hbar, 0, P.status, 6);
            int it = 0;
            for (int t = blockIdx.x; ok && t < P.n_tiles; t += gridDim.x, ++it) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                if (!mbar_wait(&S->abort_flag, &S->full[s], ph, P.status, 2)) break;
                if (!mbar_wait(&S->abort_flag, &S->tempty[s], ph ^ 1, P.status, 3)) break;
                tc_fence_after();
                // only the address fields (bytes >> 4, low words) of the two K-major descriptors change between
                // k-steps: 32 bytes inside the 128-byte swizzled row, the second K block TILE*128 bytes further
                unsigned x_lo = xd_lo0 + (unsigned)s * (TILE_BYTES >> 4), h_lo = hd_lo0;
                const unsigned d_tmem = tmem_base + s * DP;
                umma_f16_words<false>(d_tmem, x_lo, xd_hi, h_lo, hd_hi, IDESC);
#pragma unroll
                for (int ks = 1; ks < DP / 16; ++ks) {
                    const unsigned step = (ks & 3) ? 2u : (unsigned)((TILE * 128 - 96) >> 4);
                    x_lo += step;
                    h_lo += step;
                    umma_f16_words<true>(d_tmem, x_lo, xd_hi, h_lo, hd_hi, IDESC);
                }
                umma_commit(&S->empty[s]);
                umma_commit(&S->tfull[s]);
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int e = (warp - 2) >> 2;            // epilogue group = TMEM / shared-memory stage it serves
        const int q = warp & 3;                   // TMEM lane quadrant this warp may access
        const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + e * DP;
        const int cpg = P.chunks_per_group;
        int n = 0;
        for (long long t = (long long)blockIdx.x + (long long)e * gridDim.x; t < P.n_tiles;
             t += (long long)STAGES * gridDim.x, ++n) {
            if (!mbar_wait(&S->abort_flag, &S->tfull[e], n & 1, P.status, 4, false)) break;
            tc_fence_after();
            const long long row = t * TILE + q * 32 + lane;
            unsigned r[32];
            // sweep 1: max|.| of each chunk of 32 rotated coordinates of this thread's row
            float mc[4];                              // max|.| (symmetric) or max (asymmetric) per chunk
            float lc[4];                              // min per chunk (asymmetric only)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                tmem_ld32_issue(taddr + c * 32, r);
                tmem_ld_wait(r);
                if (ASYM) minmax32(r, lc[c], mc[c]);
                else mc[c] = absmax32(r);
            }
            if (cpg == 4) {
                mc[0] = mc[1] = mc[2] = mc[3] = fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
                if (ASYM) lc[0] = lc[1] = lc[2] = lc[3] = fminf(fminf(lc[0], lc[1]), fminf(lc[2], lc[3]));
            } else if (cpg == 2) {
                mc[0] = mc[1] = fmaxf(mc[0], mc[1]);
                mc[2] = mc[3] = fmaxf(mc[2], mc[3]);
                if (ASYM) {
                    lc[0] = lc[1] = fminf(lc[0], lc[1]);
                    lc[2] = lc[3] = fminf(lc[2], lc[3]);
                }
            }
            const bool live = row < P.n_rows;
            if constexpr (CLIP) {
                // Squared quantization error of this thread's row under every candidate clip ratio (Sections
                // 2.1, 3.1), eight candidates per sweep over the four chunks: per value and candidate clamp
                // (fma.sat), round half-even (magic add), residual, square-accumulate.  The row's sums are
                // thread-local; the totals are folded across the warp and added to the CTA's fp64 sums.
                const float twoD = (float)(2 * P.levels);
                const float MAGIC = 8388608.f;
                const float mD = MAGIC + (float)P.levels;
                float rM[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) rM[c] = (mc[c] > 0.f) ? (1.f / mc[c]) : 0.f;
                for (int k0 = 0; k0 < P.K; k0 += 8) {
                    float acc[8];
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) acc[kk] = 0.f;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        tmem_ld32_issue(taddr + c * 32, r);
                        tmem_ld_wait(r);
                        float a1[8], dl[8];
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            a1[kk] = P.clip_half[k0 + kk] * rM[c];
                            dl[kk] = -P.clip_scale[k0 + kk] * mc[c];
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float y = __uint_as_float(r[i]);
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                const float w = __saturatef(fmaf(y, a1[kk], 0.5f));
                                const float qv = fmaf(w, twoD, MAGIC) - mD;
                                const float err = fmaf(qv, dl[kk], y);
                                acc[kk] = fmaf(err, err, acc[kk]);
                            }
                        }
                    }
                    if (P.err_rows && live) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            if (k0 + kk < P.K) P.err_rows[row * P.K + k0 + kk] = acc[kk] * P.norm2;
                    }
                    const float h1 = warp_fold8(acc, lane);
                    const int kk = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
                    if ((lane & 3) == 0 && k0 + kk < P.K) atomicAdd(&S->csum[k0 + kk], (double)h1);
                }
                // the accumulators have been read for the last time: hand the TMEM stage back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S->tempty[e]);
                continue;
            }
            // sweep 2: Delta, round / clip, pack
            unsigned out[4 * BITS];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                tmem_ld32_issue(taddr + c * 32, r);
                tmem_ld_wait(r);
                if (c == 3) {
                    // the accumulators have been read for the last time: hand the TMEM stage back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&S->tempty[e]);
                }
                if (ASYM) {
                    const float range = P.alpha * (mc[c] - lc[c]);          // hi - lo of the clipped range
                    const float a1 = (range > 0.f) ? (1.f / range) : 0.f;
                    quantize_pack32_u<BITS>(r, a1, -(P.alpha * lc[c]) * a1, out + c * BITS);
                } else {
                    const float a1 = (mc[c] > 0.f) ? (P.c_half / mc[c]) : 0.f;
                    quantize_pack32<BITS>(r, a1, out + c * BITS);
                }
                if (P.y_opt && live) {
                    float4* yo = reinterpret_cast<float4*>(P.y_opt + row * DP + c * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        yo[i] = make_float4(__uint_as_float(r[4 * i]) * P.norm, __uint_as_float(r[4 * i + 1]) * P.norm,
                                            __uint_as_float(r[4 * i + 2]) * P.norm, __uint_as_float(r[4 * i + 3]) * P.norm);
                }
            }
            if (live) {
                uint4* dst = reinterpret_cast<uint4*>(P.codes + row * P.code_row_bytes);
#pragma unroll
                for (int i = 0; i < BITS; ++i) dst[i] = make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
                float* sc = P.scales + row * P.spr * (ASYM ? 2 : 1);
                if (ASYM) {
                    // (Delta, lo) per group
#pragma unroll
                    for (int c = 0; c < 4; c += 1) {
                        if (c % cpg == 0) {
                            sc[2 * (c / cpg)] = P.a_delta * (mc[c] - lc[c]);
                            sc[2 * (c / cpg) + 1] = P.a_zero * lc[c];
                        }
                    }
                } else if (cpg == 4) {
                    sc[0] = P.c_scale * mc[0];
                } else if (cpg == 2) {
                    sc[0] = P.c_scale * mc[0];
                    sc[1] = P.c_scale * mc[2];
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) sc[c] = P.c_scale * mc[c];
                }
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
    if (CLIP && (int)threadIdx.x < P.K) atomicAdd(&P.err_sum[threadIdx.x], S->csum[threadIdx.x] * (double)P.norm2);
}

template <typename KernelT>
cudaError_t launch(KernelT kernel, int grid, int smem, cudaStream_t stream, bool pdl, const CUtensorMap& tmap,
                   const RowParams& P)
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

bool gbs_tc_row_supported(const gbs_plan* p)
{
    if (p->d_pad != DP || p->m != 1) return false;
    if (p->group != 0 && p->group != 32 && p->group != 64 && p->group != 128) return false;
    return get_encode() != nullptr && p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

namespace {

int row_prepare(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, CUtensorMap* tmap, RowParams* P)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - TILE) return (int)cudaErrorInvalidValue;      // TMA coordinates are 32-bit
    const cuuint64_t gdim[2] = {(cuuint64_t)p->d, (cuuint64_t)n_rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)(stride * 2)};
    const cuuint32_t box[2] = {64, TILE};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;
    memset(P, 0, sizeof(*P));
    P->n_rows = n_rows;
    P->n_tiles = (int)((n_rows + TILE - 1) / TILE);
    P->code_row_bytes = DP * p->bits / 8;
    P->chunks_per_group = (p->group ? p->group : DP) / 32;
    P->spr = p->group ? DP / p->group : 1;
    P->c_scale = p->c_scale;
    P->c_half = (float)(1.0 / (2.0 * (double)p->alpha));
    P->norm = p->norm;
    P->alpha = p->alpha;
    P->a_delta = (float)((double)p->alpha / (sqrt((double)DP) * (double)((1 << p->bits) - 1)));
    P->a_zero = (float)((double)p->alpha / sqrt((double)DP));
    P->h_img = p->d_aimg;
    P->status = p->d_status;
    P->levels = p->levels;
    P->norm2 = (float)(1.0 / (double)DP);
    return 0;
}

// opt in to the large dynamic shared memory once per device (not a stream operation); callable from several
// host threads at once
cudaError_t row_opt_in(const gbs_plan* p, int smem)
{
    static std::mutex mu;
    static bool attr_done[64] = {false};
    std::lock_guard<std::mutex> lock(mu);
    if (p->device >= 0 && p->device < 64 && attr_done[p->device]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(k_tc_row_rq<3, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_row_rq<4, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_row_rq<3, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_row_rq<4, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_row_rq<4, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && p->device >= 0 && p->device < 64) attr_done[p->device] = true;
    return e;
}

}  // namespace

int gbs_tc_row_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream)
{
    CUtensorMap tmap;
    RowParams P;
    const int rc = row_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    P.codes = (unsigned char*)codes;
    P.scales = scales;
    P.y_opt = y_opt;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = P.n_tiles < p->sm_count ? P.n_tiles : p->sm_count;
    cudaError_t e = row_opt_in(p, smem);
    if (e != cudaSuccess) return (int)e;
    if (p->asym) {
        if (p->bits == 3) e = launch(k_tc_row_rq<3, true, false>, grid, smem, stream, p->pdl != 0, tmap, P);
        else e = launch(k_tc_row_rq<4, true, false>, grid, smem, stream, p->pdl != 0, tmap, P);
    } else {
        if (p->bits == 3) e = launch(k_tc_row_rq<3, false, false>, grid, smem, stream, p->pdl != 0, tmap, P);
        else e = launch(k_tc_row_rq<4, false, false>, grid, smem, stream, p->pdl != 0, tmap, P);
    }
    return (int)e;
}

// Clip-ratio scoring for d' = 128 rows: the same contraction, the row stays in the thread's TMEM lane.
int gbs_tc_row_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                          double* err_sum, float* err_rows, cudaStream_t stream)
{
    CUtensorMap tmap;
    RowParams P;
    const int rc = row_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    P.K = K;
    for (int i = 0; i < K; ++i) {
        P.clip_half[i] = (float)(1.0 / (2.0 * (double)alphas[i]));
        P.clip_scale[i] = (float)((double)alphas[i] / (double)p->levels);
    }
    P.err_sum = err_sum;
    P.err_rows = err_rows;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = P.n_tiles < p->sm_count ? P.n_tiles : p->sm_count;
    cudaError_t e = row_opt_in(p, smem);
    if (e != cudaSuccess) return (int)e;
    e = launch(k_tc_row_rq<4, false, true>, grid, smem, stream, p->pdl != 0, tmap, P);
    return (int)e;
}
