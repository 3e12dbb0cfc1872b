// Tensor-core family "UVM": bf16 rows of padded width d' = U * G * 32 with U = m * 2^j <= 128 and
// G = 2, 4 or 8 (widths 4096 < d' <= 32768, e.g. the MLP width 20480 = 20 * 1024: U = 80, G = 8).
//
// A padded row is viewed as X[u][c][v] (flat index (u*G + c)*32 + v).  With 2^k = 2^j * G * 32 the rotation
// factors as (H_m (x) H_{2^j}) (x) H_G (x) H_32 (Eq. (1) on the three bit fields of the Sylvester index,
// Algorithm 2 for H_m):
//   * A = H_m (x) H_{2^j} (U x U, +-1) runs on the tensor cores exactly as in the UV family, one token
//     per MMA batch, N = G*32 columns: TMEM lane u' holds G chunks of 32 consecutive coordinates.
//   * H_32 inside each chunk and H_G across the chunks are butterflies in registers, in two sweeps over
//     TMEM (a thread cannot hold its 256 values at once): sweep 1 transforms each chunk in place,
//     sweep 2 loads 4 columns of every chunk, runs the G-point butterflies, takes max|.| and writes back.
//   * sweep 3 scales, rounds, clips (Sections 2.1, 3.1) and packs each chunk.  Scales are per token, or
//     per group of 32 * 2^e consecutive coordinates (GROUPED): a group is 2^e chunks of one lane, or,
//     beyond the G chunks of a lane, up to 32 whole lanes of a warp; the two warps that share a lane
//     quadrant exchange their per-chunk maxima through shared memory at the second barrier.
// The sixteen epilogue warps form two groups of eight that take alternate tokens (so that one group's
// barrier waits are filled by the other's arithmetic): in a group, warp (q, w) serves lane quadrant q,
// chunks w, w+2, .. in sweeps 1 and 3 and column groups 4w .. 4w+3 in sweep 2; two 256-thread named
// barriers per token separate the sweeps (the second also carries the per-token maximum).  Roles, pipeline, bounded waits and teardown
// are those of the UV family.
#include <math.h>
#include <string.h>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int V = 32;
constexpr int UMAX = 128;
constexpr int A_BYTES = UMAX * UMAX * 2;
constexpr int B_BYTES = 160 * 1024;               // shared memory for the row stages
constexpr int MAX_STAGES = 4;
constexpr int EPI_WARPS = 16;
// With G = 2 a token is one 128 x 64 x K contraction and the epilogue per token is short: the thread that issues
// the MMAs (about 200 cycles each in the running kernel) is then the bottleneck, and a second issuing thread on
// another scheduler takes every other token (55 -> 42 us for 8192 x 8192).  With G = 4 or 8 it does not pay.
// Every shared-memory and TMEM stage stays with one issuer (both stage counts are even), so the phase
// parities an issuer waits for cannot alias.
__host__ __device__ constexpr int issuers_for(int glog) { return glog == 1 ? 2 : 1; }
__host__ __device__ constexpr int threads_for(int glog) { return 32 * (1 + issuers_for(glog) + EPI_WARPS); }
constexpr int TMEM_COLS = 512;

struct __align__(1024) Smem {
    unsigned char a[A_BYTES];
    unsigned char b[B_BYTES];
    unsigned long long full[MAX_STAGES], empty[MAX_STAGES], tfull[MAX_STAGES], tempty[MAX_STAGES];
    unsigned long long abar;
    __align__(16) float red[2][2][8];          // [group][iteration parity][warp of the group]: max of the token
    int gabort[2][2];                          // [group][iteration parity]: a warp of the group gave up waiting
    // GROUPED: [group][warp half w][lane u'][chunk]: max|.| of the chunk's scale group over the columns warp w
    // swept.  Written between a token's two barriers and read after the second, so one copy is enough.
    __align__(16) float gm[2][2][UMAX][8];
    // CLIP: [group][warp of the group][candidate]: a warp's error sums over its lanes and chunks of the token.
    // Written in sweep 3 and read after the third barrier; the next token's writes come two barriers later.
    float cpart[2][8][GBS_MAX_CANDIDATES];
    unsigned tmem_base;
    volatile int abort_flag;
};

struct UvmParams {
    long long n_rows;
    int U;                        // m * 2^j
    int Upad;                     // U rounded up to a multiple of 16
    int ksteps;                   // Upad / 16
    int n_stages;                 // shared-memory stages in use
    int stage_bytes;              // Upad * G * 64
    int code_row_bytes;
    int d_pad;
    int gsh;                      // GROUPED: scale group = 2^gsh chunks of 32 coordinates
    int spr;                      // scales per row
    float c_scale, c_half, norm;
    const unsigned char* a_img;
    unsigned char* codes;
    float* scales;
    float* y_opt;
    int* status;
    // clip-ratio scoring (the CLIP instantiations only)
    int K;                        // candidates
    int levels;                   // D
    float norm2;                  // 1 / d'
    float clip_half[GBS_MAX_CANDIDATES];    // 1 / (2 alpha_k), zero beyond K
    float clip_scale[GBS_MAX_CANDIDATES];   // alpha_k / D,     zero beyond K
    double* err_sum;
    float* err_rows;
};

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tmem_ld4_issue(unsigned taddr, unsigned r[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st4(unsigned taddr, const unsigned r[4])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%4], {%0, %1, %2, %3};"
                 ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const unsigned r[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// H_32 on 32 registers, in place, natural order (no max: the transform is not finished yet).
__device__ __forceinline__ void fwht32(unsigned r[32])
{
    f32x2 p[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) p[i] = pk(r[2 * i], r[2 * i + 1]);
#pragma unroll
    for (int h = 1; h < 16; h <<= 1)
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if ((i & h) == 0) {
                const f32x2 a = p[i], b = p[i + h];
                p[i] = add2(a, b);
                p[i + h] = sub2(a, b);
            }
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        unsigned ua, ub;
        unpk(p[i], ua, ub);
        const float a = __uint_as_float(ua), b = __uint_as_float(ub);
        r[2 * i] = __float_as_uint(a + b);
        r[2 * i + 1] = __float_as_uint(a - b);
    }
}

// tcgen05.wait::ld that names the loaded registers, so that nothing using them is scheduled before it
template <int N>
__device__ __forceinline__ void tmem_ld_wait_n(unsigned* r);
template <>
__device__ __forceinline__ void tmem_ld_wait_n<8>(unsigned* r)
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7])::"memory");
}
template <>
__device__ __forceinline__ void tmem_ld_wait_n<16>(unsigned* r)
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 ::"memory");
}
template <>
__device__ __forceinline__ void tmem_ld_wait_n<32>(unsigned* r)
{
    tmem_ld_wait(r);
}

// ---------------------------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------------------------
// CLIP = true: instead of quantizing, sweep 3 scores K clip ratios (Sections 2.1, 3.1) as the UV family does:
// per value and candidate clamp (fma.sat), round half-even (magic add), residual, square-accumulate, eight
// candidates at a time over the warp's chunks; warp sums go to shared memory, a third named barrier, and the
// first warp of the group adds the eight parts in a fixed order (per-row output, fp64 running totals).
template <int BITS, int GLOG, bool GROUPED, bool CLIP>
__global__ void __launch_bounds__(threads_for(GLOG), 1) k_tc_uvm_rq(const __grid_constant__ CUtensorMap tmap,
                                                          const __grid_constant__ UvmParams P)
{
    constexpr int G = 1 << GLOG;                  // chunks of 32 coordinates per TMEM lane
    constexpr int NCOLS = G * V;                  // accumulator columns per token
    constexpr int TSTAGES = (G == 8) ? 2 : 4;     // TMEM stages
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nst = P.n_stages;
    const int n_tok = (int)P.n_rows;

    int it_p = 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) mbar_init(&S->full[s], 1);
        mbar_init(&S->abar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->abar, A_BYTES);
        bulk_load(S->a, P.a_img, A_BYTES, &S->abar);          // plan-owned, immutable: needs no ordering
        asm volatile("griddepcontrol.wait;" ::: "memory");   // nothing of the caller's memory is touched before
        for (int tk = blockIdx.x; it_p < nst && tk < n_tok; tk += gridDim.x, ++it_p) {
            mbar_arrive_expect_tx(&S->full[it_p], (unsigned)P.stage_bytes);
            for (int c = 0; c < G; ++c)          // one box per chunk: U rows of 32 values
                tma_load_4d(S->b + (size_t)it_p * P.stage_bytes + (size_t)c * (P.stage_bytes >> GLOG), &tmap,
                            &S->full[it_p], 0, c, 0, tk);
        }
    }
    if (threadIdx.x == 64) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(&S->empty[s], 1);
            mbar_init(&S->tfull[s], 1);
            mbar_init(&S->tempty[s], EPI_WARPS / 2);
        }
        S->gabort[0][0] = S->gabort[0][1] = S->gabort[1][0] = S->gabort[1][1] = 0;
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
            for (int tk = blockIdx.x + it * (int)gridDim.x; tk < n_tok; tk += gridDim.x, ++it) {
                const int s = it % nst;
                const unsigned ph = (it / nst) & 1;
                if (!mbar_wait(&S->abort_flag, &S->empty[s], ph ^ 1, P.status, 1)) break;
                mbar_arrive_expect_tx(&S->full[s], (unsigned)P.stage_bytes);
                for (int c = 0; c < G; ++c)
                    tma_load_4d(S->b + (size_t)s * P.stage_bytes + (size_t)c * (P.stage_bytes >> GLOG), &tmap,
                                &S->full[s], 0, c, 0, tk);
            }
            if (S->abort_flag) drain_copies(S->full, nst, it);
        }
    } else if (warp == 1 || warp >= 2 + EPI_WARPS) {
        constexpr int NISS = issuers_for(GLOG);
        const int issuer = warp == 1 ? 0 : warp - (2 + EPI_WARPS) + 1;      // takes tokens issuer, issuer + NISS, ..
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr unsigned IDESC = instr_desc(UMAX, NCOLS);
            const unsigned a_base = smem_u32(S->a);
            const unsigned chunk_bytes = (unsigned)(P.Upad * V * 2);  // one chunk (N atom of 32): Upad rows of 64 bytes
            const unsigned long long ad0 = smem_desc(a_base, 16, 1024, 2);
            const unsigned long long bd0 = smem_desc(smem_u32(S->b), chunk_bytes, 512, 4);
            const unsigned ad_lo0 = (unsigned)ad0, ad_hi = (unsigned)(ad0 >> 32);
            const unsigned bd_lo0 = (unsigned)bd0, bd_hi = (unsigned)(bd0 >> 32);
            bool ok = mbar_wait(&S->abort_flag, &S->abar, 0, P.status, 6);
            int it = issuer;
            for (int tk = blockIdx.x + issuer * (int)gridDim.x; ok && tk < n_tok; tk += NISS * (int)gridDim.x, it += NISS) {
                const int s = it % nst, ts = it % TSTAGES;
                if (!mbar_wait(&S->abort_flag, &S->full[s], (it / nst) & 1, P.status, 2)) break;
                if (!mbar_wait(&S->abort_flag, &S->tempty[ts], ((it / TSTAGES) & 1) ^ 1, P.status, 3)) break;
                tc_fence_after();
                // only the address fields (bytes >> 4, low words) of the descriptors change between k-steps
                unsigned a_lo = ad_lo0, b_lo = bd_lo0 + (unsigned)s * ((unsigned)P.stage_bytes >> 4);
                const unsigned d_tmem = tmem_base + ts * NCOLS;
                umma_f16_words<false>(d_tmem, a_lo, ad_hi, b_lo, bd_hi, IDESC);
                for (int ks = 1; ks < P.ksteps; ++ks) {
                    a_lo += (ks & 3) ? 2u : (unsigned)((UMAX * 128 - 96) >> 4);
                    b_lo += 1024u >> 4;
                    umma_f16_words<true>(d_tmem, a_lo, ad_hi, b_lo, bd_hi, IDESC);
                }
                umma_commit(&S->empty[s]);
                umma_commit(&S->tfull[ts]);
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int grp = (warp - 2) >> 3;          // group: takes tokens it = grp, grp + 2, ..
        const int w = ((warp - 2) >> 2) & 1;      // which chunks / column groups of the token this warp takes
        const int q = warp & 3;                   // TMEM lane quadrant this warp may access
        const int ew = w * 4 + q;                 // index inside the group
        const int up = q * 32 + lane;             // u'
        const bool quad_live = q * 32 < P.U;      // a quadrant wholly beyond U has nothing to do
        const bool lane_live = up < P.U;
        const unsigned tq = tmem_base + ((unsigned)(q * 32) << 16);
        double dacc0 = 0.0, dacc1 = 0.0;          // CLIP, first warp of a group: totals of candidates lane, lane + 32
        int it = grp, n = 0;
        for (long long row = (long long)blockIdx.x + (long long)grp * gridDim.x; row < P.n_rows;
             row += 2ll * gridDim.x, it += 2, ++n) {
            const int ts = it % TSTAGES;
            const unsigned gp = n & 1;
            const bool ok = mbar_wait(&S->abort_flag, &S->tfull[ts], (it / TSTAGES) & 1, P.status, 4, false);
            if (!ok && lane == 0) S->gabort[grp][gp] = 1;
            const unsigned tcol = tq + ts * NCOLS;
            unsigned r[32];
            // sweep 1: H_32 inside the chunks this warp owns
            if (ok && quad_live) {
                tc_fence_after();
#pragma unroll
                for (int c = w; c < G; c += 2) {
                    tmem_ld32_issue(tcol + c * V, r);
                    tmem_ld_wait(r);
                    fwht32(r);
                    tmem_st32(tcol + c * V, r);
                }
                tmem_wait_st();
                tc_fence_before();
            }
            asm volatile("bar.sync %0, 256;" ::"r"(1 + grp) : "memory");
            if (S->gabort[grp][gp]) break;
            // sweep 2: H_G across the chunks, four columns at a time; max|.| of the finished transform
            float M = 0.f;
            float Mc[G];                                  // GROUPED: max|.| per chunk, then per scale group
#pragma unroll
            for (int c = 0; c < G; ++c) Mc[c] = 0.f;
            if (quad_live) {
                tc_fence_after();
#pragma unroll
                for (int cg = 0; cg < 4; ++cg) {
                    const unsigned col0 = tcol + (4 * w + cg) * 4;
                    unsigned x[G * 4];
#pragma unroll
                    for (int c = 0; c < G; ++c) tmem_ld4_issue(col0 + c * V, x + 4 * c);
                    tmem_ld_wait_n<G * 4>(x);
                    f32x2 p[G * 2];
#pragma unroll
                    for (int i = 0; i < G * 2; ++i) p[i] = pk(x[2 * i], x[2 * i + 1]);
#pragma unroll
                    for (int h = 1; h < G; h <<= 1)
#pragma unroll
                        for (int c = 0; c < G; ++c)
                            if ((c & h) == 0) {
#pragma unroll
                                for (int i = 0; i < 2; ++i) {
                                    const f32x2 a = p[2 * c + i], b = p[2 * (c + h) + i];
                                    p[2 * c + i] = add2(a, b);
                                    p[2 * (c + h) + i] = sub2(a, b);
                                }
                            }
#pragma unroll
                    for (int i = 0; i < G * 2; ++i) {
                        unpk(p[i], x[2 * i], x[2 * i + 1]);
                        if (GROUPED)
                            Mc[i >> 1] = max3(fabsf(__uint_as_float(x[2 * i])), fabsf(__uint_as_float(x[2 * i + 1])), Mc[i >> 1]);
                        else
                            M = max3(fabsf(__uint_as_float(x[2 * i])), fabsf(__uint_as_float(x[2 * i + 1])), M);
                    }
#pragma unroll
                    for (int c = 0; c < G; ++c) tmem_st4(col0 + c * V, x + 4 * c);
                }
                tmem_wait_st();
                tc_fence_before();
                if (GROUPED) {
                    // chunk maxima -> group maxima: over the 2^gsh chunks of a group inside the lane, then, for
                    // a group of several whole lanes, over those lanes (every chunk of the lane is in it)
#pragma unroll
                    for (int h = 1; h < G; h <<= 1)
                        if (h < (1 << P.gsh)) {
#pragma unroll
                            for (int c = 0; c < G; ++c)
                                if ((c & h) == 0) Mc[c] = Mc[c + h] = fmaxf(Mc[c], Mc[c + h]);
                        }
                    if (P.gsh > GLOG) {
                        float m = Mc[0];
                        for (int o = 1; o < (1 << (P.gsh - GLOG)); o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
#pragma unroll
                        for (int c = 0; c < G; ++c) Mc[c] = m;
                    }
                    float* gw = &S->gm[grp][w][up][0];
                    if (G == 2) {
                        *reinterpret_cast<float2*>(gw) = make_float2(Mc[0], Mc[1]);
                    } else {
#pragma unroll
                        for (int c = 0; c < G; c += 4)
                            *reinterpret_cast<float4*>(gw + c) = make_float4(Mc[c], Mc[c + 1], Mc[(c + 2) % G], Mc[(c + 3) % G]);
                    }
                }
            }
            if (!GROUPED) {
                const unsigned mw = __reduce_max_sync(0xffffffffu, __float_as_uint(M));
                if (lane == 0) S->red[grp][gp][ew] = __uint_as_float(mw);
            }
            asm volatile("bar.sync %0, 256;" ::"r"(1 + grp) : "memory");
            float Ms[G / 2];                              // GROUPED: group maximum for chunk 2 i + w
            if (GROUPED) {
                // the other warp of this lane quadrant swept the other sixteen columns of every chunk
                const float* go = &S->gm[grp][w ^ 1][up][0];
#pragma unroll
                for (int i = 0; i < G / 2; ++i) Ms[i] = fmaxf(w ? Mc[2 * i + 1] : Mc[2 * i], go[2 * i + w]);
            } else {
                const float4* rp = reinterpret_cast<const float4*>(&S->red[grp][gp][0]);
                const float4 m0 = rp[0], m1 = rp[1];
                M = fmaxf(fmaxf(fmaxf(m0.x, m0.y), fmaxf(m0.z, m0.w)), fmaxf(fmaxf(m1.x, m1.y), fmaxf(m1.z, m1.w)));
            }
            if constexpr (CLIP) {
                float* part = &S->cpart[grp][ew][0];
                if (quad_live) {
                    tc_fence_after();
                    const float twoD = (float)(2 * P.levels);
                    const float MAGIC = 8388608.f;             // 2^23: w * 2D + MAGIC has rint(w * 2D) in its low bits
                    const float mD = MAGIC + (float)P.levels;
                    for (int k0 = 0; k0 < P.K; k0 += 8) {
                        float acc[8];
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) acc[kk] = 0.f;
#pragma unroll
                        for (int i = 0; i < G / 2; ++i) {
                            tmem_ld32_issue(tcol + (2 * i + w) * V, r);
                            tmem_ld_wait(r);
                            const float mg = GROUPED ? Ms[i] : M;
                            const float rM = (mg > 0.f) ? (1.f / mg) : 0.f;
                            float a1k[8], dl[8];
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                a1k[kk] = P.clip_half[k0 + kk] * rM;
                                dl[kk] = -P.clip_scale[k0 + kk] * mg;          // -Delta_k
                            }
#pragma unroll
                            for (int e = 0; e < 32; ++e) {
                                const float y = __uint_as_float(r[e]);
#pragma unroll
                                for (int kk = 0; kk < 8; ++kk) {
                                    const float wv = __saturatef(fmaf(y, a1k[kk], 0.5f));
                                    const float qv = fmaf(wv, twoD, MAGIC) - mD;    // the code, as a float
                                    const float err = fmaf(qv, dl[kk], y);
                                    acc[kk] = fmaf(err, err, acc[kk]);
                                }
                            }
                        }
                        const float h1 = warp_fold8(acc, lane);
                        const int kk = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
                        if ((lane & 3) == 0 && k0 + kk < P.K) part[k0 + kk] = h1;
                    }
                    tc_fence_before();
                } else {
                    for (int k = lane; k < P.K; k += 32) part[k] = 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&S->tempty[ts]);
                asm volatile("bar.sync %0, 256;" ::"r"(1 + grp) : "memory");
                if (ew == 0) {
                    for (int k = lane; k < P.K; k += 32) {
                        float rk = 0.f;
#pragma unroll
                        for (int e8 = 0; e8 < 8; ++e8) rk += S->cpart[grp][e8][k];
                        if (P.err_rows) P.err_rows[row * P.K + k] = rk * P.norm2;
                        if (k < 32) dacc0 += (double)rk; else dacc1 += (double)rk;
                    }
                }
                continue;
            }
            // sweep 3: Delta, round / clip, pack, store
            float a1 = (M > 0.f) ? __fdividef(P.c_half, M) : 0.f;
            if (quad_live) {
                tc_fence_after();
#pragma unroll
                for (int i = 0; i < G / 2; ++i) {
                    const int c = 2 * i + w;
                    tmem_ld32_issue(tcol + c * V, r);
                    tmem_ld_wait(r);
                    if (lane_live) {
                        if (GROUPED) {
                            const float mg = Ms[i];
                            a1 = (mg > 0.f) ? __fdividef(P.c_half, mg) : 0.f;
                            // one writer per group: its first chunk, in its first lane
                            const bool writer = (P.gsh <= GLOG) ? ((c & ((1 << P.gsh) - 1)) == 0)
                                                                : (c == 0 && (lane & ((1 << (P.gsh - GLOG)) - 1)) == 0);
                            if (writer) P.scales[row * P.spr + ((up * G + c) >> P.gsh)] = P.c_scale * mg;
                        }
                        unsigned out[BITS];
                        quantize_pack32<BITS>(r, a1, out);
                        unsigned* dst = reinterpret_cast<unsigned*>(P.codes + row * P.code_row_bytes +
                                                                    (size_t)(up * G + c) * (V * BITS / 8));
                        if (BITS == 4) {
                            *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
                        } else {
                            dst[0] = out[0]; dst[1] = out[1]; dst[2] = out[2];
                        }
                        if (P.y_opt) {
                            float4* yo = reinterpret_cast<float4*>(P.y_opt + row * (long long)P.d_pad + (size_t)(up * G + c) * V);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                yo[i] = make_float4(__uint_as_float(r[4 * i]) * P.norm, __uint_as_float(r[4 * i + 1]) * P.norm,
                                                    __uint_as_float(r[4 * i + 2]) * P.norm, __uint_as_float(r[4 * i + 3]) * P.norm);
                        }
                    }
                }
                tc_fence_before();
            }
            if (!GROUPED && ew == 0 && lane == 0) P.scales[row] = P.c_scale * M;
            // the accumulators have been read for the last time: hand the TMEM stage back to the MMA issuer
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->tempty[ts]);
        }
        if (CLIP && ew == 0) {
            if (lane < P.K) atomicAdd(&P.err_sum[lane], dacc0 * (double)P.norm2);
            if (lane + 32 < P.K) atomicAdd(&P.err_sum[lane + 32], dacc1 * (double)P.norm2);
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

template <typename KernelT>
cudaError_t launch(KernelT kernel, int threads, int grid, int smem, cudaStream_t stream, bool pdl, const CUtensorMap& tmap,
                   const UvmParams& P)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
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

// Smallest G in {2, 4, 8} for which U = d' / (32 G) fits the tensor-core factor; 0 if the family does not apply.
int gbs_tc_uvm_glog(const gbs_plan* p)
{
    if (p->d_pad <= 4096) return 0;
    int gsh = 0;                                   // group = 32 * 2^gsh coordinates
    if (p->group != 0) {
        if (p->group % V != 0) return 0;
        while ((V << gsh) < p->group) ++gsh;
        if ((V << gsh) != p->group) return 0;
    }
    for (int g = 1; g <= 3; ++g) {
        const int span = V << g;
        if (p->d_pad % span != 0 || p->d % span != 0) continue;
        if (p->group != 0 && gsh > g + 5) continue;          // a group may span at most the 32 lanes of a warp
        const int U = p->d_pad / span;
        if (U > UMAX || U < 16 || p->k - 5 - g < 0) continue;
        if (get_encode() == nullptr || p->smem_optin < (int)(sizeof(Smem) + 1024)) return 0;
        return g;
    }
    return 0;
}

namespace {

// Tensor map of the rows and the parameters common to both uses of the kernel.
int uvm_prepare(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, CUtensorMap* tmap_out, UvmParams* P_out)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - 1) return (int)cudaErrorInvalidValue;      // TMA coordinates are 32-bit
    const int glog = p->uvm_glog, G = 1 << glog;
    const int U = p->d_pad / (V * G);
    // dims: v (32 values), chunk c (G), u, token; one box = chunk c of one token: U rows of 32 values
    CUtensorMap& tmap = *tmap_out;
    const cuuint64_t gdim[4] = {(cuuint64_t)V, (cuuint64_t)G, (cuuint64_t)(p->d / (V * G)), (cuuint64_t)n_rows};
    const cuuint64_t gstr[3] = {(cuuint64_t)(V * 2), (cuuint64_t)(V * G * 2), (cuuint64_t)(stride * 2)};
    const int Upad = (U + 15) & ~15;       // the contraction is padded to the MMA's K = 16; TMA zero-fills the rows
    const cuuint32_t box[4] = {V, 1, (cuuint32_t)Upad, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;

    UvmParams& P = *P_out;
    memset(&P, 0, sizeof(P));
    P.n_rows = n_rows;
    P.U = U;
    P.Upad = Upad;
    P.ksteps = Upad / 16;
    P.stage_bytes = Upad * G * V * 2;
    P.n_stages = B_BYTES / P.stage_bytes < MAX_STAGES ? B_BYTES / P.stage_bytes : MAX_STAGES;
    P.code_row_bytes = p->d_pad * p->bits / 8;
    P.d_pad = p->d_pad;
    if (p->group != 0) {
        while ((V << P.gsh) < p->group) ++P.gsh;
    }
    P.spr = p->group ? p->d_pad / p->group : 1;
    P.c_scale = p->c_scale;
    P.c_half = (float)(1.0 / (2.0 * (double)p->alpha));
    P.norm = p->norm;
    P.a_img = p->d_aimg;
    P.status = p->d_status;
    P.levels = p->levels;
    P.norm2 = (float)(1.0 / (double)p->d_pad);
    return 0;
}

}  // namespace

int gbs_tc_uvm_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream)
{
    CUtensorMap tmap;
    UvmParams P;
    const int rc = uvm_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    const int glog = p->uvm_glog;
    P.codes = (unsigned char*)codes;
    P.scales = scales;
    P.y_opt = y_opt;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = (int)(n_rows < p->sm_count ? n_rows : p->sm_count);
    const bool pdl = p->pdl != 0;
    cudaError_t e;
#define GBS_UVM_LAUNCH(B, GL)                                                                   \
    (p->group ? launch(k_tc_uvm_rq<B, GL, true, false>, threads_for(GL), grid, smem, stream, pdl, tmap, P)        \
              : launch(k_tc_uvm_rq<B, GL, false, false>, threads_for(GL), grid, smem, stream, pdl, tmap, P))
    if (p->bits == 3) {
        if (glog == 1) e = GBS_UVM_LAUNCH(3, 1);
        else if (glog == 2) e = GBS_UVM_LAUNCH(3, 2);
        else e = GBS_UVM_LAUNCH(3, 3);
    } else {
        if (glog == 1) e = GBS_UVM_LAUNCH(4, 1);
        else if (glog == 2) e = GBS_UVM_LAUNCH(4, 2);
        else e = GBS_UVM_LAUNCH(4, 3);
    }
#undef GBS_UVM_LAUNCH
    return (int)e;
}

// Clip-ratio scoring on the same front end (sweeps 1 and 2), with sweep 3 scoring instead of packing.
int gbs_tc_uvm_clip_error(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, const float* alphas, int K,
                          double* err_sum, float* err_rows, cudaStream_t stream)
{
    CUtensorMap tmap;
    UvmParams P;
    const int rc = uvm_prepare(p, x, n_rows, stride, &tmap, &P);
    if (rc != 0) return rc;
    P.K = K;
    for (int i = 0; i < K; ++i) {
        P.clip_half[i] = (float)(1.0 / (2.0 * (double)alphas[i]));
        P.clip_scale[i] = (float)((double)alphas[i] / (double)p->levels);
    }
    P.err_sum = err_sum;
    P.err_rows = err_rows;
    const int glog = p->uvm_glog;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = (int)(n_rows < p->sm_count ? n_rows : p->sm_count);
    const bool pdl = p->pdl != 0;
    cudaError_t e;
#define GBS_UVM_CLIP(GL)                                                                        \
    (p->group ? launch(k_tc_uvm_rq<4, GL, true, true>, threads_for(GL), grid, smem, stream, pdl, tmap, P)         \
              : launch(k_tc_uvm_rq<4, GL, false, true>, threads_for(GL), grid, smem, stream, pdl, tmap, P))
    if (glog == 1) e = GBS_UVM_CLIP(1);
    else if (glog == 2) e = GBS_UVM_CLIP(2);
    else e = GBS_UVM_CLIP(3);
#undef GBS_UVM_CLIP
    return (int)e;
}
