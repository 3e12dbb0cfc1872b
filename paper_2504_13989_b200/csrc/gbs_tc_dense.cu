// Tensor-core family "DENSE": d' = m, the rotation is the full Paley matrix H_m itself (no Sylvester factor).
//
// Section 5.2.2 names the case: a width of 1536 admits no useful power-of-two split, but 1536 + 8 = 1544 = 1543 + 1
// with 1543 a prime = 3 (mod 4), so Algorithm 2 gives a Hadamard matrix of exactly the expanded order.  There is no
// fast transform for it; Y = X_pad H_m^T is a dense contraction with a +-1 matrix, which is what tensor cores are
// for: bf16 x (+-1) products are exact, the accumulation is fp32 in TMEM.
//
//   * A tile is 256 token rows, two sub-tiles of 128 (MMA M = 128: TMEM lane = token).  The m output coordinates are
//     produced in blocks of 256 (MMA N; the last block is narrower), the contraction runs over chunks of 64 input
//     coordinates through a ring of shared-memory stages: two X chunks (128 x 64 each, TMA, columns beyond d
//     zero-filled = the zero-pad expansion of Section 4.2) and ONE H chunk (256 x 64 from the plan's bf16 image of H_m,
//     rows and columns beyond m zero-filled) that both sub-tiles contract with: the kernel is bound by the L2
//     bandwidth that feeds these stages, and sharing the H chunk takes a third of that traffic away.
//   * TMEM lane t holds coordinates of token t only, so one thread owns one token: max|.|, Delta, rounding, clipping
//     and packing (Sections 2.1, 3.1) are thread-local.  A token's m fp32 values do not fit in TMEM (512 columns), so
//     the tile is contracted TWICE: the first sweep over the output blocks only takes max|.|, the second quantizes.
//     The two sub-tiles' accumulators (256 columns each) fill TMEM, so a block's epilogue (short against its 2 x 100
//     MMAs) and the next block's MMAs take turns.
//   * The kernel is bound by the tensor pipe (2 * 2 * m^2 flops per token against 2 d + m b / 8 bytes), as the method
//     itself is for this order: the paper fuses such a matrix into the weights offline where it can.
// Every wait is bounded; an expired wait records a code in the plan's status word.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int TM = 128;                 // tokens per MMA (M)
constexpr int MAX_SUB = 2;              // 128-token sub-tiles per CTA tile (1 or 2): they share every H chunk on chip
constexpr int BN = 256;                 // output coordinates per block
constexpr int KC = 64;                  // input coordinates per stage (one 128-byte swizzled line of bf16)
constexpr int STAGES = 3;              // 3 x (2 x 16 + 32) KB
constexpr int A_STAGE = TM * KC * 2;    // 16 KB per sub-tile
constexpr int B_STAGE = BN * KC * 2;    // 32 KB
constexpr int THREADS = 32 * (2 + 4 * MAX_SUB);
constexpr int TMEM_COLS = 512;

struct __align__(1024) Smem {
    unsigned char a[STAGES][MAX_SUB][A_STAGE];
    unsigned char b[STAGES][B_STAGE];
    unsigned long long full[STAGES], empty[STAGES], tfull, tempty;
    unsigned tmem_base;
    volatile int abort_flag;
};

struct DenseParams {
    long long n_rows;
    int n_tiles;
    int m;                        // d' = order of H_m
    int nblk;                     // ceil(m / 256)
    int n_last;                   // width of the last block, rounded up to 16
    int kchunks;                  // ceil(m / 64)
    int ksteps_last;              // MMAs (K = 16) of the last chunk
    int code_row_bytes;
    float c_scale, c_half, norm;
    unsigned char* codes;
    float* scales;
    float* y_opt;
    int* status;
};

// The first `nbytes` of a thread's NW packed words to a row position of any alignment (rows of m * bits / 8 bytes
// start wherever they start: 579-byte rows at m = 1544, b = 3).
template <int NW>
__device__ __forceinline__ void store_bytes(unsigned char* dst, const unsigned (&w)[NW], int nbytes)
{
    if ((reinterpret_cast<uintptr_t>(dst) & 3u) == 0 && nbytes == 4 * NW) {
#pragma unroll
        for (int i = 0; i < NW; ++i) reinterpret_cast<unsigned*>(dst)[i] = w[i];
    } else {
#pragma unroll
        for (int i = 0; i < 4 * NW; ++i)
            if (i < nbytes) dst[i] = (unsigned char)(w[i >> 2] >> (8 * (i & 3)));
    }
}

// SUB = 2: a 256-token tile, the H chunk of a stage contracted with both sub-tiles (a third less L2 traffic per token;
// pays when the batch gives every SM at least a tile of that size).  SUB = 1: 128-token tiles, the four warps of the
// second sub-tile idle.
template <int BITS, int SUB>
__global__ void __launch_bounds__(THREADS, 1) k_tc_dense_rq(const __grid_constant__ CUtensorMap xmap,
                                                            const __grid_constant__ CUtensorMap hmap,
                                                            const __grid_constant__ DenseParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TT = TM * SUB;                   // tokens per CTA tile
    constexpr int EPI_WARPS = 4 * SUB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->full[s], 1);
            mbar_init(&S->empty[s], 1);
        }
        mbar_init(&S->tfull, 1);
        mbar_init(&S->tempty, EPI_WARPS);
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&S->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = S->tmem_base;
    const int n_mine = ((int)blockIdx.x < P.n_tiles) ? (P.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int blocks_per_tile = 2 * P.nblk;               // two sweeps over the output blocks

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int c = 0;                                     // stage uses so far
            bool ok = true;
            for (int i = 0; ok && i < n_mine; ++i) {
                const int row0 = ((int)blockIdx.x + i * (int)gridDim.x) * TT;
                for (int bl = 0; ok && bl < blocks_per_tile; ++bl) {
                    const int n0 = (bl % P.nblk) * BN;
                    for (int kc = 0; kc < P.kchunks; ++kc, ++c) {
                        const int s = c % STAGES;
                        if (!mbar_wait(&S->abort_flag, &S->empty[s], ((c / STAGES) & 1) ^ 1, P.status, 1)) { ok = false; break; }
                        mbar_arrive_expect_tx(&S->full[s], SUB * A_STAGE + B_STAGE);
                        for (int u = 0; u < SUB; ++u) tma_load_2d(S->a[s][u], &xmap, &S->full[s], kc * KC, row0 + u * TM);
                        tma_load_2d(S->b[s], &hmap, &S->full[s], kc * KC, n0);
                    }
                }
            }
            if (!ok) drain_copies(S->full, STAGES, c);
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const unsigned idesc_full = instr_desc(TM, BN, false);
            const unsigned idesc_last = instr_desc(TM, P.n_last, false);
            int c = 0, nb_count = 0;
            bool ok = true;
            for (int i = 0; ok && i < n_mine; ++i) {
                for (int bl = 0; ok && bl < blocks_per_tile; ++bl, ++nb_count) {
                    const unsigned idesc = (bl % P.nblk == P.nblk - 1) ? idesc_last : idesc_full;
                    // the two accumulators (one per sub-tile) fill all of TMEM: the next block waits for the epilogue
                    if (!mbar_wait(&S->abort_flag, &S->tempty, (nb_count & 1) ^ 1, P.status, 3)) { ok = false; break; }
                    tc_fence_after();
                    for (int kc = 0; kc < P.kchunks; ++kc, ++c) {
                        const int s = c % STAGES;
                        if (!mbar_wait(&S->abort_flag, &S->full[s], (c / STAGES) & 1, P.status, 2)) { ok = false; break; }
                        tc_fence_after();
                        const unsigned long long bd = smem_desc(smem_u32(S->b[s]), 16, 1024, 2);
                        const int ks_n = (kc == P.kchunks - 1) ? P.ksteps_last : KC / 16;
                        for (int u = 0; u < SUB; ++u) {
                            const unsigned long long ad = smem_desc(smem_u32(S->a[s][u]), 16, 1024, 2);
                            for (int ks = 0; ks < ks_n; ++ks)
                                umma_f16(tmem_base + u * BN, ad + (unsigned long long)(2 * ks), bd + (unsigned long long)(2 * ks),
                                         idesc, (kc | ks) != 0 ? 1u : 0u);
                        }
                        umma_commit(&S->empty[s]);
                    }
                    if (ok) umma_commit(&S->tfull);
                }
            }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // ------------------------------ epilogue: one thread = one token ------------------------------
        const int q = warp & 3;                        // TMEM lane quadrant this warp may access
        const int sub = (warp - 2) >> 2;               // which 128-token sub-tile (= which accumulator) it serves
        const unsigned lane_base = tmem_base + ((unsigned)(q * 32) << 16) + (unsigned)(sub * BN);
        int nb_count = 0;
        bool ok = true;
        for (int i = 0; ok && i < n_mine; ++i) {
            const long long row = ((long long)blockIdx.x + (long long)i * gridDim.x) * TT + sub * TM + q * 32 + lane;
            const bool live = row < P.n_rows;
            float M = 0.f, a1 = 0.f;
            for (int bl = 0; ok && bl < blocks_per_tile; ++bl, ++nb_count) {
                const int nb = bl % P.nblk;
                const bool second = bl >= P.nblk;
                if (!mbar_wait(&S->abort_flag, &S->tfull, nb_count & 1, P.status, 4)) { ok = false; break; }
                tc_fence_after();
                if (second && nb == 0) a1 = __fdividef(P.c_half, fmaxf(M, 1e-30f));
                const int width = (P.m - nb * BN) < BN ? (P.m - nb * BN) : BN;        // live coordinates of this block
                for (int c0 = 0; c0 < width; c0 += 32) {
                    unsigned r[32];
                    tmem_ld32_issue(lane_base + (unsigned)c0, r);
                    tmem_ld_wait(r);
                    const int n_here = (width - c0) < 32 ? (width - c0) : 32;
                    if (n_here < 32) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (e >= n_here) r[e] = 0u;                                // columns no MMA wrote
                    }
                    if (!second) {
                        M = fmaxf(M, absmax32(r));
                    } else if (live) {
                        unsigned out[BITS];
                        quantize_pack32<BITS>(r, a1, out);
                        unsigned char* dst = P.codes + row * P.code_row_bytes + (long long)(nb * BN + c0) * BITS / 8;
                        store_bytes(dst, out, n_here * BITS / 8);
                        if (P.y_opt) {
                            float* yo = P.y_opt + row * (long long)P.m + nb * BN + c0;
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (e < n_here) yo[e] = __uint_as_float(r[e]) * P.norm;
                        }
                    }
                }
                // this block's accumulators have been read: hand TMEM back to the MMA issuer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S->tempty);
            }
            if (ok && live) P.scales[row] = P.c_scale * M;
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

// The plans this family serves: d' = m (no Sylvester factor), a large Paley order, one scale per token.
bool gbs_tc_dense_supported(const gbs_plan* p)
{
    return p->k == 0 && p->m >= 128 && p->m % 8 == 0 && p->d % 8 == 0 && p->group == 0 && !p->asym &&
           get_encode() != nullptr && p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

// bf16 image of H_m, row-major (row = output coordinate, column = input coordinate): m * m * 2 bytes.
void gbs_tc_dense_image(const int8_t* hm, int m, unsigned short* img)
{
    for (size_t i = 0; i < (size_t)m * m; ++i) img[i] = hm[i] < 0 ? 0xBF80 : 0x3F80;
}

int gbs_tc_dense_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                                 float* scales, float* y_opt, cudaStream_t stream)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - TM * MAX_SUB) return (int)cudaErrorInvalidValue;
    CUtensorMap xmap, hmap;
    const cuuint32_t estr[2] = {1, 1};
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)p->d, (cuuint64_t)n_rows};
        const cuuint64_t gstr[1] = {(cuuint64_t)(stride * 2)};
        const cuuint32_t box[2] = {KC, TM};          // one sub-tile per copy
        if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), gdim, gstr, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return (int)cudaErrorInvalidValue;
    }
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)p->m, (cuuint64_t)p->m};
        const cuuint64_t gstr[1] = {(cuuint64_t)(p->m * 2)};
        const cuuint32_t box[2] = {KC, BN};
        if (encode(&hmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->d_aimg, gdim, gstr, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return (int)cudaErrorInvalidValue;
    }
    DenseParams P;
    memset(&P, 0, sizeof(P));
    P.n_rows = n_rows;
    // tile size: a 256-token tile costs about 1.8 x a 128-token tile; take it when it gives fewer, cheaper rounds
    const long long t1 = (n_rows + TM - 1) / TM, t2 = (n_rows + 2 * TM - 1) / (2 * TM);
    const long long w1 = (t1 + p->sm_count - 1) / p->sm_count, w2 = (t2 + p->sm_count - 1) / p->sm_count;
    const int sub = (9 * w2 < 5 * w1) ? 2 : 1;
    P.n_tiles = (int)(sub == 2 ? t2 : t1);
    P.m = p->m;
    P.nblk = (p->m + BN - 1) / BN;
    P.n_last = ((p->m - (P.nblk - 1) * BN) + 15) & ~15;
    P.kchunks = (p->m + KC - 1) / KC;
    P.ksteps_last = ((p->m - (P.kchunks - 1) * KC) + 15) / 16;
    P.code_row_bytes = p->m * p->bits / 8;
    P.c_scale = p->c_scale;
    P.c_half = (float)(1.0 / (2.0 * (double)p->alpha));
    P.norm = p->norm;
    P.codes = (unsigned char*)codes;
    P.scales = scales;
    P.y_opt = y_opt;
    P.status = p->d_status;
    const int smem = (int)sizeof(Smem) + 1024;
    {
        // opt in to the large dynamic shared memory once per device (not a stream operation)
        static std::mutex mu;
        static bool done[64] = {false};
        std::lock_guard<std::mutex> lock(mu);
        if (!(p->device >= 0 && p->device < 64 && done[p->device])) {
            cudaError_t e = cudaFuncSetAttribute(k_tc_dense_rq<3, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_dense_rq<4, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_dense_rq<3, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tc_dense_rq<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return (int)e;
            if (p->device >= 0 && p->device < 64) done[p->device] = true;
        }
    }
    const int grid = P.n_tiles < p->sm_count ? P.n_tiles : p->sm_count;
    if (sub == 2) {
        if (p->bits == 3) k_tc_dense_rq<3, 2><<<grid, THREADS, smem, stream>>>(xmap, hmap, P);
        else k_tc_dense_rq<4, 2><<<grid, THREADS, smem, stream>>>(xmap, hmap, P);
    } else {
        if (p->bits == 3) k_tc_dense_rq<3, 1><<<grid, THREADS, smem, stream>>>(xmap, hmap, P);
        else k_tc_dense_rq<4, 1><<<grid, THREADS, smem, stream>>>(xmap, hmap, P);
    }
    return (int)cudaGetLastError();
}
