// gbs_dequantize with inverse rotation for the full Paley order (d' = m): xhat = (H_m^T yhat / sqrt(m))[0:d], with
// yhat = q * Delta (Section 2.1; rotations are undone by the transpose, Section 2.3.1).
//
// Like the forward direction there is no fast transform, so Xhat = (Delta / sqrt(m)) * (Q H_m) is a dense contraction
// on the tensor cores: A = the integer codes of 128 token rows, unpacked by four warps into bf16 (exact: |q| <= 7) in
// the K-major 128-byte-swizzled tile layout; B = 64 x 256 pieces of the plan's bf16 image of H_m read as an N-major
// operand (row = rotated coordinate k, contiguous along the output coordinate n), so the image of the transpose is
// not needed.  All sums are integers below 2^24: the fp32 accumulators are exact and the product with
// Delta / sqrt(m) is the only rounding.  TMEM lane = token; a thread scales and stores its token's 256 outputs of a
// block while the next block's MMAs run on the other half of TMEM.  Every wait is bounded.
#include <math.h>
#include <string.h>

#include <mutex>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int TM = 128;                 // tokens per tile (MMA M)
constexpr int BN = 256;                 // output coordinates per block (MMA N)
constexpr int KC = 64;                  // rotated coordinates per stage
constexpr int STAGES = 4;
constexpr int A_STAGE = TM * KC * 2;    // 16 KB: codes as bf16
constexpr int B_STAGE = KC * BN * 2;    // 32 KB: four 64 x 64 pieces of H_m
constexpr int UNPACK_WARPS = 4, EPI_WARPS = 4;
constexpr int THREADS = 32 * (2 + UNPACK_WARPS + EPI_WARPS);
constexpr int TMEM_COLS = 512;

struct __align__(1024) Smem {
    unsigned char a[STAGES][A_STAGE];
    unsigned char b[STAGES][B_STAGE];
    unsigned long long full[STAGES], empty[STAGES], tfull[2], tempty[2];
    unsigned tmem_base;
    volatile int abort_flag;
};

struct DenseInvParams {
    long long n_rows;
    int n_tiles;
    int m, d;
    int nblk;                     // ceil(d / 256)
    int n_last;                   // width of the last block, rounded up to 16
    int kchunks;                  // ceil(m / 64)
    int ksteps_last;
    int code_row_bytes;
    float norm;                   // 1 / sqrt(m)
    const unsigned char* codes;
    const float* scales;
    void* out;
    int* status;
};

__device__ __forceinline__ void st_shared_v4(unsigned addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// bf16 bit pattern of a small integer (exact for |q| <= 256)
__device__ __forceinline__ unsigned bf16_of_int(int q) { return __float_as_uint((float)q) >> 16; }

template <int BITS, typename OutT>
__global__ void __launch_bounds__(THREADS, 1) k_tc_dense_inv(const __grid_constant__ CUtensorMap hmap,
                                                             const __grid_constant__ DenseInvParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->full[s], 1 + UNPACK_WARPS);          // the TMA's expect-tx arrival and the four unpack warps
            mbar_init(&S->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&S->tfull[i], 1);
            mbar_init(&S->tempty[i], EPI_WARPS);
        }
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&S->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = S->tmem_base;
    const int n_mine = ((int)blockIdx.x < P.n_tiles) ? (P.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

    if (warp == 0) {
        // ------------------------------ TMA producer: pieces of H_m ------------------------------
        if (lane == 0) {
            int c = 0;
            bool ok = true;
            for (int i = 0; ok && i < n_mine; ++i)
                for (int nb = 0; ok && nb < P.nblk; ++nb)
                    for (int kc = 0; kc < P.kchunks; ++kc, ++c) {
                        const int s = c % STAGES;
                        if (!mbar_wait(&S->abort_flag, &S->empty[s], ((c / STAGES) & 1) ^ 1, P.status, 1)) { ok = false; break; }
                        mbar_arrive_expect_tx(&S->full[s], B_STAGE);
                        for (int j = 0; j < BN / 64; ++j)        // 64 output coordinates x 64 rotated coordinates each
                            tma_load_2d(S->b[s] + j * (KC * 128), &hmap, &S->full[s], nb * BN + j * 64, kc * KC);
                    }
            // (a stage's barrier also counts the unpacking warps, which may have left: the time limit ends the wait)
            if (!ok) drain_copies(S->full, STAGES, c);
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const unsigned idesc_full = instr_desc(TM, BN, true);
            const unsigned idesc_last = instr_desc(TM, P.n_last, true);
            int c = 0, nb_count = 0;
            bool ok = true;
            for (int i = 0; ok && i < n_mine; ++i)
                for (int nb = 0; ok && nb < P.nblk; ++nb, ++nb_count) {
                    const int buf = nb_count & 1;
                    const unsigned idesc = (nb == P.nblk - 1) ? idesc_last : idesc_full;
                    if (!mbar_wait(&S->abort_flag, &S->tempty[buf], ((nb_count >> 1) & 1) ^ 1, P.status, 3)) { ok = false; break; }
                    tc_fence_after();
                    for (int kc = 0; kc < P.kchunks; ++kc, ++c) {
                        const int s = c % STAGES;
                        if (!mbar_wait(&S->abort_flag, &S->full[s], (c / STAGES) & 1, P.status, 2)) { ok = false; break; }
                        tc_fence_after();
                        // A: K-major, one 128-byte line per token, 32 bytes per k-step.  B: N-major, atoms of 8 rotated
                        // coordinates x 64 output coordinates (1024 bytes), the next 64 output coordinates 8 KB away;
                        // a k-step is two atoms.
                        const unsigned long long ad = smem_desc(smem_u32(S->a[s]), 16, 1024, 2);
                        const unsigned long long bd = smem_desc(smem_u32(S->b[s]), KC * 128, 1024, 2);
                        const int ks_n = (kc == P.kchunks - 1) ? P.ksteps_last : KC / 16;
                        for (int ks = 0; ks < ks_n; ++ks)
                            umma_f16(tmem_base + buf * BN, ad + (unsigned long long)(2 * ks), bd + (unsigned long long)(128 * ks),
                                     idesc, (kc | ks) != 0 ? 1u : 0u);
                        umma_commit(&S->empty[s]);
                    }
                    if (ok) umma_commit(&S->tfull[buf]);
                }
        }
    } else if (warp < 2 + UNPACK_WARPS) {
        // ------------------------------ unpack: one thread = one token row of the A tile ------------------------------
        // The 64 codes of a stage are 8 * BITS bytes of the row, at any byte offset (rows of m * BITS / 8 bytes start
        // wherever they start): the thread fetches the aligned words that cover them one stage ahead (the loads of the
        // next stage are in flight while it waits for its buffer) and shifts them into place.
        constexpr int NW = 2 * BITS + 1;          // aligned words that cover 8 * BITS bytes at any offset
        const int r = (warp - 2) * 32 + lane;
        int c = 0;
        bool ok = true;
        unsigned raw[NW];
        auto fetch = [&](const unsigned char* crow, bool live, int kc) {
            const int k0 = kc * KC;
            const unsigned char* src = crow + (long long)k0 * BITS / 8;
            const unsigned* w0 = reinterpret_cast<const unsigned*>(reinterpret_cast<uintptr_t>(src) & ~(uintptr_t)3);
            const unsigned char* end = crow + P.code_row_bytes;
#pragma unroll
            for (int i = 0; i < NW; ++i)          // words wholly beyond the row are not read (the last row ends the buffer)
                raw[i] = (live && reinterpret_cast<const unsigned char*>(w0 + i) < end) ? __ldg(w0 + i) : 0u;
        };
        for (int i = 0; ok && i < n_mine; ++i) {
            const long long row = ((long long)blockIdx.x + (long long)i * gridDim.x) * TM + r;
            const bool live = row < P.n_rows;
            const unsigned char* crow = P.codes + (live ? row : 0) * P.code_row_bytes;
            const unsigned sh = (unsigned)((reinterpret_cast<uintptr_t>(crow) & 3u) * 8u);   // kc * KC * BITS / 8 is a multiple of 4
            fetch(crow, live, 0);
            for (int nb = 0; ok && nb < P.nblk; ++nb)
                for (int kc = 0; kc < P.kchunks; ++kc, ++c) {
                    unsigned f[2 * BITS];         // the stage's 8 * BITS bytes, in place
#pragma unroll
                    for (int w = 0; w < 2 * BITS; ++w) f[w] = __funnelshift_r(raw[w], raw[w + 1], sh);
                    {
                        const int kn = kc + 1 < P.kchunks ? kc + 1 : 0;      // next stage (of this block or the next)
                        if (kc + 1 < P.kchunks || nb + 1 < P.nblk) fetch(crow, live, kn);
                    }
                    const int s = c % STAGES;
                    ok = mbar_wait(&S->abort_flag, &S->empty[s], ((c / STAGES) & 1) ^ 1, P.status, 1);
                    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                    const unsigned base = smem_u32(S->a[s]) + (unsigned)r * 128u;
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {            // eight 16-byte chunks of eight codes each
                        unsigned w[4] = {0u, 0u, 0u, 0u};
                        if (kc * KC + ch * 8 < P.m) {           // m is a multiple of 8: a chunk is whole or beyond the end
                            // the chunk's 8 * BITS bits start at bit ch * 8 * BITS of f
                            unsigned fld;
                            if (BITS == 4) fld = f[ch];
                            else fld = __funnelshift_r(f[(ch * 24) >> 5], f[((ch * 24) >> 5) + (((ch * 24) & 31) > 8 ? 1 : 0)], (ch * 24) & 31);   // 24 bits
#pragma unroll
                            for (int e = 0; e < 8; e += 2) {
                                const int q0 = ((int)(fld << (32 - BITS * (e + 1)))) >> (32 - BITS);
                                const int q1 = ((int)(fld << (32 - BITS * (e + 2)))) >> (32 - BITS);
                                w[e >> 1] = bf16_of_int(q0) | (bf16_of_int(q1) << 16);
                            }
                        }
                        st_shared_v4(base + (unsigned)((ch ^ (r & 7)) << 4), make_uint4(w[0], w[1], w[2], w[3]));
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&S->full[s]);
                }
        }
    } else {
        // ------------------------------ epilogue: one thread = one token ------------------------------
        const int q = warp & 3;
        const unsigned lane_base = tmem_base + ((unsigned)(q * 32) << 16);
        int nb_count = 0;
        bool ok = true;
        for (int i = 0; ok && i < n_mine; ++i) {
            const long long row = ((long long)blockIdx.x + (long long)i * gridDim.x) * TM + q * 32 + lane;
            const bool live = row < P.n_rows;
            const float sc = live ? __ldg(P.scales + row) * P.norm : 0.f;
            OutT* orow = reinterpret_cast<OutT*>(P.out) + row * (long long)P.d;
            for (int nb = 0; ok && nb < P.nblk; ++nb, ++nb_count) {
                const int buf = nb_count & 1;
                if (!mbar_wait(&S->abort_flag, &S->tfull[buf], (nb_count >> 1) & 1, P.status, 4)) { ok = false; break; }
                tc_fence_after();
                const int width = (P.d - nb * BN) < BN ? (P.d - nb * BN) : BN;
                for (int c0 = 0; c0 < width; c0 += 32) {
                    unsigned rr[32];
                    tmem_ld32_issue(lane_base + (unsigned)(buf * BN + c0), rr);
                    tmem_ld_wait(rr);
                    if (live && c0 + 32 <= width) {                 // rows of d elements, d a multiple of 8: 16-byte stores
                        if (sizeof(OutT) == 4) {
                            float4* o4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(orow) + nb * BN + c0);
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                o4[e] = make_float4(__uint_as_float(rr[4 * e]) * sc, __uint_as_float(rr[4 * e + 1]) * sc,
                                                    __uint_as_float(rr[4 * e + 2]) * sc, __uint_as_float(rr[4 * e + 3]) * sc);
                        } else {
                            uint4* o4 = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(orow) + nb * BN + c0);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                unsigned w[4];
#pragma unroll
                                for (int h = 0; h < 4; ++h) {
                                    const __nv_bfloat162 v2 = __floats2bfloat162_rn(__uint_as_float(rr[8 * e + 2 * h]) * sc,
                                                                                    __uint_as_float(rr[8 * e + 2 * h + 1]) * sc);
                                    w[h] = *reinterpret_cast<const unsigned*>(&v2);
                                }
                                o4[e] = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                    } else if (live) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c0 + e < width) {
                                const float v = __uint_as_float(rr[e]) * sc;
                                if (sizeof(OutT) == 4) reinterpret_cast<float*>(orow)[nb * BN + c0 + e] = v;
                                else reinterpret_cast<__nv_bfloat16*>(orow)[nb * BN + c0 + e] = __float2bfloat16_rn(v);
                            }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&S->tempty[buf]);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

bool gbs_tc_denseinv_supported(const gbs_plan* p)
{
    return p->variant == GBS_VARIANT_TC_DENSE && get_encode() != nullptr && p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

int gbs_tc_denseinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                               int out_dtype, cudaStream_t stream)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - TM) return (int)cudaErrorInvalidValue;
    CUtensorMap hmap;
    const cuuint32_t estr[2] = {1, 1};
    const cuuint64_t gdim[2] = {(cuuint64_t)p->m, (cuuint64_t)p->m};         // inner: input coordinate n, outer: rotated k
    const cuuint64_t gstr[1] = {(cuuint64_t)(p->m * 2)};
    const cuuint32_t box[2] = {64, KC};
    if (encode(&hmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->d_aimg, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return (int)cudaErrorInvalidValue;
    DenseInvParams P;
    memset(&P, 0, sizeof(P));
    P.n_rows = n_rows;
    P.n_tiles = (int)((n_rows + TM - 1) / TM);
    P.m = p->m;
    P.d = p->d;
    P.nblk = (p->d + BN - 1) / BN;
    P.n_last = ((p->d - (P.nblk - 1) * BN) + 15) & ~15;
    P.kchunks = (p->m + KC - 1) / KC;
    P.ksteps_last = ((p->m - (P.kchunks - 1) * KC) + 15) / 16;
    P.code_row_bytes = p->m * p->bits / 8;
    P.norm = p->norm;
    P.codes = (const unsigned char*)codes;
    P.scales = scales;
    P.out = out;
    P.status = p->d_status;
    const int smem = (int)sizeof(Smem) + 1024;
    typedef void (*Kernel)(const CUtensorMap, const DenseInvParams);
    Kernel kernel = p->bits == 3 ? (out_dtype == GBS_DTYPE_F32 ? (Kernel)k_tc_dense_inv<3, float> : (Kernel)k_tc_dense_inv<3, __nv_bfloat16>)
                                 : (out_dtype == GBS_DTYPE_F32 ? (Kernel)k_tc_dense_inv<4, float> : (Kernel)k_tc_dense_inv<4, __nv_bfloat16>);
    {
        // opt in to the large dynamic shared memory once per device and instantiation (not a stream operation)
        static std::mutex mu;
        static bool done[64][4] = {{false}};
        const int ki = (p->bits - 3) * 2 + (out_dtype == GBS_DTYPE_F32 ? 0 : 1);
        std::lock_guard<std::mutex> lock(mu);
        if (!(p->device >= 0 && p->device < 64 && done[p->device][ki])) {
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return (int)e;
            if (p->device >= 0 && p->device < 64) done[p->device][ki] = true;
        }
    }
    const int grid = P.n_tiles < p->sm_count ? P.n_tiles : p->sm_count;
    kernel<<<grid, THREADS, smem, stream>>>(hmap, P);
    return (int)cudaGetLastError();
}
