// Tensor-core inverse path of gbs_dequantize for the UV family's shapes with one scale per token:
//     xhat = (H^T yhat / sqrt(d'))[0:d],  yhat = q * Delta          (Section 2.1; inverse by the transpose,
//                                                                     Section 2.3)
// With H = A (x) H_32 (A = H_m (x) H_{2^j}, U x U) the transpose is A^T (x) H_32, and Delta is one number per
// token, so xhat = (Delta / sqrt(d')) * (A^T Q H_32) with Q the U x 32 matrix of the token's integer codes.
//   * The codes are unpacked by the epilogue warps straight into the bf16 operand tile the MMA reads
//     (same [token][u][v] layout and 64-byte swizzle the forward kernel gets from TMA).  No conversion
//     instruction is needed: the 16-bit pattern 0x4300 | k is the bf16 number 128 + k, so a field f is stored
//     as 128 + (f ^ 2^(b-1)) = q + OFF with OFF = 128 + 2^(b-1), built with shifts and masks only.
//   * A^T (Q + OFF) = A^T Q + OFF * rowsum(A^T): the second term is the same in all 32 columns of a TMEM lane,
//     so after the H_32 butterflies it sits in coordinate 0 alone (32 * OFF * rowsum) and one subtraction
//     removes it.  Every intermediate is an integer below 2^24: the rotation of the codes is exact in fp32,
//     and the only rounding is the final multiplication by Delta / sqrt(d').
//   * tcgen05.mma with the plan's image of A^T, accumulators in TMEM, H_32 in registers, 64 or 128 contiguous
//     bytes stored per thread: the kernel is bound by the output write.
// Roles: warp 0 loads the A^T image, warp 1 issues the MMAs, warps 2..17 unpack (two tiles ahead) and run
// the epilogue; warp (q, t) owns TMEM lane quadrant q and token t of every tile.  Every wait is bounded.
#include <math.h>
#include <string.h>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"
#include "gbs_tc_inv.cuh"

namespace {

constexpr int V = 32;
constexpr int UMAX = 128;
constexpr int TOK = 4;                            // tokens per tile (MMA N = 128)
constexpr int STAGES = 4;
constexpr int STAGE_COLS = TOK * V;
constexpr int TMEM_COLS = STAGES * STAGE_COLS;
constexpr int A_BYTES = UMAX * UMAX * 2;
constexpr int B_STAGE_BYTES = TOK * UMAX * V * 2;
constexpr int EPI_WARPS = 16;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int AHEAD = 2;                          // tiles unpacked ahead of the one in the epilogue

struct __align__(1024) Smem {
    unsigned char a[A_BYTES];
    unsigned char b[STAGES][B_STAGE_BYTES];
    unsigned long long full[STAGES], empty[STAGES], tfull[STAGES], tempty[STAGES];
    unsigned long long abar;
    unsigned tmem_base;
    volatile int abort_flag;
};

struct InvParams {
    long long n_rows;
    int n_groups;                 // ceil(n_rows / TOK)
    int U, Upad, ksteps;
    int d;                        // output width (multiple of 32)
    int code_row_bytes;
    float norm;                   // 1 / sqrt(d')
    const unsigned char* at_img;  // image of A^T
    const unsigned char* codes;
    const float* scales;
    void* out;
    int* status;
    float corr[UMAX];             // 32 * OFF * sum_u A[u][u']  (what the offset of the stored codes adds to coordinate 0)
};

// ---------------------------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------------------------
template <int BITS, typename OutT>
__global__ void __launch_bounds__(THREADS, 1) k_tc_uv_inv(const __grid_constant__ InvParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned tok_bytes = (unsigned)(P.Upad * V * 2);

    if (threadIdx.x == 0) {
        mbar_init(&S->abar, 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->full[s], EPI_WARPS);
            mbar_init(&S->empty[s], 1);
            mbar_init(&S->tfull[s], 1);
            mbar_init(&S->tempty[s], EPI_WARPS);
        }
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->abar, A_BYTES);
        bulk_load(S->a, P.at_img, A_BYTES, &S->abar);         // plan-owned, immutable: needs no ordering
        // programmatic dependent launch: the codes and scales may still be being written until this returns;
        // the block barrier below orders every other thread of the CTA behind it
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&S->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned tmem_base = S->tmem_base;

    if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr unsigned IDESC = instr_desc(UMAX, STAGE_COLS);
            const unsigned a_base = smem_u32(S->a);
            const unsigned long long ad0 = smem_desc(a_base, 16, 1024, 2);
            const unsigned long long bd0 = smem_desc(smem_u32(S->b[0]), tok_bytes, 512, 4);
            const unsigned ad_lo0 = (unsigned)ad0, ad_hi = (unsigned)(ad0 >> 32);
            const unsigned bd_lo0 = (unsigned)bd0, bd_hi = (unsigned)(bd0 >> 32);
            bool ok = mbar_wait(&S->abort_flag, &S->abar, 0, P.status, 6);
            int it = 0;
            for (int g = blockIdx.x; ok && g < P.n_groups; g += gridDim.x, ++it) {
                const int s = it % STAGES;
                const unsigned ph = (it / STAGES) & 1;
                if (!mbar_wait(&S->abort_flag, &S->full[s], ph, P.status, 2)) break;
                if (!mbar_wait(&S->abort_flag, &S->tempty[s], ph ^ 1, P.status, 3)) break;
                tc_fence_after();
                // only the address fields (bytes >> 4, low words) of the descriptors change between k-steps
                unsigned a_lo = ad_lo0, b_lo = bd_lo0 + (unsigned)s * (B_STAGE_BYTES >> 4);
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
    } else if (warp >= 2) {
        // ------------------------------ unpack + epilogue ------------------------------
        const int t = (warp - 2) >> 2;            // token slot inside every tile
        const int q = warp & 3;                   // TMEM lane quadrant this warp may access
        const int up = q * 32 + lane;             // row u of the operand tile it writes; output row u' it reads
        const unsigned taddr0 = tmem_base + ((unsigned)(q * 32) << 16) + t * V;
        const unsigned row_off = (unsigned)t * tok_bytes + (unsigned)up * 64u;
        const unsigned swz = (unsigned)((up >> 1) & 3);
        const float corr = P.corr[up];
        const long long row_step = (long long)gridDim.x * TOK;
        const int n_mine = (P.n_groups - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // tiles of this CTA

        // codes of tile j of this CTA -> operand tile, stage j % STAGES
        auto unpack_tile = [&](int j) -> bool {
            const int s = j % STAGES;
            if (!mbar_wait(&S->abort_flag, &S->empty[s], ((j / STAGES) & 1) ^ 1, P.status, 1)) return false;
            const long long row = ((long long)blockIdx.x + (long long)j * gridDim.x) * TOK + t;
            if (up < P.Upad) {
                uint4 chunk[4];
                if (up < P.U && row < P.n_rows) {
                    unpack_row<BITS, false>(P.codes + row * P.code_row_bytes + up * (V * BITS / 8), chunk);
                } else {
                    // rows that pad U to a multiple of 16 and tokens beyond the last: bf16 zeros (A^T has zero
                    // columns for the former, the latter are never stored)
                    chunk[0] = chunk[1] = chunk[2] = chunk[3] = make_uint4(0u, 0u, 0u, 0u);
                }
                const unsigned base = smem_u32(S->b[s]) + row_off;
#pragma unroll
                for (int c = 0; c < 4; ++c) st_shared_v4(base + ((c ^ swz) << 4), chunk[c]);
            }
            // make the generic-proxy writes visible to the tensor cores' (async proxy) reads, then signal
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->full[s]);
            return true;
        };

        bool alive = true;
        for (int j = 0; alive && j < AHEAD && j < n_mine; ++j) alive = unpack_tile(j);
        long long row = (long long)blockIdx.x * TOK + t;
        for (int it = 0; alive && it < n_mine; ++it, row += row_step) {
            if (it + AHEAD < n_mine) {
                alive = unpack_tile(it + AHEAD);
                if (!alive) break;
            }
            const int s = it % STAGES;
            if (!mbar_wait(&S->abort_flag, &S->tfull[s], (it / STAGES) & 1, P.status, 4)) break;
            unsigned r[32];
            tc_fence_after();
            tmem_ld32_issue(taddr0 + s * STAGE_COLS, r);
            tmem_ld_wait(r);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->tempty[s]);
            (void)fwht32_absmax(r);
            r[0] = __float_as_uint(__uint_as_float(r[0]) - corr);      // the offset of the stored codes
            if (row < P.n_rows && up * V < P.d) {
                const float sc = __ldg(P.scales + row) * P.norm;
                store_row32<OutT>(reinterpret_cast<OutT*>(P.out) + row * (long long)P.d + up * V, r, sc, 0.f);
            }
        }
    }

    // ---- teardown: every role leaves its loop (normally or after a wait expired), then TMEM is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <typename KernelT>
cudaError_t launch(KernelT kernel, int grid, int smem, cudaStream_t stream, bool pdl, const InvParams& P)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
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
    return cudaLaunchKernelEx(&cfg, kernel, P);
}

}  // namespace

// The plans this path serves: the UV family's shapes with one symmetric scale per token.
bool gbs_tc_uvinv_supported(const gbs_plan* p)
{
    return p->variant == GBS_VARIANT_TC_UV && p->group == 0 && !p->asym && p->d_aimg_t != nullptr &&
           p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

int gbs_tc_uvinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                            int out_dtype, cudaStream_t stream)
{
    if (n_rows > (int64_t)0x7fffffff - TOK) return (int)cudaErrorInvalidValue;
    InvParams P;
    memset(&P, 0, sizeof(P));
    const int U = p->d_pad / V;
    P.n_rows = n_rows;
    P.n_groups = (int)((n_rows + TOK - 1) / TOK);
    P.U = U;
    P.Upad = (U + 15) & ~15;
    P.ksteps = P.Upad / 16;
    P.d = p->d;
    P.code_row_bytes = p->d_pad * p->bits / 8;
    P.norm = p->norm;
    P.at_img = p->d_aimg_t;
    P.codes = (const unsigned char*)codes;
    P.scales = scales;
    P.out = out;
    P.status = p->d_status;
    const float off = 128.f + (float)(1 << (p->bits - 1));
    for (int u = 0; u < UMAX; ++u) P.corr[u] = u < U ? 32.f * off * (float)p->a_colsum[u] : 0.f;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = P.n_groups < p->sm_count ? P.n_groups : p->sm_count;
    const bool pdl = p->pdl != 0;
    cudaError_t e;
    if (out_dtype == GBS_DTYPE_F32) {
        if (p->bits == 3) e = launch(k_tc_uv_inv<3, float>, grid, smem, stream, pdl, P);
        else e = launch(k_tc_uv_inv<4, float>, grid, smem, stream, pdl, P);
    } else {
        if (p->bits == 3) e = launch(k_tc_uv_inv<3, __nv_bfloat16>, grid, smem, stream, pdl, P);
        else e = launch(k_tc_uv_inv<4, __nv_bfloat16>, grid, smem, stream, pdl, P);
    }
    return (int)e;
}
