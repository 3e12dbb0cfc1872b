// Tensor-core inverse path of gbs_dequantize for d' = 128 rows (KV entries) with one scale per row
// (group 0 or 128), symmetric or asymmetric quantizer:
//     xhat = (H_128^T yhat / sqrt(128))[0:d],   yhat = q * Delta   or   code * Delta + lo
// (Section 2.1 / 5.1; inverse by the transpose, Section 2.3; H_128 of Eq. (1) is symmetric).
// 128 rows form a tile and Xhat = C H_128 is one tcgen05 contraction per tile, as in the forward ROW kernel:
// A = the tile of codes as bf16, written by the thread that owns the row into the K-major, 128-byte-swizzled
// layout the MMA reads; B = the plan's image of H_128; accumulators in TMEM, lane r = row r.  A field f is
// stored as the bf16 number 128 + (f ^ 2^(b-1)) = q + OFF (asymmetric: 128 + code) with shifts and masks
// only; the offset adds OFF * colsum(H_128) = 128 * OFF to column 0 and nothing elsewhere, which one
// subtraction removes, and the zero point adds 128 * lo there.  All intermediates are small integers: the
// rotation is exact in fp32.
// Roles: warp 0 loads the image, warp 1 issues the MMAs, warps 2..17 are four groups of four warps; group e
// owns stage e and every fourth tile: it unpacks a tile, reads its accumulators when they are complete,
// unpacks its next tile at once (so that the tensor cores work on it meanwhile) and then scales and stores.
#include <math.h>
#include <string.h>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"
#include "gbs_tc_inv.cuh"

namespace {

constexpr int DP = 128;
constexpr int TILE = 128;
constexpr int STAGES = 4;
constexpr int TILE_BYTES = TILE * DP * 2;
constexpr int H_BYTES = DP * DP * 2;
constexpr int EPI_WARPS = 4 * STAGES;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int TMEM_COLS = 512;

struct __align__(1024) Smem {
    unsigned char h[H_BYTES];
    unsigned char x[STAGES][TILE_BYTES];
    unsigned long long full[STAGES], empty[STAGES], tfull[STAGES], tempty[STAGES];
    unsigned long long hbar;
    unsigned tmem_base;
    volatile int abort_flag;
};

struct RowInvParams {
    long long n_rows;
    long long n_tiles;
    int d;                        // output width
    int code_row_bytes;           // 128 * bits / 8
    float norm;                   // 1 / sqrt(128)
    float corr;                   // 128 * OFF
    const unsigned char* h_img;
    const unsigned char* codes;
    const float* scales;          // Delta per row, or (Delta, lo) per row
    void* out;
    int* status;
};

template <int BITS, bool ASYM, typename OutT>
__global__ void __launch_bounds__(THREADS, 1) k_tc_row_inv(const __grid_constant__ RowInvParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(&S->hbar, 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->full[s], 4);             // the four warps of the stage's group
            mbar_init(&S->empty[s], 1);
            mbar_init(&S->tfull[s], 1);
            mbar_init(&S->tempty[s], 4);
        }
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->hbar, H_BYTES);
        bulk_load(S->h, P.h_img, H_BYTES, &S->hbar);          // plan-owned, immutable: needs no ordering
        // programmatic dependent launch: codes and scales may still be being written until this returns; the
        // block barrier below orders every other thread of the CTA behind it
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
            constexpr unsigned IDESC = instr_desc(TILE, DP, false);
            const unsigned h_base = smem_u32(S->h);
            const unsigned long long xd0 = smem_desc(smem_u32(S->x[0]), 16, 1024, 2);
            const unsigned long long hd0 = smem_desc(h_base, 16, 1024, 2);
            const unsigned xd_lo0 = (unsigned)xd0, xd_hi = (unsigned)(xd0 >> 32);
            const unsigned hd_lo0 = (unsigned)hd0, hd_hi = (unsigned)(hd0 >> 32);
            bool ok = mbar_wait(&S->abort_flag, &S->hbar, 0, P.status, 6);
            int it = 0;
            for (long long t = blockIdx.x; ok && t < P.n_tiles; t += gridDim.x, ++it) {
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
    } else if (warp >= 2) {
        // ------------------------------ unpack + epilogue ------------------------------
        const int e = (warp - 2) >> 2;            // group = stage
        const int q = warp & 3;                   // TMEM lane quadrant
        const int rt = q * 32 + lane;             // row inside the tile = TMEM lane
        const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + e * DP;
        const unsigned x_row = smem_u32(S->x[e]) + (unsigned)rt * 128u;
        const unsigned swz = (unsigned)(rt & 7);
        const long long t_step = (long long)STAGES * gridDim.x;

        // codes of row rt of tile t -> the two 128-byte halves of the operand row (n-th tile of this group)
        auto unpack_tile = [&](long long t, int n) -> bool {
            if (!mbar_wait(&S->abort_flag, &S->empty[e], (n & 1) ^ 1, P.status, 1)) return false;
            const long long row = t * TILE + rt;
#pragma unroll
            for (int seg = 0; seg < 4; ++seg) {           // 32 codes = four 16-byte chunks of bf16
                uint4 chunk[4];
                if (row < P.n_rows) {
                    unpack_row<BITS, ASYM>(P.codes + row * P.code_row_bytes + seg * (32 * BITS / 8), chunk);
                } else {
                    chunk[0] = chunk[1] = chunk[2] = chunk[3] = make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const unsigned cg = (unsigned)(seg * 4 + c);      // chunk of the row: K block cg / 8, chunk cg % 8
                    st_shared_v4(x_row + (cg >> 3) * (TILE * 128) + (((cg & 7) ^ swz) << 4), chunk[c]);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->full[e]);
            return true;
        };

        long long t = (long long)blockIdx.x + (long long)e * gridDim.x;
        bool alive = true;
        if (t < P.n_tiles) alive = unpack_tile(t, 0);
        for (int n = 0; alive && t < P.n_tiles; t += t_step, ++n) {
            if (!mbar_wait(&S->abort_flag, &S->tfull[e], n & 1, P.status, 4)) break;
            tc_fence_after();
            const long long row = t * TILE + rt;
            const bool live = row < P.n_rows;
            float delta = 0.f, lo = 0.f;
            if (live) {
                if (ASYM) {
                    const float2 sl = __ldg(reinterpret_cast<const float2*>(P.scales) + row);
                    delta = sl.x; lo = sl.y;
                } else {
                    delta = __ldg(P.scales + row);
                }
            }
            const float sc = delta * P.norm;
            OutT* dst = reinterpret_cast<OutT*>(P.out) + row * (long long)P.d;
            // column 0 carries the offset of the stored codes and, asymmetric, 128 * lo of the zero point
            const float add0 = ASYM ? 128.f * lo * P.norm : 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                unsigned r[32];
                tmem_ld32_issue(taddr + c * 32, r);
                tmem_ld_wait(r);
                if (c == 3) {
                    // the accumulators are in registers: hand the TMEM stage back, and give the tensor cores
                    // this group's next tile before the stores of this one
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&S->tempty[e]);
                }
                if (live && c * 32 < P.d) {
                    if (c == 0) r[0] = __float_as_uint(__uint_as_float(r[0]) - P.corr);    // exact: integers
                    store_row32<OutT>(dst + c * 32, r, sc, c == 0 ? add0 : 0.f);
                }
            }
            if (t + t_step < P.n_tiles) alive = unpack_tile(t + t_step, n + 1);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <typename KernelT>
cudaError_t launch(KernelT kernel, int grid, int smem, cudaStream_t stream, bool pdl, const RowInvParams& P)
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

// The plans this path serves: the ROW family with one scale (pair) per row and whole 32-value output chunks.
bool gbs_tc_rowinv_supported(const gbs_plan* p, const float* scales)
{
    if (p->variant != GBS_VARIANT_TC_ROW || !(p->group == 0 || p->group == DP) || p->d % 32 != 0) return false;
    if (p->asym && (reinterpret_cast<uintptr_t>(scales) & 7u)) return false;       // (Delta, lo) pairs are read as one 8-byte word
    return p->smem_optin >= (int)(sizeof(Smem) + 1024);
}

int gbs_tc_rowinv_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows, void* out,
                             int out_dtype, cudaStream_t stream)
{
    RowInvParams P;
    memset(&P, 0, sizeof(P));
    P.n_rows = n_rows;
    P.n_tiles = (n_rows + TILE - 1) / TILE;
    P.d = p->d;
    P.code_row_bytes = DP * p->bits / 8;
    P.norm = p->norm;
    P.corr = 128.f * (p->asym ? 128.f : 128.f + (float)(1 << (p->bits - 1)));
    P.h_img = p->d_aimg;
    P.codes = (const unsigned char*)codes;
    P.scales = scales;
    P.out = out;
    P.status = p->d_status;
    const int smem = (int)sizeof(Smem) + 1024;
    const int grid = (int)(P.n_tiles < p->sm_count ? P.n_tiles : p->sm_count);
    const bool pdl = p->pdl != 0;
    cudaError_t e;
#define GBS_ROWINV(B, A)                                                                                     \
    (out_dtype == GBS_DTYPE_F32 ? launch(k_tc_row_inv<B, A, float>, grid, smem, stream, pdl, P)              \
                                : launch(k_tc_row_inv<B, A, __nv_bfloat16>, grid, smem, stream, pdl, P))
    if (p->asym) e = p->bits == 3 ? GBS_ROWINV(3, true) : GBS_ROWINV(4, true);
    else e = p->bits == 3 ? GBS_ROWINV(3, false) : GBS_ROWINV(4, false);
#undef GBS_ROWINV
    return (int)e;
}
