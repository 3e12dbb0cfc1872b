// gbs_quantized_matmul: the consumer on the other side of the path (Section 4.2, Eq. (2); Section 2.3.1).
//
// The online path leaves, per token, b-bit codes q_x and one scale Delta_x of the rotated, zero-padded activation
// H x_pad / sqrt(d'); the weights W (one row per output channel) go through the same rotation and quantizer once,
// offline (gbs_weight_rotate_quantize), leaving codes q_w and one scale Delta_w per output channel.  Because the
// rotation is orthogonal and the padding adds zeros, (H x_pad)^T (H w_pad) / d' = x^T w (Eq. (2)), so the layer's
// output is, up to quantization error,
//
//        out[t][o] = Delta_x[t] * Delta_w[o] * sum_j q_x[t][j] * q_w[o][j],
//
// an INTEGER contraction over the d' codes followed by one multiplication per output.  The rotated activation never
// exists in memory as floats: this kernel reads the packed codes of both operands.
//
//   * One CTA per 128 x 256 tile of the output (tokens x output channels); the contraction runs over blocks of 128
//     codes through a ring of shared-memory stages.
//   * Sixteen warps unpack: each thread fetches the packed 3- or 4-bit codes of its slice of the next block straight
//     from global memory (whole lines: 256 codes of a row per eight threads, two such super-blocks ahead, held in
//     registers), turns them into int8 with byte-wise logic (a field moved to the top bits of its byte IS the int8
//     q * 2^(8-b); the epilogue removes the power of two), and writes 16-byte chunks into the K-major,
//     128-byte-swizzled operand tiles the tensor cores read.  Both operands use the same order of the codes inside a chunk (even
//     fields first, then odd), which a dot product does not see.
//   * One thread issues tcgen05.mma kind::i8 (int8 x int8 -> int32, 128 x 256 x 32 per instruction), accumulators
//     in TMEM; tcgen05.commit hands the stage back to the unpackers.
//   * After the last block the sixteen warps read the int32 sums from TMEM (exact), convert (a multiple of
//     2^(16-bx-bw) whose quotient is below 2^24: exact in fp32), scale by Delta_x[t] * Delta_w[o], store fp32 or bf16.
// Every wait is bounded; an expired wait records a code in the activation plan's status word.
#include <math.h>
#include <string.h>

#include <mutex>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int TM = 128;                 // tokens per tile (MMA M)
constexpr int TN = 256;                 // output channels per tile (MMA N)
constexpr int KB = 128;                 // codes per stage and row: one 128-byte swizzled line of int8
constexpr int STAGES = 4;
constexpr int A_STAGE = TM * KB;        // 16 KB
constexpr int B_STAGE = TN * KB;        // 32 KB
constexpr int UNPACK_WARPS = 16;
constexpr int THREADS = 32 * (1 + UNPACK_WARPS);
constexpr int TMEM_COLS = 256;

struct __align__(1024) Smem {
    unsigned char a[STAGES][A_STAGE];
    unsigned char b[STAGES][B_STAGE];
    float dw[TN];                       // Delta_w of the tile's output channels
    unsigned long long full[STAGES], empty[STAGES], tfull;
    unsigned tmem_base;
    volatile int abort_flag;
};

struct QgemmParams {
    long long n_tok, n_out;
    int kblocks;                        // d' / 128
    int rbx, rbw;                       // bytes per row of packed codes
    const unsigned char* cx;
    const unsigned char* cw;
    const float* sx;
    const float* sw;
    void* out;
    long long out_stride;               // elements
    int vec;                            // rows of `out` start on 16-byte boundaries: vector stores allowed
    int* status;
};

// Instruction descriptor, kind::i8: int32 accumulate, signed 8-bit A and B, both K-major, M x N.
__host__ __device__ constexpr unsigned instr_desc_i8(int M, int N)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(N >> 3) << 17) | ((unsigned)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_i8(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned idesc,
                                        unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void st_shared_v4(unsigned addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Eight two's-complement fields (24 or 32 bits) -> two words of four int8 each: the even fields, the odd fields.
// No sign extension is computed: a field moved to the TOP bits of its byte is the int8 value q * 2^(8 - BITS) (the
// field's sign bit becomes the byte's), products are then scaled by a power of two that the epilogue's scale factor
// takes out exactly, and the int32 sums stay far below 2^31 (49 * d' * 2^10 at most).  Four-bit fields already sit in
// nibbles: one mask for the odd ones, a shift and a mask for the even ones.  Three-bit fields are first spread to one
// per nibble by three mask-and-shift steps.
template <int BITS>
__device__ __forceinline__ void fields_to_int8(unsigned f, unsigned& even, unsigned& odd)
{
    if (BITS == 4) {
        odd = f & 0xf0f0f0f0u;
        even = (f << 4) & 0xf0f0f0f0u;
    } else {
        f = (f & 0x00000fffu) | ((f & 0x00fff000u) << 4);       // 12 bits per half-word
        f = (f & 0x003f003fu) | ((f & 0x0fc00fc0u) << 2);       // 6 bits per byte
        f = (f & 0x07070707u) | ((f & 0x38383838u) << 1);       // 3 bits per nibble (bit 3 of every nibble clear)
        odd = (f << 1) & 0xe0e0e0e0u;
        even = (f << 5) & 0xe0e0e0e0u;
    }
}

// NF fields of a row slice, from its packed words (3 words per 4 fields at 3 bits, 1 word per field at 4 bits).
template <int BITS, int NF>
__device__ __forceinline__ void load_raw(const unsigned char* src, bool live, unsigned raw[NF])
{
    constexpr int NW = NF * BITS / 4;
#pragma unroll
    for (int i = 0; i < NF; ++i) raw[i] = 0u;
    if (!live) return;
    if (BITS == 4 && NF % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NF / 4; ++i) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(src) + i);
            raw[4 * i] = v.x; raw[4 * i + 1] = v.y; raw[4 * i + 2] = v.z; raw[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < NW; ++i) raw[i] = __ldg(reinterpret_cast<const unsigned*>(src) + i);
    }
}

// raw words -> NF/2 chunks of 16 int8 (fields 2c and 2c+1: even, odd, even, odd), written to the swizzled row.
template <int BITS, int NF>
__device__ __forceinline__ void unpack_store(const unsigned raw[NF], unsigned row_addr, int chunk0, int swz)
{
    unsigned f[NF];
    if (BITS == 4) {
#pragma unroll
        for (int i = 0; i < NF; ++i) f[i] = raw[i];
    } else {
#pragma unroll
        for (int g = 0; g < NF / 4; ++g) {
            const unsigned w0 = raw[3 * g], w1 = raw[3 * g + 1], w2 = raw[3 * g + 2];
            f[4 * g] = w0;                                   // bits above 24 are dropped by the masks below
            f[4 * g + 1] = __funnelshift_r(w0, w1, 24);
            f[4 * g + 2] = __funnelshift_r(w1, w2, 16);
            f[4 * g + 3] = w2 >> 8;
        }
    }
#pragma unroll
    for (int c = 0; c < NF / 2; ++c) {
        uint4 v;
        fields_to_int8<BITS>(f[2 * c], v.x, v.y);
        fields_to_int8<BITS>(f[2 * c + 1], v.z, v.w);
        st_shared_v4(row_addr + (unsigned)(((chunk0 + c) ^ swz) << 4), v);
    }
}

template <int XBITS, int WBITS, typename OutT>
__global__ void __launch_bounds__(THREADS, 1) k_tc_qgemm(const __grid_constant__ QgemmParams P)
{
    extern __shared__ unsigned char smem_raw[];
    Smem* S = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long tok0 = (long long)blockIdx.y * TM;
    const long long out0 = (long long)blockIdx.x * TN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&S->full[s], UNPACK_WARPS);
            mbar_init(&S->empty[s], 1);
        }
        mbar_init(&S->tfull, 1);
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(&S->tmem_base, TMEM_COLS);
    if (threadIdx.x >= 32 && threadIdx.x < 32 + TN) {
        const long long o = out0 + (threadIdx.x - 32);
        S->dw[threadIdx.x - 32] = o < P.n_out ? __ldg(P.sw + o) : 0.f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = S->tmem_base;

    if (warp == 0) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr unsigned IDESC = instr_desc_i8(TM, TN);
            for (int kb = 0; kb < P.kblocks; ++kb) {
                const int s = kb % STAGES;
                if (!mbar_wait(&S->abort_flag, &S->full[s], (kb / STAGES) & 1, P.status, 2)) break;
                tc_fence_after();
                // one stage = one 128-byte line per row; an instruction takes 32 codes = 32 bytes of it
                const unsigned long long ad = smem_desc(smem_u32(S->a[s]), 16, 1024, 2);
                const unsigned long long bd = smem_desc(smem_u32(S->b[s]), 16, 1024, 2);
#pragma unroll
                for (int ks = 0; ks < KB / 32; ++ks)
                    umma_i8(tmem_base, ad + (unsigned long long)(2 * ks), bd + (unsigned long long)(2 * ks), IDESC,
                            (kb | ks) != 0 ? 1u : 0u);
                umma_commit(&S->empty[s]);
            }
            umma_commit(&S->tfull);
        }
    } else {
        // ------------------------------ unpack, then epilogue ------------------------------
        const int ut = threadIdx.x - 32;              // 0 .. 511
        // Work is cut into SUPER-BLOCKS of 256 codes per row (two stages) so that the global loads are whole lines: an
        // item is 32 codes (four fields, 16 or 12 bytes) of one row; the eight threads ut & 7 = 0..7 take the eight
        // items of a row's 256 codes (128 or 96 contiguous bytes), so a warp's load instruction covers four rows'
        // full lines.  (Loading per 128-code block, with two or four threads per row, asked the L1 for 32 sectors per
        // request and kept it 89 % busy: that, not the arithmetic or shared memory, bound the kernel.)
        // A thread's item position seg is fixed: stage half h = seg >> 2, chunks 2 (seg & 3) and + 1 of the row; its
        // rows are r0 + 64 i: two of the activation tile, four of the weight tile.
        // Lane bits, low to high: part (2), row bit 0, half, row bit 1.  A 16-byte shared-memory store is served eight
        // lanes at a time: eight consecutive lanes then hold two rows x four parts of ONE stage, whose swizzled chunk
        // positions are all different (both halves of a row would collide: same banks, other stage).
        const int part = lane & 3, half = (lane >> 3) & 1, seg = 4 * half + part;
        const int r0 = (ut >> 5) * 4 + ((lane >> 4) & 1) * 2 + ((lane >> 2) & 1);
        constexpr int NA = TM / 64, NB = TN / 64;
        constexpr int XSB = 256 * XBITS / 8, WSB = 256 * WBITS / 8;        // bytes of a super-block per row
        const unsigned char* ax = P.cx + (tok0 + r0) * (long long)P.rbx + seg * (32 * XBITS / 8);
        const unsigned char* bw = P.cw + (out0 + r0) * (long long)P.rbw + seg * (32 * WBITS / 8);
        bool a_live[NA], b_live[NB];
#pragma unroll
        for (int i = 0; i < NA; ++i) a_live[i] = tok0 + r0 + 64 * i < P.n_tok;
#pragma unroll
        for (int i = 0; i < NB; ++i) b_live[i] = out0 + r0 + 64 * i < P.n_out;
        const int n_sb = (P.kblocks + 1) >> 1;
        // the packed codes of the next PF super-blocks are in flight (in registers) while one is unpacked
        constexpr int PF = 2;
        unsigned ra[PF][NA][4], rb[PF][NB][4];
        auto load_sb = [&](int sb, unsigned (&qa)[NA][4], unsigned (&qb)[NB][4]) {
            const bool in = 2 * sb + half < P.kblocks;                  // an odd number of blocks: no second half
#pragma unroll
            for (int i = 0; i < NA; ++i)
                load_raw<XBITS, 4>(ax + (long long)sb * XSB + (long long)(64 * i) * P.rbx, in && a_live[i], qa[i]);
#pragma unroll
            for (int i = 0; i < NB; ++i)
                load_raw<WBITS, 4>(bw + (long long)sb * WSB + (long long)(64 * i) * P.rbw, in && b_live[i], qb[i]);
        };
#pragma unroll
        for (int j = 0; j < PF; ++j) load_sb(j, ra[j], rb[j]);
        bool alive = true;
        for (int sb0 = 0; alive && sb0 < n_sb; sb0 += PF) {
#pragma unroll
            for (int j = 0; j < PF; ++j) {
                const int sb = sb0 + j;
                if (sb >= n_sb) break;
                const int kb = 2 * sb + half;                           // the block this thread's items belong to
                const bool mine = kb < P.kblocks;
                const int s = kb % STAGES;
                bool ok = true;
                if (mine) ok = mbar_wait(&S->abort_flag, &S->empty[s], ((kb / STAGES) & 1) ^ 1, P.status, 1);
                if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }       // the warp leaves as one
                if (mine) {
#pragma unroll
                    for (int i = 0; i < NA; ++i) {
                        const int r = r0 + 64 * i;
                        unpack_store<XBITS, 4>(ra[j][i], smem_u32(S->a[s]) + (unsigned)r * 128u, 2 * part, r & 7);
                    }
#pragma unroll
                    for (int i = 0; i < NB; ++i) {
                        const int r = r0 + 64 * i;
                        unpack_store<WBITS, 4>(rb[j][i], smem_u32(S->b[s]) + (unsigned)r * 128u, 2 * part, r & 7);
                    }
                }
                if (sb + PF < n_sb) load_sb(sb + PF, ra[j], rb[j]);
                // make the generic-proxy writes visible to the tensor cores' (async proxy) reads, then signal: a warp
                // holds items of both halves, so it reports to both stages of the super-block
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&S->full[(2 * sb) % STAGES]);
                    if (2 * sb + 1 < P.kblocks) mbar_arrive(&S->full[(2 * sb + 1) % STAGES]);
                }
            }
        }
        if (alive && mbar_wait(&S->abort_flag, &S->tfull, 0, P.status, 4)) {
            tc_fence_after();
            const int q = warp & 3;                    // TMEM lane quadrant this warp may access
            const int cb = (warp - 1) >> 2;            // 64-column block of the tile
            const long long tok = tok0 + q * 32 + lane;
            // the int8 operands were q * 2^(8 - bits): take the two powers of two out again (exact)
            const float dx = tok < P.n_tok ? __ldg(P.sx + tok) * (1.f / (float)(1 << (16 - XBITS - WBITS))) : 0.f;
            OutT* orow = reinterpret_cast<OutT*>(P.out) + tok * P.out_stride + out0;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const int c0 = cb * 64 + h * 32;
                unsigned r[32];
                tmem_ld32_issue(tmem_base + ((unsigned)(q * 32) << 16) + (unsigned)c0, r);
                tmem_ld_wait(r);
                if (tok < P.n_tok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        float v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) v[e] = (float)(int)r[i + e] * (dx * S->dw[c0 + i + e]);
                        const long long o = out0 + c0 + i;
                        if (P.vec && o + 3 < P.n_out) {
                            if (sizeof(OutT) == 4) {
                                *reinterpret_cast<float4*>(orow + c0 + i) = make_float4(v[0], v[1], v[2], v[3]);
                            } else {
                                __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
                                *reinterpret_cast<uint2*>(orow + c0 + i) =
                                    make_uint2(*reinterpret_cast<unsigned*>(&p0), *reinterpret_cast<unsigned*>(&p1));
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (o + e < P.n_out) {
                                    if (sizeof(OutT) == 4) reinterpret_cast<float*>(orow)[c0 + i + e] = v[e];
                                    else reinterpret_cast<__nv_bfloat16*>(orow)[c0 + i + e] = __float2bfloat16_rn(v[e]);
                                }
                        }
                    }
                }
            }
        }
    }

    // ---- teardown: every role has left its loop (normally or after a wait expired); TMEM is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

typedef void (*QgemmKernel)(const QgemmParams);
QgemmKernel pick(int xbits, int wbits, int out_dtype)
{
    static const QgemmKernel table[2][2][2] = {
        {{k_tc_qgemm<3, 3, float>, k_tc_qgemm<3, 3, __nv_bfloat16>}, {k_tc_qgemm<3, 4, float>, k_tc_qgemm<3, 4, __nv_bfloat16>}},
        {{k_tc_qgemm<4, 3, float>, k_tc_qgemm<4, 3, __nv_bfloat16>}, {k_tc_qgemm<4, 4, float>, k_tc_qgemm<4, 4, __nv_bfloat16>}}};
    return table[xbits - 3][wbits - 3][out_dtype == GBS_DTYPE_F32 ? 0 : 1];
}

}  // namespace

extern "C" int gbs_quantized_matmul(const gbs_plan_t* px, const void* codes_x, const float* scales_x, int64_t n_tokens,
                                    const gbs_plan_t* pw, const void* codes_w, const float* scales_w, int64_t n_out,
                                    void* out, int out_dtype, int64_t out_row_stride, void* cuda_stream)
{
    if (!px || !pw) return GBS_ERR_INVALID_ARG;
    if (out_dtype != GBS_DTYPE_F32 && out_dtype != GBS_DTYPE_BF16) return GBS_ERR_INVALID_ARG;
    if (n_tokens < 0 || n_out < 0 || out_row_stride < n_out) return GBS_ERR_INVALID_ARG;
    if (px->d_pad != pw->d_pad || px->d != pw->d || px->m != pw->m) return GBS_ERR_INVALID_ARG;   // one rotation for both sides
    if (px->device != pw->device) return GBS_ERR_INVALID_ARG;
    // one symmetric scale per token and per output channel, so that the scales leave the contraction
    if (px->group != 0 || pw->group != 0 || px->asym || pw->asym) return GBS_ERR_UNSUPPORTED;
    if (px->d_pad % KB != 0) return GBS_ERR_UNSUPPORTED;
    if (px->smem_optin < (int)(sizeof(Smem) + 1024)) return GBS_ERR_UNSUPPORTED;
    if (n_tokens == 0 || n_out == 0) return GBS_OK;
    if (!codes_x || !scales_x || !codes_w || !scales_w || !out) return GBS_ERR_INVALID_ARG;
    const int esz = out_dtype == GBS_DTYPE_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(codes_x) & 15u) || (reinterpret_cast<uintptr_t>(codes_w) & 15u) ||
        (reinterpret_cast<uintptr_t>(out) & (uintptr_t)(esz - 1)) ||
        (reinterpret_cast<uintptr_t>(scales_x) & 3u) || (reinterpret_cast<uintptr_t>(scales_w) & 3u))
        return GBS_ERR_ALIGNMENT;
    if ((n_out + TN - 1) / TN > 0x7fffffff || (n_tokens + TM - 1) / TM > 65535) return GBS_ERR_INVALID_ARG;
    gbs_device_guard guard;
    if (guard.enter(px->device) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }

    QgemmParams P;
    memset(&P, 0, sizeof(P));
    P.n_tok = n_tokens;
    P.n_out = n_out;
    P.kblocks = px->d_pad / KB;
    P.rbx = px->d_pad * px->bits / 8;
    P.rbw = pw->d_pad * pw->bits / 8;
    P.cx = (const unsigned char*)codes_x;
    P.cw = (const unsigned char*)codes_w;
    P.sx = scales_x;
    P.sw = scales_w;
    P.out = out;
    P.out_stride = out_row_stride;
    P.vec = ((reinterpret_cast<uintptr_t>(out) & 15u) == 0 && ((out_row_stride * esz) & 15) == 0) ? 1 : 0;
    P.status = px->d_status;
    const int smem = (int)sizeof(Smem) + 1024;
    QgemmKernel kernel = pick(px->bits, pw->bits, out_dtype);
    {
        // opt in to the large dynamic shared memory once per device and instantiation (not a stream operation)
        static std::mutex mu;
        static bool done[64][8] = {{false}};
        const int ki = (px->bits - 3) * 4 + (pw->bits - 3) * 2 + (out_dtype == GBS_DTYPE_F32 ? 0 : 1);
        std::lock_guard<std::mutex> lock(mu);
        if (!(px->device >= 0 && px->device < 64 && done[px->device][ki])) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
                cudaGetLastError();
                return GBS_ERR_CUDA;
            }
            if (px->device >= 0 && px->device < 64) done[px->device][ki] = true;
        }
    }
    const dim3 grid((unsigned)((n_out + TN - 1) / TN), (unsigned)((n_tokens + TM - 1) / TM));
    kernel<<<grid, THREADS, smem, static_cast<cudaStream_t>(cuda_stream)>>>(P);
    if (cudaGetLastError() != cudaSuccess) return GBS_ERR_CUDA;
    return GBS_OK;
}

// Weight side of Eq. (2): every row of W (one output channel, width d) is zero-padded, rotated and quantized like a
// token row -- round to nearest, one scale per output channel when the plan has group 0.
extern "C" int gbs_weight_rotate_quantize(const gbs_plan_t* plan, const void* w, int w_dtype, int64_t n_out,
                                          int64_t w_row_stride, void* codes, float* scales, void* cuda_stream)
{
    if (!plan) return GBS_ERR_INVALID_ARG;
    if (plan->asym) return GBS_ERR_UNSUPPORTED;
    return gbs_rotate_quantize(plan, w, w_dtype, n_out, w_row_stride, codes, scales, nullptr, cuda_stream);
}
