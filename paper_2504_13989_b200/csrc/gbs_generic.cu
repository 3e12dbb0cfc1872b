// Generic kernel family: works for every supported (m, k), fp32 or bf16 rows, 3 or 4 bits, per-token
// or per-group scales.  A team of up to 256 threads owns one token row; the padded row lives in
// shared memory as fp32.
//
//   S0/S1  load the row, append zeros up to d'                     (Section 4.2, Eq. (2))
//   S3     Sylvester butterflies inside each block of 2^k          (Eq. (1))
//   S2     m x m Paley mix across the m blocks                     (Algorithm 2)
//   S4-S8  1/sqrt(d'), absmax, Delta, round/clip, pack, store      (Appendix A; Sections 2.1, 3.1)
//
// The two factors of H_m (x) H_{2^k} act on different index digits and commute; the butterflies
// run first because the first three stages are done in registers straight from the global load.
//
// The specialised tensor-core families reuse none of this file; it is the fallback and the path for
// fp32 inputs.
#include <cuda_bf16.h>

#include <stdlib.h>

#include "gbs_internal.h"

namespace {

constexpr int NT = 256;             // threads per block
constexpr unsigned FULL = 0xffffffffu;

struct GenericParams {
    int d, d_pad, k, m, n2;          // n2 = 2^k
    int group, G, spr;               // G = group ? group : d_pad ; spr = scales per row
    int asym;                        // dequantize: asymmetric plan (unsigned codes, (Delta, lo) pairs)
    int levels;
    float norm, c_scale, c_inv;
    int tt_log2, rows_per_cta;       // team = 1 << tt_log2 threads per row
    int chunks;                      // d_pad / 8
    int red_mode, seg_lanes;         // absmax reduction strategy (see reduce_group_max)
    int row_floats;                  // d_pad + d_pad/32 (one pad word per 32)
    int row_bytes;                   // d_pad * bits / 8
    int stage_bytes;                 // row_bytes rounded up to 16
    int n_pass;
    int pass_s[8], pass_r[8];        // butterfly passes over bits [s, s+r) in shared memory
    long long n_rows, stride;
    const float* hm;                 // device H_m (forward) or H_m^T (inverse), m*m floats
};

__device__ __forceinline__ int pidx(int i) { return i + (i >> 5); }

// ---- global loads of one chunk of 8 consecutive elements, zero beyond d ---------------------------
__device__ __forceinline__ void load_chunk8(const float* xrow, int idx, int d, float v[8])
{
    if (idx + 8 <= d) {
        float4 a = __ldg(reinterpret_cast<const float4*>(xrow + idx));
        float4 b = __ldg(reinterpret_cast<const float4*>(xrow + idx + 4));
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = (idx + e < d) ? __ldg(xrow + idx + e) : 0.f;
    }
}

__device__ __forceinline__ void load_chunk8(const __nv_bfloat16* xrow, int idx, int d, float v[8])
{
    if (idx + 8 <= d) {
        uint4 r = __ldg(reinterpret_cast<const uint4*>(xrow + idx));
        unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[2 * e] = __uint_as_float(w[e] << 16);
            v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
    } else {
        const unsigned short* xs = reinterpret_cast<const unsigned short*>(xrow);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            v[e] = (idx + e < d) ? __uint_as_float(((unsigned)__ldg(xs + idx + e)) << 16) : 0.f;
    }
}

template <int N>
__device__ __forceinline__ void butterflies(float v[N])
{
#pragma unroll
    for (int h = 1; h < N; h <<= 1)
#pragma unroll
        for (int i = 0; i < N; ++i)
            if ((i & h) == 0) {
                float a = v[i], b = v[i + h];
                v[i] = a + b;
                v[i + h] = a - b;
            }
}

// One butterfly pass over index bits [s, s+R) of a row held in shared memory.
template <int R>
__device__ __forceinline__ void fwht_pass(float* row, int s, int d_pad, int j, int tt)
{
    const int items = d_pad >> R;
    for (int w = j; w < items; w += tt) {
        int low = w & ((1 << s) - 1);
        int base = ((w >> s) << (s + R)) | low;
        float v[1 << R];
#pragma unroll
        for (int t = 0; t < (1 << R); ++t) v[t] = row[pidx(base + (t << s))];
        butterflies<(1 << R)>(v);
#pragma unroll
        for (int t = 0; t < (1 << R); ++t) row[pidx(base + (t << s))] = v[t];
    }
}

// U = H_m * X_mat: thread-owned columns, signs (as +-1.0f) read from shared memory.
template <int M>
__device__ __forceinline__ void paley_mix(float* row, const float* hm_s, int n2, int j, int tt)
{
    for (int c = j; c < n2; c += tt) {
        float u[M];
#pragma unroll
        for (int a = 0; a < M; ++a) u[a] = row[pidx(a * n2 + c)];
#pragma unroll 4
        for (int a = 0; a < M; ++a) {
            const float4* hr = reinterpret_cast<const float4*>(hm_s + a * M);
            float acc = 0.f;
#pragma unroll
            for (int q = 0; q < M / 4; ++q) {
                float4 h = hr[q];
                acc = fmaf(h.x, u[4 * q], acc);
                acc = fmaf(h.y, u[4 * q + 1], acc);
                acc = fmaf(h.z, u[4 * q + 2], acc);
                acc = fmaf(h.w, u[4 * q + 3], acc);
            }
            row[pidx(a * n2 + c)] = acc;
        }
    }
}

// WIDE selects the orders above 28: their register-held columns (up to 108 values per thread) would
// double the register count of every kernel here, so they get instantiations of their own.
template <bool WIDE>
__device__ __forceinline__ void run_passes_and_mix(const GenericParams& P, float* row, const float* hm_s,
                                                   int j, int tt)
{
    for (int ps = 0; ps < P.n_pass; ++ps) {
        __syncthreads();
        const int s = P.pass_s[ps];
        switch (P.pass_r[ps]) {
            case 1: fwht_pass<1>(row, s, P.d_pad, j, tt); break;
            case 2: fwht_pass<2>(row, s, P.d_pad, j, tt); break;
            case 3: fwht_pass<3>(row, s, P.d_pad, j, tt); break;
            default: fwht_pass<4>(row, s, P.d_pad, j, tt); break;
        }
    }
    if (P.m > 1) {
        __syncthreads();
        if constexpr (!WIDE) {
            switch (P.m) {
                case 12: paley_mix<12>(row, hm_s, P.n2, j, tt); break;
                case 20: paley_mix<20>(row, hm_s, P.n2, j, tt); break;
                case 24: paley_mix<24>(row, hm_s, P.n2, j, tt); break;
                default: paley_mix<28>(row, hm_s, P.n2, j, tt); break;
            }
        } else switch (P.m) {
            case 44: paley_mix<44>(row, hm_s, P.n2, j, tt); break;
            case 48: paley_mix<48>(row, hm_s, P.n2, j, tt); break;
            case 60: paley_mix<60>(row, hm_s, P.n2, j, tt); break;
            case 68: paley_mix<68>(row, hm_s, P.n2, j, tt); break;
            case 72: paley_mix<72>(row, hm_s, P.n2, j, tt); break;
            case 80: paley_mix<80>(row, hm_s, P.n2, j, tt); break;
            case 84: paley_mix<84>(row, hm_s, P.n2, j, tt); break;
            case 104: paley_mix<104>(row, hm_s, P.n2, j, tt); break;
            default: paley_mix<108>(row, hm_s, P.n2, j, tt); break;
        }
    }
    __syncthreads();
}

// Load + pad + first three butterfly stages in registers -> shared memory, then the rest.
template <typename InT, bool WIDE>
__device__ __forceinline__ void rotate_row_to_smem(const GenericParams& P, const InT* x, long long row,
                                                   bool active, float* rowbuf, const float* hm_s, int j,
                                                   int tt)
{
    if (active) {
        const InT* xrow = x + row * P.stride;
        for (int ch = j; ch < P.chunks; ch += tt) {
            float v[8];
            load_chunk8(xrow, ch * 8, P.d, v);
            butterflies<8>(v);
            const int p = ch * 8 + (ch >> 2);
#pragma unroll
            for (int e = 0; e < 8; ++e) rowbuf[p + e] = v[e];
        }
    }
    run_passes_and_mix<WIDE>(P, rowbuf, hm_s, j, tt);
}

// max|.| of a group of G consecutive values, each thread holding the max of its 8-value chunk.
//   mode 1: G is a power of two <= 256: xor-shuffle over the G/8 adjacent lanes, leader stores
//   mode 2: G is a multiple of 256: the whole warp shares one group: warp max, one atomic
//   mode 3: anything else: one shared-memory atomic per chunk
__device__ __forceinline__ void reduce_group_max(const GenericParams& P, float amax, int ch, bool valid,
                                                 unsigned* gmax)
{
    const int lane = threadIdx.x & 31;
    if (P.red_mode == 1) {
        for (int o = P.seg_lanes >> 1; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, o));
        if (valid && (lane & (P.seg_lanes - 1)) == 0) gmax[(ch * 8) / P.G] = __float_as_uint(amax);
    } else if (P.red_mode == 2) {
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, o));
        if (valid && lane == 0) atomicMax(&gmax[(ch * 8) / P.G], __float_as_uint(amax));
    } else {
        if (valid) atomicMax(&gmax[(ch * 8) / P.G], __float_as_uint(amax));
    }
}

__device__ __forceinline__ void read_chunk_smem(const float* rowbuf, int ch, float v[8])
{
    const int p = ch * 8 + (ch >> 2);
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = rowbuf[p + e];
}

// Team-wide absmax of the rotated row into gmax[0 .. spr).  Ends with a block barrier.
__device__ __forceinline__ void row_group_max(const GenericParams& P, const float* rowbuf, unsigned* gmax,
                                              bool active, int j, int tt)
{
    const int iters = (P.chunks + tt - 1) / tt;
    for (int it = 0; it < iters; ++it) {
        const int ch = j + it * tt;
        const bool valid = active && ch < P.chunks;
        float amax = 0.f;
        if (valid) {
            float v[8];
            read_chunk_smem(rowbuf, ch, v);
#pragma unroll
            for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(v[e]));
        }
        reduce_group_max(P, amax, valid ? ch : 0, valid, gmax);
    }
    __syncthreads();
}

struct SmemLayout {
    float* rowbuf;      // [R][row_floats]
    unsigned* gmax;     // [R][spr]
    float* hm_s;        // [m*m]
    unsigned char* tail;  // kernel-specific
};

__device__ __forceinline__ SmemLayout carve(const GenericParams& P, unsigned char* smem)
{
    SmemLayout L;
    L.rowbuf = reinterpret_cast<float*>(smem);
    size_t off = sizeof(float) * (size_t)P.rows_per_cta * P.row_floats;
    L.gmax = reinterpret_cast<unsigned*>(smem + off);
    off += sizeof(unsigned) * (size_t)P.rows_per_cta * P.spr;
    off = (off + 15) & ~(size_t)15;
    L.hm_s = reinterpret_cast<float*>(smem + off);
    off += sizeof(float) * (size_t)((P.m > 1) ? P.m * P.m : 0);
    off = (off + 15) & ~(size_t)15;
    L.tail = smem + off;
    return L;
}

__device__ __forceinline__ void stage_hm(const GenericParams& P, float* hm_s)
{
    if (P.m > 1)
        for (int i = threadIdx.x; i < P.m * P.m; i += NT) hm_s[i] = P.hm[i];
}

__device__ __forceinline__ void clear_gmax(const GenericParams& P, unsigned* gmax)
{
    for (int i = threadIdx.x; i < P.rows_per_cta * P.spr; i += NT) gmax[i] = 0u;
}

// ======================================================================================
// rotate + quantize + pack
// ======================================================================================
template <typename InT, int BITS, bool WIDE>
__global__ void __launch_bounds__(NT) k_rotate_quantize(GenericParams P, const InT* __restrict__ x,
                                                        unsigned char* __restrict__ codes,
                                                        float* __restrict__ scales, float* __restrict__ y_opt)
{
    extern __shared__ __align__(16) unsigned char smem[];
    SmemLayout L = carve(P, smem);
    unsigned char* stage_all = L.tail;
    stage_hm(P, L.hm_s);

    const int tt = 1 << P.tt_log2;
    const int team = threadIdx.x >> P.tt_log2;
    const int j = threadIdx.x & (tt - 1);
    float* rowbuf = L.rowbuf + (size_t)team * P.row_floats;
    unsigned* gmax = L.gmax + (size_t)team * P.spr;
    unsigned char* stage = stage_all + (size_t)team * P.stage_bytes;
    const float fD = (float)P.levels;

    for (long long row0 = (long long)blockIdx.x * P.rows_per_cta; row0 < P.n_rows;
         row0 += (long long)gridDim.x * P.rows_per_cta) {
        const long long row = row0 + team;
        const bool active = row < P.n_rows;
        clear_gmax(P, L.gmax);
        rotate_row_to_smem<InT, WIDE>(P, x, row, active, rowbuf, L.hm_s, j, tt);
        row_group_max(P, rowbuf, gmax, active, j, tt);

        if (active) {
            for (int ch = j; ch < P.chunks; ch += tt) {
                float v[8];
                read_chunk_smem(rowbuf, ch, v);
                const int g = (ch * 8) / P.G;
                const float M = __uint_as_float(gmax[g]);
                const float delta = P.c_scale * M;
                const float inv = (M > 0.f) ? (P.c_inv / M) : 0.f;
                if ((ch * 8) % P.G == 0) scales[row * P.spr + g] = delta;
                unsigned word = 0;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float t = fminf(fmaxf(v[e] * inv, -fD), fD);
                    int q = __float2int_rn(t);
                    word |= ((unsigned)q & ((1u << BITS) - 1u)) << (BITS * e);
                }
                if (BITS == 4) {
                    *reinterpret_cast<unsigned*>(stage + ch * 4) = word;
                } else {
                    stage[ch * 3] = (unsigned char)(word & 0xff);
                    stage[ch * 3 + 1] = (unsigned char)((word >> 8) & 0xff);
                    stage[ch * 3 + 2] = (unsigned char)((word >> 16) & 0xff);
                }
                if (y_opt) {
                    float4* yo = reinterpret_cast<float4*>(y_opt + row * P.d_pad + ch * 8);
                    yo[0] = make_float4(v[0] * P.norm, v[1] * P.norm, v[2] * P.norm, v[3] * P.norm);
                    yo[1] = make_float4(v[4] * P.norm, v[5] * P.norm, v[6] * P.norm, v[7] * P.norm);
                }
            }
        }
        __syncthreads();
        if (active) {
            unsigned char* dst = codes + row * P.row_bytes;
            if ((P.row_bytes & 15) == 0) {
                const uint4* s4 = reinterpret_cast<const uint4*>(stage);
                uint4* d4 = reinterpret_cast<uint4*>(dst);
                for (int i = j; i < (P.row_bytes >> 4); i += tt) d4[i] = s4[i];
            } else {
                for (int i = j; i < P.row_bytes; i += tt) dst[i] = stage[i];
            }
        }
        __syncthreads();
    }
}

// ======================================================================================
// clip-ratio scoring
// ======================================================================================
constexpr int KT = 8;   // candidates scored per sweep over the row

struct ClipConsts {
    float c_scale[GBS_MAX_CANDIDATES];   // alpha_k / (D sqrt(d'))
    float c_inv[GBS_MAX_CANDIDATES];     // D / alpha_k
};

template <typename InT, bool WIDE>
__global__ void __launch_bounds__(NT) k_clip_error(GenericParams P, ClipConsts C, int K,
                                                   const InT* __restrict__ x, double* __restrict__ err_sum,
                                                   float* __restrict__ err_rows)
{
    extern __shared__ __align__(16) unsigned char smem[];
    SmemLayout L = carve(P, smem);
    // tail: double cta_sum[K]; float row_err[R][K]
    double* cta_sum = reinterpret_cast<double*>(L.tail);
    float* row_err_all = reinterpret_cast<float*>(L.tail + sizeof(double) * GBS_MAX_CANDIDATES);
    stage_hm(P, L.hm_s);
    for (int i = threadIdx.x; i < K; i += NT) cta_sum[i] = 0.0;

    const int tt = 1 << P.tt_log2;
    const int team = threadIdx.x >> P.tt_log2;
    const int j = threadIdx.x & (tt - 1);
    const int lane = threadIdx.x & 31;
    float* rowbuf = L.rowbuf + (size_t)team * P.row_floats;
    unsigned* gmax = L.gmax + (size_t)team * P.spr;
    float* row_err = row_err_all + (size_t)team * GBS_MAX_CANDIDATES;
    const float fD = (float)P.levels;
    const float MAGIC = 12582912.f;   // 1.5 * 2^23: adding and subtracting rounds to nearest-even integer

    for (long long row0 = (long long)blockIdx.x * P.rows_per_cta; row0 < P.n_rows;
         row0 += (long long)gridDim.x * P.rows_per_cta) {
        const long long row = row0 + team;
        const bool active = row < P.n_rows;
        clear_gmax(P, L.gmax);
        for (int i = threadIdx.x; i < P.rows_per_cta * GBS_MAX_CANDIDATES; i += NT) row_err_all[i] = 0.f;
        rotate_row_to_smem<InT, WIDE>(P, x, row, active, rowbuf, L.hm_s, j, tt);
        row_group_max(P, rowbuf, gmax, active, j, tt);

        for (int k0 = 0; k0 < K; k0 += KT) {
            float acc[KT];
#pragma unroll
            for (int kk = 0; kk < KT; ++kk) acc[kk] = 0.f;
            if (active) {
                for (int ch = j; ch < P.chunks; ch += tt) {
                    float v[8];
                    read_chunk_smem(rowbuf, ch, v);
                    const float M = __uint_as_float(gmax[(ch * 8) / P.G]);
                    // y / Delta_k = Y * (D / alpha_k) / max|Y| and y = Y * norm, so on y the factor is
                    // (D / alpha_k) * sM with sM = 1 / (max|Y| * norm)
                    const float sM = (M > 0.f) ? (1.f / (M * P.norm)) : 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] *= P.norm;          // y = Y / sqrt(d')
#pragma unroll
                    for (int kk = 0; kk < KT; ++kk) {
                        if (k0 + kk < K) {
                            const float delta = C.c_scale[k0 + kk] * M;   // Delta_k = c_scale_k * max|Y|
                            const float inv = C.c_inv[k0 + kk] * sM;
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                float t = fminf(fmaxf(v[e] * inv, -fD), fD);
                                float q = (t + MAGIC) - MAGIC;
                                float err = fmaf(-q, delta, v[e]);
                                acc[kk] = fmaf(err, err, acc[kk]);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int kk = 0; kk < KT; ++kk) {
                float a = acc[kk];
                if (tt >= 32) {
                    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(FULL, a, o);
                    if (active && lane == 0 && k0 + kk < K) atomicAdd(&row_err[k0 + kk], a);
                } else {
                    for (int o = tt >> 1; o > 0; o >>= 1) a += __shfl_xor_sync(FULL, a, o);
                    if (active && j == 0 && k0 + kk < K) row_err[k0 + kk] = a;
                }
            }
        }
        __syncthreads();
        // per-row results out, block totals in double
        for (int i = threadIdx.x; i < P.rows_per_cta * K; i += NT) {
            const int t = i / K, kx = i - t * K;
            const long long r = row0 + t;
            if (r < P.n_rows && err_rows) err_rows[r * K + kx] = row_err_all[t * GBS_MAX_CANDIDATES + kx];
        }
        if (threadIdx.x < K) {
            double s = 0.0;
            for (int t = 0; t < P.rows_per_cta; ++t)
                if (row0 + t < P.n_rows) s += (double)row_err_all[t * GBS_MAX_CANDIDATES + threadIdx.x];
            cta_sum[threadIdx.x] += s;
        }
        __syncthreads();
    }
    if (threadIdx.x < K) atomicAdd(&err_sum[threadIdx.x], cta_sum[threadIdx.x]);
}

// ======================================================================================
// dequantize
// ======================================================================================
// asym: unsigned fields, v = field * delta + zero (the asymmetric quantizer); else two's-complement fields.
template <int BITS>
__device__ __forceinline__ void unpack8(const unsigned char* src, float delta, float v[8], bool asym = false,
                                        float zero = 0.f)
{
    unsigned word;
    if (BITS == 4) word = (unsigned)src[0] | ((unsigned)src[1] << 8) | ((unsigned)src[2] << 16) | ((unsigned)src[3] << 24);
    else word = (unsigned)src[0] | ((unsigned)src[1] << 8) | ((unsigned)src[2] << 16);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int f = (int)((word >> (BITS * e)) & ((1u << BITS) - 1u));
        if (!asym) f = (f << (32 - BITS)) >> (32 - BITS);    // sign-extend
        v[e] = fmaf((float)f, delta, zero);
    }
}

__device__ __forceinline__ void store8(float* dst, const float v[8])
{
    reinterpret_cast<float4*>(dst)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(dst)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

__device__ __forceinline__ void store8(__nv_bfloat16* dst, const float v[8])
{
    unsigned w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
        w[e] = *reinterpret_cast<unsigned*>(&h);
    }
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void store1(float* dst, float v) { *dst = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* dst, float v) { *dst = __float2bfloat16_rn(v); }

// yhat = q * Delta, rotated domain: pure streaming, one thread per chunk of 8 codes.
template <typename OutT, int BITS>
__global__ void __launch_bounds__(NT) k_dequantize_plain(int d_pad, int G, int spr, int asym, long long n_chunks,
                                                         const unsigned char* __restrict__ codes,
                                                         const float* __restrict__ scales,
                                                         OutT* __restrict__ out)
{
    const int chunks = d_pad >> 3;
    for (long long g = (long long)blockIdx.x * NT + threadIdx.x; g < n_chunks; g += (long long)gridDim.x * NT) {
        const long long row = g / chunks;
        const int ch = (int)(g - row * chunks);
        const long long si = (row * spr + (ch * 8) / G) * (asym ? 2 : 1);
        const float delta = __ldg(scales + si);
        const float zero = asym ? __ldg(scales + si + 1) : 0.f;
        float v[8];
        unpack8<BITS>(codes + g * BITS, delta, v, asym != 0, zero);
        store8(out + g * 8, v);
    }
}

// The same for rows whose width is a multiple of 256 (or is 128), warp-cooperative: one warp item is 256 consecutive
// codes of the flat code stream (96 or 128 bytes, read as coalesced 32-bit words) and 512 or 1024 contiguous output
// bytes, and every store instruction of the warp covers 512 contiguous bytes.  Lane l turns codes [8l, 8l+8) of the
// item into bf16, or codes [4l, 4l+4) and [128+4l, 128+4l+4) into fp32.  The kernel is bound by the device's write
// bandwidth (the output is 5 to 11 times the size of the input).
template <typename OutT, int BITS>
__global__ void __launch_bounds__(NT) k_dequantize_stream(int d_pad, int glog, int spr, int asym, long long total_codes,
                                                          const unsigned* __restrict__ words,
                                                          const float* __restrict__ scales, OutT* __restrict__ out)
{
    constexpr bool WIDE = sizeof(OutT) == 4;        // fp32 output: two groups of four codes per lane
    constexpr int PER = WIDE ? 4 : 8;               // codes per lane and store
    constexpr int NST = WIDE ? 2 : 1;               // groups (= stores) per lane and item
    constexpr int UNR = 4;                          // items per warp and pass: all their loads are issued first
    const int lane = threadIdx.x & 31;
    const long long n_items = (total_codes + 255) >> 8;
    const long long last_word = (total_codes * BITS >> 5) - 1;
    const long long stride = (long long)gridDim.x * (NT / 32) * UNR;
    long long item0 = ((long long)blockIdx.x * (NT / 32) + (threadIdx.x >> 5)) * UNR;
    // position of the pass's first code, kept up to date without a division per item
    long long row = (item0 << 8) / d_pad;
    int col = (int)((item0 << 8) - row * d_pad);
    const long long row_step = (stride << 8) / d_pad;
    const int col_step = (int)((stride << 8) - row_step * d_pad);
    // per-lane constants: where this lane's group starts inside an item (codes, words, bit shift), and whether its
    // field runs into a second word
    int c_of[NST], w_of[NST], sh_of[NST];
    bool two[NST];
#pragma unroll
    for (int h = 0; h < NST; ++h) {
        c_of[h] = WIDE ? 128 * h + 4 * lane : 8 * lane;
        w_of[h] = (c_of[h] * BITS) >> 5;
        sh_of[h] = (c_of[h] * BITS) & 31;
        two[h] = sh_of[h] + PER * BITS > 32;
    }
    const int amul = asym ? 2 : 1;
    for (; item0 < n_items; item0 += stride) {
        // every item of the pass complete and not the buffer's last: no bound checks on the loads and stores
        const bool inner = item0 + UNR < n_items;
        const unsigned* wp = words + item0 * (8 * BITS);
        OutT* op = out + (item0 << 8);
        unsigned field[UNR][NST];
        float delta[UNR][NST], zero[UNR][NST];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
#pragma unroll
            for (int h = 0; h < NST; ++h) {
                field[u][h] = 0u; delta[u][h] = 0.f; zero[u][h] = 0.f;
                const int widx = u * (8 * BITS) + w_of[h];
                if (inner || ((item0 + u) << 8) + c_of[h] < total_codes) {
                    const unsigned lo = __ldg(wp + widx);
                    unsigned hi = 0u;
                    if (two[h] && (inner || item0 * (8 * BITS) + widx < last_word)) hi = __ldg(wp + widx + 1);
                    field[u][h] = __funnelshift_r(lo, hi, sh_of[h]);
                    // the group's row and scale (rows of 128 codes: an item spans two rows)
                    int cc = col + 256 * u + c_of[h];
                    long long r = row;
                    while (cc >= d_pad) { cc -= d_pad; ++r; }
                    const float* sp = scales + (r * spr + (cc >> glog)) * amul;
                    delta[u][h] = __ldg(sp);
                    if (asym) zero[u][h] = __ldg(sp + 1);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
#pragma unroll
            for (int h = 0; h < NST; ++h) {
                if (!inner && !(((item0 + u) << 8) + c_of[h] < total_codes)) continue;
                // Fields -> floats without integer conversions: the group's fields are spread to one per nibble
                // (3-bit fields by three mask-and-shift steps), symmetric codes turned into offset binary by one XOR
                // of every sign bit, each nibble dropped into the mantissa of 2^23 by a byte permute, and the
                // offset removed by an exact subtraction:  2^23 + (q + off)  -  (2^23 + off)  =  q.
                unsigned nib = field[u][h];
                if (BITS == 3) {
                    nib = (nib & 0x00000fffu) | ((nib & 0x00fff000u) << 4);       // 12 bits per half-word
                    nib = (nib & 0x003f003fu) | ((nib & 0x0fc00fc0u) << 2);       // 6 bits per byte
                    nib = (nib & 0x07070707u) | ((nib & 0x38383838u) << 1);       // 3 bits per nibble
                }
                constexpr unsigned SIGNS = BITS == 3 ? 0x44444444u : 0x88888888u;
                constexpr float OFF = BITS == 3 ? 4.f : 8.f;
                if (!asym) nib ^= SIGNS;
                const unsigned even = nib & 0x0f0f0f0fu, odd = (nib >> 4) & 0x0f0f0f0fu;
                const float bias = 8388608.f + (asym ? 0.f : OFF);
                float v[PER];
#pragma unroll
                for (int e = 0; e < PER; ++e) {
                    // byte e/2 of the even or odd word, below the three upper bytes of 2^23 (0x4B000000)
                    const unsigned fb = __byte_perm((e & 1) ? odd : even, 0x4B000000u, 0x7440u + (unsigned)(e >> 1));
                    v[e] = fmaf(__uint_as_float(fb) - bias, delta[u][h], zero[u][h]);
                }
                OutT* dst = op + 256 * u + c_of[h];
                if (WIDE) {
                    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                } else {
                    unsigned o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                        o[e] = *reinterpret_cast<unsigned*>(&b2);
                    }
                    *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
        row += row_step;
        col += col_step;
        if (col >= d_pad) { col -= d_pad; ++row; }
    }
}

// The same work with the codes staged through shared memory: a CTA takes tiles of 64 items (16 384 codes, 6 or 8 KB
// of packed bytes), brought in by 16-byte asynchronous copies three tiles ahead of their use, so that the unpacking
// threads read their fields from shared memory and never wait on a global load (the direct-load form above is bound
// by exactly that wait).  The scales (one load per lane and item) are fetched one tile ahead into registers.
constexpr int DQ_TILE_ITEMS = 64;
constexpr int DQ_STAGES = 4;
#ifndef DQ_BLOCKS_PER_SM
#define DQ_BLOCKS_PER_SM 4
#endif

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}

template <typename OutT, int BITS>
__global__ void __launch_bounds__(NT) k_dequantize_staged(int d_pad, int glog, int spr, int asym, long long total_codes,
                                                          const unsigned* __restrict__ words,
                                                          const float* __restrict__ scales, OutT* __restrict__ out)
{
    constexpr bool WIDE = sizeof(OutT) == 4;
    constexpr int PER = WIDE ? 4 : 8;
    constexpr int NST = WIDE ? 2 : 1;
    constexpr int IPW = DQ_TILE_ITEMS / (NT / 32);           // items per warp and tile: 8
    constexpr int TILE_WORDS = DQ_TILE_ITEMS * 8 * BITS;     // 32-bit words of packed codes per tile
    __shared__ __align__(16) unsigned stage[DQ_STAGES][TILE_WORDS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long n_items = (total_codes + 255) >> 8;
    const long long n_tiles = (n_items + DQ_TILE_ITEMS - 1) / DQ_TILE_ITEMS;
    const long long total_chunks = (total_codes * BITS) >> 7;            // 16-byte pieces of the code stream
    const int amul = asym ? 2 : 1;

    int c_of[NST], w_of[NST], sh_of[NST];
#pragma unroll
    for (int h = 0; h < NST; ++h) {
        c_of[h] = WIDE ? 128 * h + 4 * lane : 8 * lane;
        w_of[h] = (c_of[h] * BITS) >> 5;
        sh_of[h] = (c_of[h] * BITS) & 31;
    }
    auto fetch = [&](long long tile, int slot) {                          // all threads: the tile's packed bytes
        if (tile < n_tiles) {
            const long long chunk0 = tile * (TILE_WORDS / 4);
            for (int i = threadIdx.x; i < TILE_WORDS / 4; i += NT)
                if (chunk0 + i < total_chunks) cp_async16(&stage[slot][4 * i], words + 4 * (chunk0 + i));
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // scale (and zero point) of every group this lane will unpack in a tile.  Rows are contiguous and a group divides a
    // row, so with groups the scale index is simply (flat code index) >> log2(group); with one scale per row it is the
    // row, found by one division per tile and counting from there (rows are a whole number of items, or half an item
    // when 128 wide).
    const int ipr = d_pad >> 8;                                            // items per row (0 for 128-wide rows)
    const bool per_row = glog >= 31;
    auto fetch_scales = [&](long long tile, float (&dl)[IPW][NST], float (&zr)[IPW][NST]) {
        const long long item0 = tile * DQ_TILE_ITEMS + warp * IPW;
        const bool whole = (tile + 1) * ((long long)DQ_TILE_ITEMS << 8) <= total_codes;     // no ragged end in this tile
        long long r = 0;
        int ci = 0;
        if (per_row) {
            r = ipr ? item0 / ipr : 2 * item0;
            ci = ipr ? (int)(item0 - r * ipr) : 0;
        }
#pragma unroll
        for (int u = 0; u < IPW; ++u) {
#pragma unroll
            for (int h = 0; h < NST; ++h) {
                dl[u][h] = 0.f; zr[u][h] = 0.f;
                const long long code = ((item0 + u) << 8) + c_of[h];
                if (whole || (tile < n_tiles && code < total_codes)) {
                    const long long si = per_row ? (ipr ? r : r + (c_of[h] >> 7)) : (code >> glog);
                    const float* sp = scales + si * amul;
                    dl[u][h] = __ldg(sp);
                    if (asym) zr[u][h] = __ldg(sp + 1);
                }
            }
            if (per_row) { if (ipr) { if (++ci == ipr) { ci = 0; ++r; } } else r += 2; }
        }
    };

    long long tile = blockIdx.x;
    const long long tstride = gridDim.x;
#pragma unroll
    for (int j = 0; j < DQ_STAGES - 1; ++j) fetch(tile + j * tstride, j);
    float dl[IPW][NST], zr[IPW][NST], dl_n[IPW][NST], zr_n[IPW][NST];
    fetch_scales(tile, dl, zr);
    for (int it = 0; tile < n_tiles; tile += tstride, ++it) {
        fetch(tile + (DQ_STAGES - 1) * tstride, (it + DQ_STAGES - 1) % DQ_STAGES);
        fetch_scales(tile + tstride, dl_n, zr_n);
        asm volatile("cp.async.wait_group %0;" ::"n"(DQ_STAGES - 1) : "memory");
        __syncthreads();
        const unsigned* sw = stage[it % DQ_STAGES];
        const bool whole = (tile + 1) * ((long long)DQ_TILE_ITEMS << 8) <= total_codes;
#pragma unroll
        for (int u = 0; u < IPW; ++u) {
            const long long item = tile * DQ_TILE_ITEMS + warp * IPW + u;
#pragma unroll
            for (int h = 0; h < NST; ++h) {
                if (!whole && (item << 8) + c_of[h] >= total_codes) continue;
                const int widx = (warp * IPW + u) * (8 * BITS) + w_of[h];
                const unsigned lo = sw[widx];
                const unsigned hi = sw[widx + 1 < TILE_WORDS ? widx + 1 : widx];
                unsigned nib = __funnelshift_r(lo, hi, sh_of[h]);
                if (BITS == 3) {
                    nib = (nib & 0x00000fffu) | ((nib & 0x00fff000u) << 4);
                    nib = (nib & 0x003f003fu) | ((nib & 0x0fc00fc0u) << 2);
                    nib = (nib & 0x07070707u) | ((nib & 0x38383838u) << 1);
                }
                constexpr unsigned SIGNS = BITS == 3 ? 0x44444444u : 0x88888888u;
                constexpr float OFF = BITS == 3 ? 4.f : 8.f;
                if (!asym) nib ^= SIGNS;
                const unsigned even = nib & 0x0f0f0f0fu, odd = (nib >> 4) & 0x0f0f0f0fu;
                const float bias = 8388608.f + (asym ? 0.f : OFF);
                float v[PER];
#pragma unroll
                for (int e = 0; e < PER; ++e) {
                    const unsigned fb = __byte_perm((e & 1) ? odd : even, 0x4B000000u, 0x7440u + (unsigned)(e >> 1));
                    v[e] = fmaf(__uint_as_float(fb) - bias, dl[u][h], zr[u][h]);
                }
                OutT* dst = out + (item << 8) + c_of[h];
                if (WIDE) {
                    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                } else {
                    unsigned o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                        o[e] = *reinterpret_cast<unsigned*>(&b2);
                    }
                    *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
        __syncthreads();                                  // the slot refilled next is the one just read
#pragma unroll
        for (int u = 0; u < IPW; ++u)
#pragma unroll
            for (int h = 0; h < NST; ++h) { dl[u][h] = dl_n[u][h]; zr[u][h] = zr_n[u][h]; }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// xhat = (H^T yhat / sqrt(d'))[0:d]: same shared-memory machinery with the transposed H_m.
template <typename OutT, int BITS, bool WIDE>
__global__ void __launch_bounds__(NT) k_dequantize_inverse(GenericParams P, const unsigned char* __restrict__ codes,
                                                           const float* __restrict__ scales,
                                                           OutT* __restrict__ out)
{
    extern __shared__ __align__(16) unsigned char smem[];
    SmemLayout L = carve(P, smem);
    stage_hm(P, L.hm_s);
    const int tt = 1 << P.tt_log2;
    const int team = threadIdx.x >> P.tt_log2;
    const int j = threadIdx.x & (tt - 1);
    float* rowbuf = L.rowbuf + (size_t)team * P.row_floats;

    for (long long row0 = (long long)blockIdx.x * P.rows_per_cta; row0 < P.n_rows;
         row0 += (long long)gridDim.x * P.rows_per_cta) {
        const long long row = row0 + team;
        const bool active = row < P.n_rows;
        if (active) {
            const unsigned char* crow = codes + row * P.row_bytes;
            for (int ch = j; ch < P.chunks; ch += tt) {
                float v[8];
                const long long si = (row * P.spr + (ch * 8) / P.G) * (P.asym ? 2 : 1);
                unpack8<BITS>(crow + ch * BITS, __ldg(scales + si), v, P.asym != 0, P.asym ? __ldg(scales + si + 1) : 0.f);
                butterflies<8>(v);
                const int p = ch * 8 + (ch >> 2);
#pragma unroll
                for (int e = 0; e < 8; ++e) rowbuf[p + e] = v[e];
            }
        }
        run_passes_and_mix<WIDE>(P, rowbuf, L.hm_s, j, tt);
        if (active) {
            OutT* orow = out + row * P.d;
            for (int i = j; i < P.d; i += tt) store1(orow + i, rowbuf[pidx(i)] * P.norm);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
int ceil_log2(int v)
{
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
}

void fill_params(const gbs_plan* p, GenericParams& P, int64_t n_rows, int64_t stride, bool inverse)
{
    P.d = p->d; P.d_pad = p->d_pad; P.k = p->k; P.m = p->m; P.n2 = 1 << p->k;
    P.group = p->group; P.G = p->group ? p->group : p->d_pad;
    P.spr = p->group ? p->d_pad / p->group : 1;
    P.asym = p->asym;
    P.levels = p->levels;
    P.norm = p->norm; P.c_scale = p->c_scale; P.c_inv = p->c_inv;
    P.chunks = p->d_pad / 8;
    int tl = ceil_log2(P.chunks);
    if (tl > 8) tl = 8;
    P.tt_log2 = tl;
    P.rows_per_cta = NT >> tl;
    if ((P.G & (P.G - 1)) == 0 && P.G <= 256) { P.red_mode = 1; P.seg_lanes = P.G / 8; }
    else if (P.G % 256 == 0) { P.red_mode = 2; P.seg_lanes = 32; }
    else { P.red_mode = 3; P.seg_lanes = 1; }
    P.row_floats = p->d_pad + p->d_pad / 32 + 1;
    P.row_bytes = p->d_pad * p->bits / 8;
    P.stage_bytes = (P.row_bytes + 15) & ~15;
    // butterfly passes over bits 3 .. k-1, at most 4 bits each, split evenly
    int rem = p->k - 3, np = (rem + 3) / 4, s = 3;
    P.n_pass = np;
    for (int i = 0; i < np; ++i) {
        int r = rem / np + (i < rem % np ? 1 : 0);
        P.pass_s[i] = s; P.pass_r[i] = r; s += r;
    }
    P.n_rows = n_rows; P.stride = stride;
    P.hm = p->d_hm ? (p->d_hm + (inverse ? p->m * p->m : 0)) : nullptr;
}

size_t base_smem(const GenericParams& P)
{
    size_t off = sizeof(float) * (size_t)P.rows_per_cta * P.row_floats;
    off += sizeof(unsigned) * (size_t)P.rows_per_cta * P.spr;
    off = (off + 15) & ~(size_t)15;
    off += sizeof(float) * (size_t)((P.m > 1) ? P.m * P.m : 0);
    off = (off + 15) & ~(size_t)15;
    return off;
}

int grid_for(const gbs_plan* p, const GenericParams& P, size_t smem)
{
    long long need = (P.n_rows + P.rows_per_cta - 1) / P.rows_per_cta;
    int per_sm = (int)((size_t)(228 * 1024) / (smem + 1024));
    if (per_sm > 2048 / NT) per_sm = 2048 / NT;
    if (per_sm < 1) per_sm = 1;
    long long cap = (long long)p->sm_count * per_sm;
    return (int)(need < cap ? need : cap);
}

template <typename KernelT>
cudaError_t prep(KernelT kernel, size_t smem)
{
    if (smem > 48 * 1024)
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    return cudaSuccess;
}

}  // namespace

size_t gbs_generic_smem_bytes(const gbs_plan* p, int* rows_per_cta)
{
    GenericParams P;
    fill_params(p, P, 0, 0, false);
    if (rows_per_cta) *rows_per_cta = P.rows_per_cta;
    size_t rq = base_smem(P) + (size_t)P.rows_per_cta * P.stage_bytes;
    size_t ce = base_smem(P) + sizeof(double) * GBS_MAX_CANDIDATES +
                sizeof(float) * (size_t)P.rows_per_cta * GBS_MAX_CANDIDATES;
    return rq > ce ? rq : ce;
}

int gbs_generic_rotate_quantize(const gbs_plan* p, const void* x, int x_dtype, int64_t n_rows, int64_t stride,
                                void* codes, float* scales, float* y_opt, cudaStream_t stream)
{
    GenericParams P;
    fill_params(p, P, n_rows, stride, false);
    const size_t smem = base_smem(P) + (size_t)P.rows_per_cta * P.stage_bytes;
    const int grid = grid_for(p, P, smem);
    cudaError_t e;
#define LAUNCH_RQ_W(T, B, W)                                                                  \
    do {                                                                                      \
        e = prep(k_rotate_quantize<T, B, W>, smem);                                           \
        if (e == cudaSuccess) {                                                               \
            k_rotate_quantize<T, B, W><<<grid, NT, smem, stream>>>(P, (const T*)x, (unsigned char*)codes, scales, y_opt); \
            e = cudaGetLastError();                                                           \
        }                                                                                     \
    } while (0)
#define LAUNCH_RQ(T, B)                                                                       \
    do {                                                                                      \
        if (p->m > 28) LAUNCH_RQ_W(T, B, true); else LAUNCH_RQ_W(T, B, false);                \
    } while (0)
    if (x_dtype == GBS_DTYPE_F32) { if (p->bits == 3) LAUNCH_RQ(float, 3); else LAUNCH_RQ(float, 4); }
    else { if (p->bits == 3) LAUNCH_RQ(__nv_bfloat16, 3); else LAUNCH_RQ(__nv_bfloat16, 4); }
#undef LAUNCH_RQ
#undef LAUNCH_RQ_W
    return (int)e;
}

int gbs_generic_clip_error(const gbs_plan* p, const void* x, int x_dtype, int64_t n_rows, int64_t stride,
                           const float* c_scale_k, const float* c_inv_k, int K, double* err_sum,
                           float* err_rows, cudaStream_t stream)
{
    GenericParams P;
    fill_params(p, P, n_rows, stride, false);
    ClipConsts C;
    for (int i = 0; i < GBS_MAX_CANDIDATES; ++i) {
        C.c_scale[i] = i < K ? c_scale_k[i] : 0.f;
        C.c_inv[i] = i < K ? c_inv_k[i] : 0.f;
    }
    const size_t smem = base_smem(P) + sizeof(double) * GBS_MAX_CANDIDATES +
                       sizeof(float) * (size_t)P.rows_per_cta * GBS_MAX_CANDIDATES;
    const int grid = grid_for(p, P, smem);
    cudaError_t e;
#define LAUNCH_CE(T, W)                                                                       \
    do {                                                                                      \
        e = prep(k_clip_error<T, W>, smem);                                                   \
        if (e == cudaSuccess) {                                                               \
            k_clip_error<T, W><<<grid, NT, smem, stream>>>(P, C, K, (const T*)x, err_sum, err_rows); \
            e = cudaGetLastError();                                                           \
        }                                                                                     \
    } while (0)
    if (x_dtype == GBS_DTYPE_F32) { if (p->m > 28) LAUNCH_CE(float, true); else LAUNCH_CE(float, false); }
    else { if (p->m > 28) LAUNCH_CE(__nv_bfloat16, true); else LAUNCH_CE(__nv_bfloat16, false); }
#undef LAUNCH_CE
    return (int)e;
}

int gbs_generic_dequantize(const gbs_plan* p, const void* codes, const float* scales, int64_t n_rows,
                           void* out, int out_dtype, int inverse, cudaStream_t stream)
{
    GenericParams P;
    fill_params(p, P, n_rows, 0, inverse != 0);
    cudaError_t e = cudaSuccess;
    if (!inverse && (P.d_pad % 256 == 0 || P.d_pad == 128)) {
        // warp-cooperative streaming form; a quantization group (a power of two >= 8) never splits a lane's codes
        const long long total = (long long)n_rows * P.d_pad;
        const long long items = (total + 255) >> 8;
        long long blocks = (items + (NT / 32) * 4 - 1) / ((NT / 32) * 4);        // four items per warp and pass
        // the kernel is bound by the latency of its (small) loads under the pressure of its own stores, i.e. by the
        // bytes in flight: measured best with four resident blocks per SM for 2-byte outputs, eight for 4-byte ones
        const long long cap = (long long)p->sm_count * (out_dtype == GBS_DTYPE_F32 ? 8 : 4);
        const int grid = (int)(blocks < cap ? blocks : cap);
        int glog = 31;                               // one scale per row: every column maps to scale 0
        if (p->group) { glog = 0; while ((1 << glog) < p->group) ++glog; }
        const long long tiles = (items + DQ_TILE_ITEMS - 1) / DQ_TILE_ITEMS;
        const long long cap2 = (long long)p->sm_count * DQ_BLOCKS_PER_SM;
        const int grid2 = (int)(tiles < cap2 ? tiles : cap2);
        // the staged form pays a three-tile prologue per block: it wins once a block has a few tiles to work through
        // (and always for 4-byte outputs, where the direct form holds too few bytes in flight); measured crossover
        const bool staged = out_dtype == GBS_DTYPE_F32 || 2 * tiles >= 5 * cap2;
#define LAUNCH_DS(T, B)                                                                            \
    do {                                                                                           \
        if (staged)                                                                                \
            k_dequantize_staged<T, B><<<grid2, NT, 0, stream>>>(P.d_pad, glog, P.spr, P.asym, total,\
                                                               (const unsigned*)codes, scales, (T*)out); \
        else                                                                                       \
        k_dequantize_stream<T, B><<<grid, NT, 0, stream>>>(P.d_pad, glog, P.spr, P.asym, total,     \
                                                           (const unsigned*)codes, scales, (T*)out); \
        e = cudaGetLastError();                                                                    \
    } while (0)
        if (out_dtype == GBS_DTYPE_F32) { if (p->bits == 3) LAUNCH_DS(float, 3); else LAUNCH_DS(float, 4); }
        else { if (p->bits == 3) LAUNCH_DS(__nv_bfloat16, 3); else LAUNCH_DS(__nv_bfloat16, 4); }
#undef LAUNCH_DS
        return (int)e;
    }
    if (!inverse) {
        const long long n_chunks = (long long)n_rows * P.chunks;
        long long blocks = (n_chunks + NT - 1) / NT;
        long long cap = (long long)p->sm_count * 8 * 4;
        const int grid = (int)(blocks < cap ? blocks : cap);
#define LAUNCH_DP(T, B)                                                                            \
    do {                                                                                           \
        k_dequantize_plain<T, B><<<grid, NT, 0, stream>>>(P.d_pad, P.G, P.spr, P.asym, n_chunks,    \
                                                          (const unsigned char*)codes, scales, (T*)out); \
        e = cudaGetLastError();                                                                    \
    } while (0)
        if (out_dtype == GBS_DTYPE_F32) { if (p->bits == 3) LAUNCH_DP(float, 3); else LAUNCH_DP(float, 4); }
        else { if (p->bits == 3) LAUNCH_DP(__nv_bfloat16, 3); else LAUNCH_DP(__nv_bfloat16, 4); }
#undef LAUNCH_DP
        return (int)e;
    }
    const size_t smem = base_smem(P);
    const int grid = grid_for(p, P, smem);
#define LAUNCH_DI_W(T, B, W)                                                                       \
    do {                                                                                           \
        e = prep(k_dequantize_inverse<T, B, W>, smem);                                             \
        if (e == cudaSuccess) {                                                                    \
            k_dequantize_inverse<T, B, W><<<grid, NT, smem, stream>>>(P, (const unsigned char*)codes, scales, (T*)out); \
            e = cudaGetLastError();                                                                \
        }                                                                                          \
    } while (0)
#define LAUNCH_DI(T, B)                                                                            \
    do {                                                                                           \
        if (p->m > 28) LAUNCH_DI_W(T, B, true); else LAUNCH_DI_W(T, B, false);                     \
    } while (0)
    if (out_dtype == GBS_DTYPE_F32) { if (p->bits == 3) LAUNCH_DI(float, 3); else LAUNCH_DI(float, 4); }
    else { if (p->bits == 3) LAUNCH_DI(__nv_bfloat16, 3); else LAUNCH_DI(__nv_bfloat16, 4); }
#undef LAUNCH_DI
#undef LAUNCH_DI_W
    return (int)e;
}
