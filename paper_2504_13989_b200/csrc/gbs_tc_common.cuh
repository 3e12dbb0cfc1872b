// Shared by the tensor-core kernel families (included once per translation unit, inside no namespace):
// PTX wrappers for mbarriers, TMA, tcgen05 (alloc / mma / commit / ld), packed fp32 pairs, the MMA
// descriptors, and the register-level epilogue arithmetic (H_32 butterflies, quantize + pack).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace {

constexpr unsigned WAIT_HINT_NS = 20000;          // a waiting thread may sleep this long per poll
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // a wait gives up after two seconds

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(void* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(WAIT_HINT_NS) : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait: gives up limit_ns (by default WAIT_LIMIT_NS) after its first unsuccessful poll.  Returns false if the wait
// expired (or, with watch_abort, once another role has aborted).  The epilogue warps wait without
// watch_abort: they leave only on their own expiry, and the four warps of a token slot leave together.
__device__ __noinline__ bool mbar_wait_slow(volatile int* abort_flag, void* bar, unsigned parity, int* status, int code,
                                            bool watch_abort, unsigned long long limit_ns = WAIT_LIMIT_NS)
{
    const unsigned long long t0 = global_ns();
    for (unsigned i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 15u) == 0) {
            if (watch_abort && *abort_flag) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    atomicCAS(status, 0, code);
    return false;
}
__device__ __forceinline__ bool mbar_wait(volatile int* abort_flag, void* bar, unsigned parity, int* status, int code,
                                          bool watch_abort = true)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(abort_flag, bar, parity, status, code, watch_abort);
}

// A producer that leaves its loop through the abort flag has copies on their way into the block's shared memory.  It
// gives the stages it armed (uses it_next - 1, it_next - 2, .. of a ring of n_stages `full` barriers; use i fills stage
// i % n_stages in phase (i / n_stages) & 1) a bounded time, two milliseconds in all, to complete before the block ends.
__device__ __noinline__ void drain_copies(unsigned long long* full, int n_stages, int it_next)
{
    const unsigned long long t0 = global_ns();
    for (int i = it_next - 1; i >= 0 && i >= it_next - n_stages; --i)
        while (!mbar_try_wait(&full[i % n_stages], (unsigned)(i / n_stages) & 1u) && global_ns() - t0 < 2000000ull) {}
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// L2 prefetch of the box a later tma_load_3d with the same coordinates will fetch.  It moves lines from
// DRAM into L2 only, and L2 is where all global writes of the device land, so it is harmless to issue
// while an earlier kernel in the stream may still be writing the tensor: nothing is read into the SM.
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global [%0, {%1, %2, %3}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, void* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(unsigned* slot, unsigned cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned addr, unsigned cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_f16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                         unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The same with the descriptors as (low, high) words and the accumulate flag fixed at compile time: the
// issuing thread shares its scheduler with busy epilogue warps, so every instruction it spends between two
// MMAs delays the tensor cores; a k-step then costs one add on each low word and the MMA itself.
template <bool ACCUMULATE>
__device__ __forceinline__ void umma_f16_words(unsigned d_tmem, unsigned a_lo, unsigned a_hi, unsigned b_lo, unsigned b_hi,
                                               unsigned idesc)
{
    if (ACCUMULATE) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.eq.b32 p, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\t"
            "mov.b64 db, {%3, %4};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, 0, 0;\n\t"
            "mov.b64 da, {%1, %2};\n\t"
            "mov.b64 db, {%3, %4};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc) : "memory");
    }
}
__device__ __forceinline__ void umma_commit(void* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane -> 32 registers.  The load is asynchronous:
// tmem_ld_wait() must be called (it names the registers so nothing is scheduled across it).
__device__ __forceinline__ void tmem_ld32_issue(unsigned taddr, unsigned r[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(unsigned r[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// packed fp32 pairs (sm_100 f32x2 arithmetic: two lanes per issue slot)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk(unsigned lo, unsigned hi)
{
    f32x2 d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
__device__ __forceinline__ void unpk(f32x2 v, unsigned& lo, unsigned& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---------------------------------------------------------------------------------------------
// descriptors
// ---------------------------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// descriptor version 1, swizzle mode in the top three bits (2 = 128B, 4 = 64B).
__device__ __forceinline__ unsigned long long smem_desc(unsigned addr, unsigned lbo_bytes, unsigned sbo_bytes,
                                                        unsigned layout_type)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3fffu);
    d |= (unsigned long long)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (unsigned long long)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= 1ull << 46;
    d |= (unsigned long long)layout_type << 61;
    return d;
}

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, A K-major, B N-major (or K-major), M x N.
__host__ __device__ constexpr unsigned instr_desc(int M, int N, bool b_n_major = true)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | ((b_n_major ? 1u : 0u) << 16) | ((unsigned)(N >> 3) << 17) |
           ((unsigned)(M >> 4) << 24);
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ float min3(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// min and max of 32 registers.
__device__ __forceinline__ void minmax32(const unsigned r[32], float& mn, float& mx)
{
    mn = __uint_as_float(r[0]);
    mx = mn;
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        mn = min3(__uint_as_float(r[i]), __uint_as_float(r[i + 1]), mn);
        mx = max3(__uint_as_float(r[i]), __uint_as_float(r[i + 1]), mx);
    }
}

// 32 consecutive UNSIGNED codes (asymmetric quantizer) -> packed little-endian bit stream.
//   w = sat(Y * a1 + c0) maps the clipped range [lo, hi] onto [0, 1]; s = w * (2^BITS - 1) + 2^23 leaves
//   rint(.) in the low mantissa bits (round-half-even by the FMA's own rounding).
template <int BITS>
__device__ __forceinline__ void quantize_pack32_u(const unsigned r[32], float a1, float c0, unsigned out[BITS])
{
    const float L = (float)((1 << BITS) - 1);
    const float MAGIC = 8388608.f;                        // 2^23
    unsigned acc[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        unsigned a = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float w = __saturatef(fmaf(__uint_as_float(r[8 * g + e]), a1, c0));
            const unsigned s = __float_as_uint(fmaf(w, L, MAGIC));
            unsigned t;
            asm("shf.l.clamp.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(0u), "r"(s), "r"((unsigned)(BITS * e)));
            a += t;
        }
        acc[g] = a;
    }
    if (BITS == 4) {
        constexpr unsigned C = 0x4B000000u + 0xB0000000u;   // sum_e 0x4B000000 << 4e (mod 2^32)
#pragma unroll
        for (int g = 0; g < 4; ++g) out[g] = acc[g] - C;
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) acc[g] &= 0x00ffffffu;  // the exponent pattern only touches bits >= 24
        out[0] = acc[0] | (acc[1] << 24);
        out[1] = (acc[1] >> 8) | (acc[2] << 16);
        out[2] = (acc[2] >> 16) | (acc[3] << 8);
    }
}

// Fold 8 per-thread sums across the 32 lanes of a warp: after three halving exchanges lane l holds
// candidate ((l>>4)&1)*4 + ((l>>3)&1)*2 + ((l>>2)&1) summed over 8 lanes; two more exchanges finish the
// warp sum (returned in every lane for that lane's candidate).
__device__ __forceinline__ float warp_fold8(const float acc[8], int lane)
{
    float h4[4], h2[2], h1;
    {
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float send = up ? acc[i] : acc[i + 4];
            const float keep = up ? acc[i + 4] : acc[i];
            h4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
    }
    {
        const bool up = (lane & 8) != 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float send = up ? h4[i] : h4[i + 2];
            const float keep = up ? h4[i + 2] : h4[i];
            h2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
    }
    {
        const bool up = (lane & 4) != 0;
        const float send = up ? h2[0] : h2[1];
        const float keep = up ? h2[1] : h2[0];
        h1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    h1 += __shfl_xor_sync(0xffffffffu, h1, 2);
    h1 += __shfl_xor_sync(0xffffffffu, h1, 1);
    return h1;
}

// max|.| of 32 registers.
__device__ __forceinline__ float absmax32(const unsigned r[32])
{
    float m = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 2) m = max3(fabsf(__uint_as_float(r[i])), fabsf(__uint_as_float(r[i + 1])), m);
    return m;
}

// ---------------------------------------------------------------------------------------------
// epilogue arithmetic
// ---------------------------------------------------------------------------------------------
// H_32 on 32 registers (in place, natural order) and max|.| of the result.  The four upper stages act on
// register pairs as they come out of TMEM (packed add/sub); the lowest stage pairs the two halves of a
// pair and is scalar, which leaves the results as the scalars the quantizer consumes.
__device__ __forceinline__ float fwht32_absmax(unsigned r[32])
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
    float m = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        unsigned ua, ub;
        unpk(p[i], ua, ub);
        const float a = __uint_as_float(ua), b = __uint_as_float(ub);
        const float y0 = a + b, y1 = a - b;
        r[2 * i] = __float_as_uint(y0);
        r[2 * i + 1] = __float_as_uint(y1);
        m = max3(fabsf(y0), fabsf(y1), m);
    }
    return m;
}

// 32 consecutive codes -> packed little-endian bit stream (BITS * 4 bytes).
//   w = sat(Y * a1 + 0.5) maps y/Delta in [-D, D] onto [0, 1] and clips outside (Section 3.1);
//   s = w * 2D + (2^23 + 1) leaves rint(y/Delta) + D + 1 = q + 2^(BITS-1) in the low mantissa bits
//   (round-half-even by the FMA's own rounding); fields are gathered with shift-adds, the constant
//   contributed by the 2^23 exponent pattern falls outside the kept bits or is subtracted, and a
//   final XOR with 2^(BITS-1) per field turns the offset code into the two's-complement field.
template <int BITS>
__device__ __forceinline__ void quantize_pack32(const unsigned r[32], float a1, unsigned out[BITS])
{
    const float twoD = (float)(2 * ((1 << (BITS - 1)) - 1));
    const float MAGIC = 8388609.f;                        // 2^23 + 1
    unsigned acc[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        unsigned a = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float w = __saturatef(fmaf(__uint_as_float(r[8 * g + e]), a1, 0.5f));
            const unsigned s = __float_as_uint(fmaf(w, twoD, MAGIC));
            // shift on the integer pipe (funnel shift), so that the FP32 pipe only sees the two FMAs
            unsigned t;
            asm("shf.l.clamp.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(0u), "r"(s), "r"((unsigned)(BITS * e)));
            a += t;
        }
        acc[g] = a;
    }
    if (BITS == 4) {
        // sum_e 0x4B000000 << 4e (mod 2^32) = 0x4B000000 + 0xB0000000
        constexpr unsigned C = 0x4B000000u + 0xB0000000u;
#pragma unroll
        for (int g = 0; g < 4; ++g) out[g] = (acc[g] - C) ^ 0x88888888u;
    } else {
        // the exponent pattern only touches bits >= 24, outside the 24 kept bits
#pragma unroll
        for (int g = 0; g < 4; ++g) acc[g] = (acc[g] & 0x00ffffffu) ^ 0x00924924u;
        out[0] = acc[0] | (acc[1] << 24);
        out[1] = (acc[1] >> 8) | (acc[2] << 16);
        out[2] = (acc[2] >> 16) | (acc[3] << 8);
    }
}


// ---------------------------------------------------------------------------------------------
// host: the driver entry point that encodes tensor maps, fetched through the runtime
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode()
{
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        return reinterpret_cast<EncodeTiledFn>(p);
    cudaGetLastError();
    return nullptr;
}

// looked up once; the initialisation of a function-local static is safe against concurrent first calls
EncodeTiledFn get_encode()
{
    static const EncodeTiledFn fn = lookup_encode();
    return fn;
}

}  // namespace
