// Tensor-core family "UVR": bf16 rows of padded width d' = 128 * U with U = m * 2^j <= 256 (4096 < d' <= 32768, e.g.
// the MLP width 20480 = 20 * 1024: U = 160), the rest of the transform held in REGISTERS.
//
// A padded row is viewed as X[u][c][v] (flat index u*128 + c*32 + v, c < 4, v < 32).  With 2^k = 2^j * 128 the
// rotation factors as (H_m (x) H_{2^j}) (x) H_4 (x) H_32 (Eq. (1) on the bit fields of the Sylvester index,
// Algorithm 2 for H_m):
//   * A = H_m (x) H_{2^j} (U x U, +-1) runs on the tensor cores, one token per accumulator: TMEM lane u' receives
//     the 128 coordinates u'*128 .. u'*128 + 127 of the half-transformed token.  U rows are 32-row slabs: slabs 0..3
//     are one 128-lane MMA block; slabs 4..7 (U > 128) are a second block, contracted with a WINDOW of the same
//     image of A that starts 128 - 32*rot rows into it, so that they land in lane quadrants rot, rot+1, .. of the
//     second accumulator (the other lanes receive rows nobody reads).  rot changes from token to token: over a few
//     tokens every lane quadrant, and with it every warp scheduler of the SM, gets the same number of slabs.
//   * One thread owns one lane of one slab: it reads its 128 values from TMEM once, hands the accumulator back at
//     once, runs H_4 across and H_32 inside the four chunks as butterflies in registers, takes max|.|, and scales,
//     rounds, clips and packs (Sections 2.1, 3.1) 48 or 64 bytes of codes.  Scales per group of up to 128 coordinates
//     never leave the thread, larger groups (up to 4096) are folded over neighbouring lanes by shuffles; for one scale
//     per token the warps of the token meet once at an mbarrier.
//   * Twelve epilogue warps, three per lane quadrant (U > 128: two for the first block of even / odd tokens, one for
//     the quadrant's slabs of the second block; U <= 128: every third token each), so every warp walks its tokens in
//     order and no warp holds two consecutive tokens.  128 live values need about 160 registers: the first warpgroup
//     (TMA producer, two MMA issuing threads) gives registers up, the three epilogue warpgroups take them.
//   * The token row reaches shared memory in slices of 32 u-rows (8 KB, two k-steps of the contraction); a stage of
//     the ring holds a token's slices (fewer where three such stages do not fit) behind one barrier and goes back to the
//     TMA producer as soon as both blocks have contracted it.
// Every wait is a bounded mbarrier wait; an expired wait records a code in the plan's status word and every role
// leaves through the abort flag.
#include <math.h>
#include <string.h>

#include <mutex>

#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int V = 32;
constexpr int NCOLS = 128;                        // accumulator columns per block: 4 chunks of 32 coordinates
constexpr int UMAX = 256;
constexpr int SLICE_ROWS = 32;
constexpr int SLICE_BYTES = SLICE_ROWS * NCOLS * 2;          // 8 KB: two 64-column halves of 32 rows x 128 bytes
constexpr int MAX_SLICES = 24;
constexpr int EPI_WARPS = 12;                     // three per lane quadrant
constexpr int THREADS = 32 * (4 + EPI_WARPS);     // warp 0: TMA, warps 1-2: MMA, warp 3 fills the first warpgroup
constexpr int REGS_LEAN = 32, REGS_EPI = 160;     // registers per thread after the warpgroups have rebalanced
constexpr int TSLOTS = 6;                         // rendezvous slots of the per-token maximum
constexpr int TMEM_COLS = 512;
constexpr int CTL_BYTES = 1024;

struct Ctl {
    unsigned long long full[MAX_SLICES], empty[MAX_SLICES];
    // A parity wait must never skip a phase of its barrier, so every barrier is indexed such that whoever waits on it
    // takes part in each of its phases.  tfull[t mod 12]: the accumulators of token t are written (U <= 128: tokens
    // twelve apart have the same issuing thread, the same epilogue warps and the same accumulator stage; U > 128:
    // only indices 0 and 1 are used, by the warps of the first block); tfull2[t mod 4]: the same event for the warps of
    // the second block, which take every second or fourth token; tempty[stage]: the stage has been read.
    unsigned long long tfull[12], tfull2[4], tempty[4], tbar[TSLOTS];
    unsigned long long abar;
    __align__(16) float red[TSLOTS][8];          // [slot][slab]: max|.| of the slab (one scale per token)
    unsigned tmem_base;
    volatile int abort_flag;
};
static_assert(sizeof(Ctl) <= CTL_BYTES, "control block");

struct UvrParams {
    long long n_rows;
    int U;                        // m * 2^j
    int slabs;                    // ceil(U / 32)
    int nb2;                      // slabs of the second block (0 .. 4)
    int ksteps;                   // ceil(U / 16): the contraction is padded with zero columns of A and zero rows of X
    int nslices;                  // ceil(U / 32)
    int g;                        // slices per shared-memory stage
    int n_ring;                   // shared-memory stages in use
    int a_bytes;                  // image of A
    int atom_stride;              // bytes between the 64-column K atoms of the image: U (rounded up to 8) * 128
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
};

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// Names 32 registers in an empty volatile statement: nothing that uses them moves above it (the asynchronous
// tcgen05.ld that fills them is only complete after the tcgen05.wait::ld that precedes this statement).
__device__ __forceinline__ void pin32(unsigned r[32])
{
    asm volatile(""
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// H_4 across the four chunks (index c of u*128 + c*32 + v), on the register pairs as they come out of TMEM.
__device__ __forceinline__ void cross4(unsigned r0[32], unsigned r1[32], unsigned r2[32], unsigned r3[32])
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const f32x2 a = pk(r0[2 * i], r0[2 * i + 1]), b = pk(r1[2 * i], r1[2 * i + 1]);
        const f32x2 c = pk(r2[2 * i], r2[2 * i + 1]), d = pk(r3[2 * i], r3[2 * i + 1]);
        const f32x2 s0 = add2(a, b), s1 = sub2(a, b), s2 = add2(c, d), s3 = sub2(c, d);
        unpk(add2(s0, s2), r0[2 * i], r0[2 * i + 1]);
        unpk(add2(s1, s3), r1[2 * i], r1[2 * i + 1]);
        unpk(sub2(s0, s2), r2[2 * i], r2[2 * i + 1]);
        unpk(sub2(s1, s3), r3[2 * i], r3[2 * i + 1]);
    }
}

template <int BITS>
__device__ __forceinline__ void store_codes(unsigned char* dst, const unsigned out[4 * BITS])
{
    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int i = 0; i < BITS; ++i) d4[i] = make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
}

__device__ __forceinline__ void store_y(float* dst, const unsigned r[32], float norm)
{
    float4* yo = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int i = 0; i < 8; ++i)
        yo[i] = make_float4(__uint_as_float(r[4 * i]) * norm, __uint_as_float(r[4 * i + 1]) * norm,
                            __uint_as_float(r[4 * i + 2]) * norm, __uint_as_float(r[4 * i + 3]) * norm);
}

// The bounded wait of gbs_tc_common.cuh, inlined: a call with 128 live values would have to spill them around it.
__device__ __forceinline__ bool mbar_wait_inline(volatile int* abort_flag, void* bar, unsigned parity, int* status, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (unsigned i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 15u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > WAIT_LIMIT_NS) break;
        }
    }
    *abort_flag = 1;
    atomicCAS(status, 0, code);
    return false;
}

// Lane quadrant at which the second block's slabs of the it-th token of this CTA start.
__device__ __forceinline__ int rot_of(int it, int nb2) { return nb2 == 3 ? (it & 1) : ((it * nb2) & 3); }

// TWO: U > 128, a token has a second block of slabs.
template <int BITS, bool GROUPED, bool TWO>
__global__ void __launch_bounds__(THREADS, 1) k_tc_uvr_rq(const __grid_constant__ CUtensorMap tmap,
                                                          const __grid_constant__ UvrParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Ctl* S = reinterpret_cast<Ctl*>(base);
    unsigned char* a_smem = base + CTL_BYTES;
    unsigned char* ring = a_smem + P.a_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tok = (int)P.n_rows;
    constexpr int tstride = TWO ? 2 * NCOLS : NCOLS;          // accumulator columns per token
    // accumulator stages: two tokens of two blocks, or four tokens of one block
    constexpr int tstages = TWO ? 2 : 4;
    constexpr int nfull = TWO ? 2 : 12;                       // tfull barriers in use

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_SLICES; ++s) {
            mbar_init(&S->full[s], 1);
            mbar_init(&S->empty[s], TWO ? 2 : 1);          // one commit per thread that contracts the slice
        }
        for (int s = 0; s < 12; ++s) mbar_init(&S->tfull[s], 1);
        for (int s = 0; s < 4; ++s) {
            mbar_init(&S->tfull2[s], 1);
            mbar_init(&S->tempty[s], (unsigned)P.slabs);
        }
        for (int s = 0; s < TSLOTS; ++s) mbar_init(&S->tbar[s], (unsigned)P.slabs);
        mbar_init(&S->abar, 1);
        for (int i = 0; i < TSLOTS * 8; ++i) (&S->red[0][0])[i] = 0.f;
        S->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(&S->abar, (unsigned)P.a_bytes);
        bulk_load(a_smem, P.a_img, (unsigned)P.a_bytes, &S->abar);        // plan-owned, immutable: needs no ordering
    }
    if (warp == 1) tmem_alloc(&S->tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned tmem_base = S->tmem_base;

    // The first warpgroup (producer, issuer, two idle warps) gives registers up, the three epilogue warpgroups take
    // them: 128 values per thread stay in registers only with more than the 128 a block of 512 threads starts with.
    if (warp < 4) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_LEAN));
      if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");   // nothing of the caller's memory is touched before
            int s = 0;
            unsigned ph = 0;
            bool ok = true;
            for (int tk = blockIdx.x; ok && tk < n_tok; tk += gridDim.x)
                for (int j0 = 0; j0 < P.nslices; j0 += P.g) {
                    if (!mbar_wait_inline(&S->abort_flag, &S->empty[s], ph ^ 1, P.status, 1)) { ok = false; break; }
                    const int cnt = P.nslices - j0 < P.g ? P.nslices - j0 : P.g;
                    mbar_arrive_expect_tx(&S->full[s], (unsigned)(cnt * SLICE_BYTES));
                    // a stage: the first halves (64 coordinates) of its slices one after the other, then the second halves
                    unsigned char* dst = ring + (size_t)s * P.g * SLICE_BYTES;
                    for (int j = 0; j < cnt; ++j) {
                        tma_load_4d(dst + j * (SLICE_BYTES / 2), &tmap, &S->full[s], 0, 0, (j0 + j) * SLICE_ROWS, tk);
                        tma_load_4d(dst + (P.g + j) * (SLICE_BYTES / 2), &tmap, &S->full[s], 0, 1, (j0 + j) * SLICE_ROWS, tk);
                    }
                    if (++s == P.n_ring) { s = 0; ph ^= 1; }
                }
            if (!ok) {
                // Leaving through the abort flag: the copies this thread started may still be on their way into this
                // block's shared memory.  Give each armed stage a short, bounded time to complete before the block ends
                // (walking back from the stage that would have been armed next; a stage never armed passes at once).
                const unsigned long long t0 = global_ns();
                for (int n = 0; n < P.n_ring; ++n) {
                    if (--s < 0) { s = P.n_ring - 1; ph ^= 1; }
                    while (!mbar_try_wait(&S->full[s], ph) && global_ns() - t0 < 2000000ull) {}
                }
            }
        }
      } else if (warp <= 2) {
        // ------------------------------ MMA issuers ------------------------------
        // Two issuing threads on two schedulers: what costs an issuing thread time is not the MMAs (64 cycles each on the
        // tensor pipe) but what stands between them (the poll of a stage's barrier, the commit that returns it, every
        // instruction of its own loop), and one thread alone does not keep the epilogue fed.  U > 128: thread 0
        // contracts the first block of every token, thread 1 the second (a stage returns to the producer after both
        // commits).  U <= 128: the threads take alternate tokens.
        if (lane == 0) {
            const int issuer = warp - 1;
            constexpr unsigned IDESC = instr_desc(128, NCOLS, true);
            // A: K-major, one 128-byte line per row and 64-column atom, 32 bytes per k-step.  B: N-major, atoms of 8
            // u-rows x 64 coordinates (1024 bytes), the other 64 coordinates of the slice 4 KB away.  Only the address
            // fields (bytes >> 4, low words) of the descriptors change between MMAs.
            // high words (1024 bytes between 8-row groups, descriptor version, 128-byte swizzle) are one constant;
            // B's leading offset is the distance between the two 64-coordinate halves of a stage
            constexpr unsigned D_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
            const unsigned ad_lo0 = ((smem_u32(a_smem) >> 4) & 0x3fffu) | ((16u >> 4) << 16);
            const unsigned bd_lo0 = ((smem_u32(ring) >> 4) & 0x3fffu) | ((unsigned)(P.g * (SLICE_BYTES / 2) >> 4) << 16);
            // few live values: the loop must fit the 32 registers this warpgroup keeps; a spill in it costs the tensor
            // pipe more than any arithmetic
            bool ok = mbar_wait_inline(&S->abort_flag, &S->abar, 0, P.status, 6);
            const int n_mine = ((int)blockIdx.x < n_tok) ? (n_tok - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
            const int chunks = (P.nslices + P.g - 1) / P.g;
            int s = 0;
            unsigned ph = 0;
            for (int it = 0; ok && it < n_mine; ++it) {
                if (!TWO && (it & 1) != issuer) {     // the other thread's token: step over its stages
                    for (int c = 0; c < chunks; ++c)
                        if (++s == P.n_ring) { s = 0; ph ^= 1; }
                    continue;
                }
                const int ts = it & (tstages - 1);
                if (!mbar_wait_inline(&S->abort_flag, &S->tempty[ts], ((it / tstages) & 1) ^ 1, P.status, 3)) break;
                tc_fence_after();
                const unsigned d = tmem_base + ts * tstride + (TWO ? issuer * NCOLS : 0);
                // the second block's rows come from a window of the image that starts 128 - 32 rot rows into it
                unsigned a_lo = ad_lo0 + ((TWO && issuer) ? (unsigned)((128 - 32 * rot_of(it, P.nb2)) * 128) >> 4 : 0u);
                int kk = 0;                           // k-step of the token
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait_inline(&S->abort_flag, &S->full[s], ph, P.status, 2)) { ok = false; break; }
                    tc_fence_after();
                    unsigned b_lo = bd_lo0 + (unsigned)(s * P.g) * (SLICE_BYTES >> 4);
                    const int kend = kk + 2 * P.g < P.ksteps ? kk + 2 * P.g : P.ksteps;
                    if (kk == 0) {
                        umma_f16_words<false>(d, a_lo, D_HI, b_lo, D_HI, IDESC);
                        a_lo += 2u;
                        b_lo += 16 * 128 >> 4;
                        kk = 1;
                    }
#pragma unroll 1
                    for (; kk < kend; ++kk) {
                        umma_f16_words<true>(d, a_lo, D_HI, b_lo, D_HI, IDESC);
                        // every fourth k-step ends a 64-column atom of the image: on to the next atom
                        a_lo += ((kk & 3) == 3) ? (unsigned)(P.atom_stride - 96) >> 4 : 2u;
                        b_lo += 16 * 128 >> 4;
                    }
                    umma_commit(&S->empty[s]);
                    if (++s == P.n_ring) { s = 0; ph ^= 1; }
                }
                if (ok) umma_commit((TWO && issuer) ? &S->tfull2[it & 3] : &S->tfull[TWO ? (it & 1) : it % 12]);
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_EPI));
        // ------------------------------ epilogue ------------------------------
        // Three warps per lane quadrant.  U > 128: two of them take the first block of even / odd tokens, the third
        // the quadrant's slab of the second block whenever the token's window puts one there.  U <= 128: the three
        // take every third token.  Every warp walks its tokens in order, and two tokens that share a rendezvous slot
        // (four, or six, tokens apart) are served by the same warps: a slot's phases cannot mix.
        const int q = warp & 3;                   // TMEM lane quadrant this warp may access
        const int pr = (warp - 4) >> 2;           // which of the quadrant's three warps
        const unsigned tq = tmem_base + ((unsigned)(q * 32) << 16);
        int it = 0, ts = 0, tb = 0, tf = 0, set = 0;
        unsigned tf_ph = 0, tb_ph = 0;
        for (long long row = blockIdx.x; row < P.n_rows;
             row += gridDim.x, ++it, ts = (ts + 1 == tstages ? 0 : ts + 1), set = (set == 2 ? 0 : set + 1),
                       tf = (tf + 1 == nfull ? 0 : tf + 1), tf_ph ^= (tf == 0 ? 1u : 0u),
                       tb = (tb + 1 == (TWO ? 4 : TSLOTS) ? 0 : tb + 1), tb_ph ^= (tb == 0 ? 1u : 0u)) {
            int slab = -1;
            if (TWO) {
                if (pr < 2) {
                    if ((it & 1) == pr) slab = q;                             // first block
                } else {
                    const int rel = q - rot_of(it, P.nb2);
                    if (rel >= 0 && rel < P.nb2) slab = 4 + rel;              // second block
                }
            } else if (set == pr && q * 32 < P.U) {
                slab = q;
            }
            if (slab < 0) continue;
            const int up = slab * 32 + lane;      // u'
            const bool lane_live = up < P.U;
            if (TWO && slab >= 4) {
                if (!mbar_wait_inline(&S->abort_flag, &S->tfull2[it & 3], (it >> 2) & 1, P.status, 4)) break;
            } else {
                if (!mbar_wait_inline(&S->abort_flag, &S->tfull[tf], tf_ph, P.status, 4)) break;
            }
            tc_fence_after();
            const unsigned tcol = tq + ts * tstride + (slab >= 4 ? NCOLS : 0);
            unsigned r0[32], r1[32], r2[32], r3[32];
            tmem_ld32_issue(tcol, r0);
            tmem_ld32_issue(tcol + 32, r1);
            tmem_ld32_issue(tcol + 64, r2);
            tmem_ld32_issue(tcol + 96, r3);
            tmem_ld_wait(r0);
            pin32(r1);
            pin32(r2);
            pin32(r3);
            // the accumulator has been read: hand it back to the MMA issuer before the arithmetic
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&S->tempty[ts]);

            cross4(r0, r1, r2, r3);
            float mc[4];
            mc[0] = fwht32_absmax(r0);
            mc[1] = fwht32_absmax(r1);
            mc[2] = fwht32_absmax(r2);
            mc[3] = fwht32_absmax(r3);
            if (!lane_live) mc[0] = mc[1] = mc[2] = mc[3] = 0.f;       // rows beyond U hold nothing of this token

            float a1t = 0.f;                          // one scale per token: the same factor for every chunk
            if (GROUPED) {
                if (P.gsh >= 1) {
                    mc[0] = mc[1] = fmaxf(mc[0], mc[1]);
                    mc[2] = mc[3] = fmaxf(mc[2], mc[3]);
                }
                if (P.gsh >= 2) mc[0] = mc[1] = mc[2] = mc[3] = fmaxf(mc[0], mc[2]);
                if (P.gsh > 2) {
                    float m = mc[0];
                    for (int o = 1; o < (1 << (P.gsh - 2)); o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                    mc[0] = mc[1] = mc[2] = mc[3] = m;
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    // one writer per group: its first chunk, in its first lane
                    const bool writer = (P.gsh <= 2) ? ((c & ((1 << P.gsh) - 1)) == 0)
                                                     : (c == 0 && (lane & ((1 << (P.gsh - 2)) - 1)) == 0);
                    if (writer && lane_live) P.scales[row * P.spr + ((up * 4 + c) >> P.gsh)] = P.c_scale * mc[c];
                }
            } else {
                const float mt = fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
                const unsigned mw = __reduce_max_sync(0xffffffffu, __float_as_uint(mt));
                if (lane == 0) {
                    S->red[tb][slab] = __uint_as_float(mw);
                    mbar_arrive(&S->tbar[tb]);
                }
                if (!mbar_wait_inline(&S->abort_flag, &S->tbar[tb], tb_ph, P.status, 5)) break;
                const float4* rp = reinterpret_cast<const float4*>(&S->red[tb][0]);
                const float4 m0 = rp[0], m1 = rp[1];
                const float M = fmaxf(fmaxf(fmaxf(m0.x, m0.y), fmaxf(m0.z, m0.w)), fmaxf(fmaxf(m1.x, m1.y), fmaxf(m1.z, m1.w)));
                a1t = (M > 0.f) ? __fdividef(P.c_half, M) : 0.f;
                if (slab == 0 && lane == 0) P.scales[row] = P.c_scale * M;
            }
            if (lane_live) {
                unsigned out[4 * BITS];
                // per-group factors are formed chunk by chunk: four more live values would not fit the register budget
                quantize_pack32<BITS>(r0, GROUPED ? ((mc[0] > 0.f) ? __fdividef(P.c_half, mc[0]) : 0.f) : a1t, out);
                quantize_pack32<BITS>(r1, GROUPED ? ((mc[1] > 0.f) ? __fdividef(P.c_half, mc[1]) : 0.f) : a1t, out + BITS);
                quantize_pack32<BITS>(r2, GROUPED ? ((mc[2] > 0.f) ? __fdividef(P.c_half, mc[2]) : 0.f) : a1t, out + 2 * BITS);
                quantize_pack32<BITS>(r3, GROUPED ? ((mc[3] > 0.f) ? __fdividef(P.c_half, mc[3]) : 0.f) : a1t, out + 3 * BITS);
                store_codes<BITS>(P.codes + row * P.code_row_bytes + (size_t)up * (NCOLS * BITS / 8), out);
                if (P.y_opt) {
                    float* yo = P.y_opt + row * (long long)P.d_pad + (size_t)up * NCOLS;
                    store_y(yo, r0, P.norm);
                    store_y(yo + 32, r1, P.norm);
                    store_y(yo + 64, r2, P.norm);
                    store_y(yo + 96, r3, P.norm);
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
}

int log2_chunks(int group)
{
    int gsh = 0;
    while ((V << gsh) < group) ++gsh;
    return gsh;
}

int image_rows(int U) { return (U + 7) & ~7; }             // lines per K atom: whole 8-line swizzle groups
int image_rows_last(int U) { return U > 128 ? 256 : 128; }
int image_atoms(int U) { return (U + 63) / 64; }

// The shared-memory opt-in is set once per kernel instantiation and device.
template <int BITS, bool GROUPED, bool TWO>
cudaError_t launch(int device, int grid, int smem, cudaStream_t stream, bool pdl, const CUtensorMap& tmap, const UvrParams& P)
{
    static std::mutex mu;
    static int done[64] = {};
    {
        std::lock_guard<std::mutex> lk(mu);
        if (device < 0 || device >= 64 || done[device] < smem) {
            const cudaError_t e = cudaFuncSetAttribute(k_tc_uvr_rq<BITS, GROUPED, TWO>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return e;
            if (device >= 0 && device < 64) done[device] = smem;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, k_tc_uvr_rq<BITS, GROUPED, TWO>, tmap, P);
}

}  // namespace

// Bytes of the image gbs_tc_uvr_image writes: the 64-column K atoms of A one after the other, U lines of 128 bytes each;
// the last atom has room for the lines a window of the second block (or a first block with U < 128) reaches beyond U.
int gbs_tc_uvr_image_bytes(const gbs_plan* p)
{
    const int U = p->d_pad / NCOLS;
    return ((image_atoms(U) - 1) * image_rows(U) + image_rows_last(U)) * 128;
}

// Image of A = H_m (x) H_{2^j} (U x U, bf16 +-1, K-major, 128-byte swizzle), zero beyond U.
void gbs_tc_uvr_image(const gbs_plan* p, unsigned char* img)
{
    const int U = p->d_pad / NCOLS, j = p->k - 7, jm = (1 << j) - 1, m = p->m;
    memset(img, 0, (size_t)gbs_tc_uvr_image_bytes(p));
    unsigned short* h = reinterpret_cast<unsigned short*>(img);
    for (int r = 0; r < U; ++r)
        for (int k = 0; k < U; ++k) {
            int sign = p->h_hm[(r >> j) * m + (k >> j)];
            if (__builtin_popcount((unsigned)(r & k & jm)) & 1) sign = -sign;
            const int atom = k >> 6, c = (k >> 3) & 7, e = k & 7;
            const size_t off = (size_t)atom * image_rows(U) * 128 + (size_t)r * 128 + (size_t)((c ^ (r & 7)) << 4) + e * 2;
            h[off / 2] = sign < 0 ? 0xBF80 : 0x3F80;
        }
}

bool gbs_tc_uvr_supported(const gbs_plan* p)
{
    if (p->asym || p->d_pad <= 4096 || p->d_pad % NCOLS != 0 || p->d % NCOLS != 0 || p->k < 7) return false;
    const int U = p->d_pad / NCOLS;
    if (U > UMAX || U < 80) return false;          // U = m 2^j is a multiple of 4; fewer than 80 rows leave lane quadrants idle
    if (p->group != 0) {
        if (p->group < V || (p->group & (p->group - 1)) != 0 || p->group > 4096) return false;
    }
    const int ring = (p->smem_optin - 1024 - CTL_BYTES - gbs_tc_uvr_image_bytes(p)) / SLICE_BYTES;
    return get_encode() != nullptr && ring >= (U + 31) / 32 + 2;
}

int gbs_tc_uvr_rotate_quantize(const gbs_plan* p, const void* x, int64_t n_rows, int64_t stride, void* codes,
                               float* scales, float* y_opt, cudaStream_t stream)
{
    EncodeTiledFn encode = get_encode();
    if (!encode) return (int)cudaErrorNotSupported;
    if (n_rows > (int64_t)0x7fffffff - 1) return (int)cudaErrorInvalidValue;      // TMA coordinates are 32-bit
    const int U = p->d_pad / NCOLS;
    // dims: 64 values, half h of the 128 coordinates of a u-row, u, token; one box = 32 u-rows of one half
    CUtensorMap tmap;
    const cuuint64_t gdim[4] = {64, 2, (cuuint64_t)(p->d / NCOLS), (cuuint64_t)n_rows};
    const cuuint64_t gstr[3] = {128, 256, (cuuint64_t)(stride * 2)};
    const cuuint32_t box[4] = {64, 1, SLICE_ROWS, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;

    UvrParams P;
    memset(&P, 0, sizeof(P));
    P.n_rows = n_rows;
    P.U = U;
    P.slabs = (U + 31) / 32;
    P.nb2 = P.slabs > 4 ? P.slabs - 4 : 0;
    P.ksteps = (U + 15) / 16;
    P.nslices = (U + 31) / 32;
    P.a_bytes = gbs_tc_uvr_image_bytes(p);
    P.atom_stride = image_rows(U) * 128;
    const int ring = (p->smem_optin - 1024 - CTL_BYTES - P.a_bytes) / SLICE_BYTES;     // slices that fit
    // A stage holds g slices behind one barrier: an issuing thread spends several hundred cycles on every poll and
    // every commit, far more than on the MMAs of a slice.  As many slices as leave three stages, at most a token's.
    P.g = ring / 3;
    if (P.g < 1) P.g = 1;
    if (P.g > P.nslices) P.g = P.nslices;
    if (P.g > ring / 2) P.g = ring / 2;
    P.n_ring = ring / P.g < MAX_SLICES ? ring / P.g : MAX_SLICES;
    P.code_row_bytes = p->d_pad * p->bits / 8;
    P.d_pad = p->d_pad;
    P.gsh = p->group ? log2_chunks(p->group) : 0;
    P.spr = p->group ? p->d_pad / p->group : 1;
    P.c_scale = p->c_scale;
    P.c_half = (float)(1.0 / (2.0 * (double)p->alpha));
    P.norm = p->norm;
    P.a_img = p->d_aimg_r;
    P.codes = (unsigned char*)codes;
    P.scales = scales;
    P.y_opt = y_opt;
    P.status = p->d_status;
    const int smem = 1024 + CTL_BYTES + P.a_bytes + P.n_ring * P.g * SLICE_BYTES;
    const int grid = (int)(n_rows < p->sm_count ? n_rows : p->sm_count);
    const bool pdl = p->pdl != 0;
    cudaError_t e;
#define GBS_UVR_LAUNCH(B, GR) (P.nb2 ? launch<B, GR, true>(p->device, grid, smem, stream, pdl, tmap, P) \
                                     : launch<B, GR, false>(p->device, grid, smem, stream, pdl, tmap, P))
    if (p->bits == 3)
        e = p->group ? GBS_UVR_LAUNCH(3, true) : GBS_UVR_LAUNCH(3, false);
    else
        e = p->group ? GBS_UVR_LAUNCH(4, true) : GBS_UVR_LAUNCH(4, false);
#undef GBS_UVR_LAUNCH
    return (int)e;
}
