// tcgen05 gather-concat-attention kernel (bf16, head_dim 32) for many queries per user.
//
// Persistent: one CTA per SM walks a static round-robin share of the work units, where a unit
// is (work item = history chunk of one user, group, block of up to 128 queries).  The history
// chunk is processed in tiles of 128 positions, each split into two halves of 64 positions.
// Roles (warp-specialised, 20 warps):
//   warps 0-11  three normalisation groups of four warps: thread i of a group owns query row i = TMEM lane i
//   warps 12-14 one issuing thread per group: the score MMAs and the weighted-sum MMAs of that group's halves;
//               warp 12 owns the TMEM allocation
//   warps 15-19 producers, one tile each in turn: gather pool rows into shared memory with
//               16-byte cp.async, patch the user-specific leading elements (Eq. K), publish the
//               tile; the owner of a unit's first tile also stages Q.  (A side that is not shared --
//               sharing only keys or only values -- is copied from the user's full-width rows instead.)
//
// The halves of the CTA's tile stream go to the groups in turn (half h to group h mod 3).  A group has two score
// buffers in TMEM; the weights of a half are written over the head of the scores they were computed from (32
// columns of bf16 pairs over 64 columns of fp32):
//   S_bi  = Q K_half^T                UMMA 128 x 64 x 32, A = Q smem, B = half K tile smem (K-major)
//   P_bi  = exp2(S_bi c - m) | silu   group b: tcgen05.ld -> math -> bf16 -> tcgen05.st, in place
//   O_b  += P_bi V_half               UMMA 128 x 32 x 64, A = P from TMEM, B = half V tile (MN-major)
// One thread issues both kinds of MMA of its group, in the order weighted sum of step t, scores of step t + 2
// (into the buffer the weighted sum has just read): the tensor core runs one thread's instructions in order, so
// the buffer needs no completion hand-off in between, and the scores of step t + 1 are there while the group
// normalises step t.  Why three groups: the normalisation of a half is a chain of dependent work for its warp
// (wait for the scores, TMEM load, arithmetic, TMEM store, publish; at a unit's end the accumulator read-out and
// the merge) during most of which the special-function unit of the warp's sub-partition is idle; measured on a
// stripped-down pipeline, two groups keep that unit 70 % busy, three 85 %, and registers (65536 / 640 threads =
// 96 each, enough for one 32-column chunk of scores at a time) and TMEM (3 x (2 x 64 + 32) = 480 columns) admit
// no fourth.  The groups keep separate accumulators O_b with separate reference maxima and row sums and merge
// them through shared memory when a unit ends; nothing drains between work units.
//
// Softmax bookkeeping.  The reference maximum m of a row is the largest of the first 32 scores of the group's
// first half of the unit and stays fixed: later scores may exceed it by up to 2^64 (fp32 accumulators and bf16
// P have the exponent range for that).  The row sum l is added up by the row's thread in fp32, chunk by chunk, and
// a chunk's share of it also tells when a row has left that bound (32 weights within it sum to at most 2^69); only
// then is the reference moved, O_b and the row sum rescaled (TMEM read-modify-write) and the chunk worked out again.
//
// Shared-memory tiles use the no-swizzle UMMA canonical layout: groups of 8 rows (512 bytes), inside a
// group one 128-byte core matrix per 16-byte row chunk, inside a core matrix row r%8 at 16 r.
//
// Every wait in this kernel is bounded: on time-out the CTA records an error code, raises a
// CTA-wide abort flag that ends every other wait, drains its own copies, frees its TMEM and
// returns.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"
#include "ptx_helpers.cuh"

namespace ckv {
namespace {

constexpr int D = 32;
constexpr int TK = 128;                  // positions per tile (one shared-memory stage)
constexpr int TH = 64;                   // positions per half tile = one MMA / normalisation step of a group
constexpr int NG = 3;                    // normalisation groups
constexpr int NS = 10;                   // K/V stages
constexpr int NQ = 3;                    // Q buffers
constexpr int kGroupThreads = 128;       // one normalisation group
constexpr int kIssueWarp0 = 4 * NG;      // warps 12..14 issue the MMAs of group 0..2; warp 12 owns the TMEM allocation
constexpr int kProducerWarp0 = kIssueWarp0 + NG;
constexpr int kProducerWarps = 5;        // each owns every fifth tile of the stream
constexpr int kThreads = (kProducerWarp0 + kProducerWarps) * 32;  // 640
constexpr int kTileK = TK * D * 2;       // 8 KB, also the Q tile
constexpr int kVGroup = 512;             // bytes of one 8-row group of a V tile
constexpr int kTileV = (TK / 8) * kVGroup;  // 8 KB
constexpr uint32_t kTmemCols = 512;
constexpr int NB = 2;                    // score / weight buffers per group
constexpr uint32_t kColGroup = 64 * NB + D;  // group b: S_bi (and P_bi over its head) at kColGroup b + 64 i, O_b behind them
static_assert(kColGroup * NG <= kTmemCols, "TMEM columns");
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kHeadroom = 64.0f;       // log2 units a score may exceed the reference maximum
constexpr float kSumLimit = 1180591620717411303424.0f;  // 2^70: a chunk's sum beyond it gives the excess away
constexpr uint32_t kSpinLimit = 1u << 18;  // polls of a wait before the CTA gives up
constexpr uint32_t kSuspendNs = 4000;      // how long one poll may stay suspended in hardware (longer hints wake later)
static_assert(NS > kProducerWarps, "every producer warp holds one stage while it copies");
static_assert(NS % kProducerWarps == 0, "a stage is always filled by the same producer warp, one use after the other");

// dynamic shared memory map
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + NQ * kTileK;
constexpr int kOffV = kOffK + NS * kTileK;
constexpr int kOffX = kOffV + NS * kTileV;          // what the other groups hand to the merging one when a unit ends: [NG - 1][34][128] floats
constexpr int kOffBar = kOffX + (NG - 1) * 34 * 128 * 4;
constexpr int kOffAbort = kOffBar + 448;
constexpr int kSmemBytes = kOffAbort + 32;

// barrier slots (8 bytes each) behind kOffBar
enum {
    BAR_FULL = 0, BAR_EMPTY = NS, BAR_QEMPTY = 2 * NS, BAR_QFULL = 2 * NS + NQ,
    BAR_SFULL = 2 * NS + 2 * NQ,          // [NB b + i]
    BAR_PREADY = BAR_SFULL + NG * NB,     // [NB b + i]
    BAR_PFREE = BAR_PREADY + NG * NB,     // [NB b + i]
    BAR_OFULL = BAR_PFREE + NG * NB,      // [b]
    BAR_XFULL = BAR_OFULL + NG,           // [slot]
    BAR_XEMPTY = BAR_XFULL + NG - 1,      // [slot]
    BAR_DRAIN = BAR_XEMPTY + NG - 1,      // [b]
    BAR_COUNT = BAR_DRAIN + NG
};
static_assert(BAR_COUNT * 8 <= 448, "barrier area");
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");


// error codes OR-ed into the context's device error word: which role gave up (bits 0..3); bits 8..11 carry the
// site code of the first wait that ran out (see SITE_*)
enum { ERR_NORMALISE = 1, ERR_MMA = 2, ERR_DRAIN = 4, ERR_PRODUCER = 8 };

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on a phase parity.  Returns false on time-out or when the CTA is aborting.
// A wait that runs out (rather than being ended by the abort flag) leaves its site code in the word behind the flag;
// the first one stays, and the kernel reports it in bits 8.. of the error word.
enum {
    SITE_SFULL = 1, SITE_OFULL, SITE_XEMPTY, SITE_XFULL, SITE_PFREE, SITE_TILE, SITE_Q, SITE_PREADY, SITE_TAIL_TILE,
    SITE_STAGE, SITE_QBUF, SITE_DRAIN, SITE_QTURN
};
__device__ __forceinline__ void note_site(const volatile int* abort_flag, int site)
{
    atomicCAS(const_cast<int*>(abort_flag) + 1, 0, site);
}
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* abort_flag, int site)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kSuspendNs)
            : "memory");
        if (ok) return true;
        if ((i & 31u) == 31u && *abort_flag) return false;
    }
    note_site(abort_flag, site);
    return false;
}
// The bounded wait with its first poll inline: most waits of the issuing threads find their phase complete.
__device__ __forceinline__ bool mbar_wait_fast(uint32_t bar, uint32_t parity, const volatile int* abort_flag, int site)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0 || mbar_wait(bar, parity, abort_flag, site);
}
// 16-byte copy global -> shared; src_bytes = 0 fills the destination with zeros instead.
// Pool rows go through L1 (with skewed indices the hot rows then stop hammering a few L2 lines
// from every SM at once); rows that are read once bypass it.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async16_once(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}

// Shared-memory matrix descriptor, no swizzle: start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1 of sm_100.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor for kind::f16: fp32 accumulate, bf16 A and B.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// 32 consecutive columns of this thread's TMEM lane.  The load is asynchronous: its registers
// hold the data only after tmem_wait_ld32 on the same array.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
        "%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// Waits for every tcgen05.ld of this thread.  Naming the registers as in/out operands keeps the
// compiler from scheduling their consumers ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld32(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                   "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),
                   "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]),
                   "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :
                 : "memory");
}
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr)
{
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r) : : "memory");
    return r;
}
__device__ __forceinline__ void tmem_st1(uint32_t taddr, uint32_t r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(r) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
        "%30,%31,%32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(
            taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Two fp32 operations in one instruction (packed pairs): the normalisation is short of issue slots, not of FMA lanes.
// (d0, d1) = (a0, a1) * b + c
__device__ __forceinline__ void fma2_scalar(float& d0, float& d1, float a0, float a1, float b, float c)
{
    asm("{\n.reg .b64 ra, rb, rc, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %4};\nmov.b64 rc, {%5, %5};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\nmov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
// (d0, d1) = (a0, a1) * (b0, b1) + (c0, c1)
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1)
{
    asm("{\n.reg .b64 ra, rb, rc, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmov.b64 rc, {%6, %7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\nmov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
// (d0, d1) += (a0, a1)
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1)
{
    asm("{\n.reg .b64 ra, rd;\nmov.b64 rd, {%0, %1};\nmov.b64 ra, {%2, %3};\nadd.rn.f32x2 rd, rd, ra;\n"
        "mov.b64 {%0, %1}, rd;\n}\n"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1));
}
// (d0, d1) = (a0, a1) * b
__device__ __forceinline__ void mul2_scalar(float& d0, float& d1, float a0, float a1, float b)
{
    asm("{\n.reg .b64 ra, rb, rd;\nmov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %4};\nmul.rn.f32x2 rd, ra, rb;\n"
        "mov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b));
}

// byte offset of (row r, 16-byte chunk c) inside a K/Q tile and inside a V tile
__device__ __forceinline__ uint32_t k_off(int r, int c) { return (uint32_t)((r >> 3) * 512 + c * 128 + (r & 7) * 16); }
__device__ __forceinline__ uint32_t v_off(int r, int c) { return (uint32_t)((r >> 3) * kVGroup + c * 128 + (r & 7) * 16); }

// Inside a tile the producers place history position 32 c + 4 q + i (q < 8, i < 4) in row
// 32 c + 8 i + q: a lane then reads the indices of four consecutive positions with one load and
// its four 16-byte copies of an instruction still fall into different shared-memory banks.
// Attention does not depend on the order of positions; only the tail mask has to know which
// position a score column belongs to.
__device__ __forceinline__ int pos_of_col(int c, int e) { return 32 * c + 4 * (e & 7) + (e >> 3); }

// ---- normalisation of one 128 x 64 score half tile by its group (thread = query row = TMEM lane) ----

// Multiplies this thread's row of O (32 columns) by f.
__device__ __noinline__ void rescale_row(uint32_t tO, float f)
{
    uint32_t o[32];
    tmem_ld32(tO, o);
    tmem_wait_ld32(o);
#pragma unroll
    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
    tmem_st32(tO, o);
}

// Multiplies the 32 weights (16 columns of bf16 pairs) this thread wrote for the first chunk of the current half
// tile by f, a power of two: exact unless a weight drops below the smallest bf16.
__device__ __noinline__ void rescale_weights(uint32_t tP, float f)
{
    for (int c = 0; c < 16; ++c) {
        const uint32_t w = tmem_ld1(tP + c);
        tmem_st1(tP + c, pack_bf16(__uint_as_float(w << 16) * f, __uint_as_float(w & 0xffff0000u) * f));
    }
}

// The weights of one 32-column chunk once more (returns their sum), from scores the caller has put into local memory (only used on
// the rare path that moves a row's reference; kept out of line so that it costs the common path nothing).
template <bool TAIL>
__device__ __noinline__ float rewrite_weights(uint32_t tP, const uint32_t* cur, float sc, float nm, int valid, int c)
{
    uint32_t p[16];
    float sum = 0.f;
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        float x0 = fmaf(__uint_as_float(cur[e]), sc, nm), x1 = fmaf(__uint_as_float(cur[e + 1]), sc, nm);
        if (TAIL) {
            if (pos_of_col(c, e) >= valid) x0 = -CUDART_INF_F;
            if (pos_of_col(c, e + 1) >= valid) x1 = -CUDART_INF_F;
        }
        const float e0 = ex2(x0), e1 = ex2(x1);
        sum += e0 + e1;
        p[e >> 1] = pack_bf16(e0, e1);
    }
    tmem_st16(tP, p);
    return sum;
}

// Largest exponent argument of one 32-column chunk (rare path only, like rewrite_weights).
template <bool TAIL>
__device__ __noinline__ float chunk_max(const uint32_t* cur, float sc, float nm, int valid, int c)
{
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int e = 0; e < 32; ++e) {
        const float x = fmaf(__uint_as_float(cur[e]), sc, nm);
        if (!TAIL || pos_of_col(c, e) < valid) mx = fmaxf(mx, x);
    }
    return mx;
}

// Softmax weights of one 32-column chunk (c = 0, 1) of a 128 x 64 score half tile: p = exp2(s c - m) as bf16
// pairs written over the head of the scores (columns 0..31 of the buffer; chunk 1 of the scores, columns 32..63,
// is still to be read when chunk 0's weights land on columns 0..15, and chunk 1's weights
// land on columns 16..31, whose scores have been consumed).  The chunk's weights are added to the row sum l.  With `first` (chunk 0 of the group's first half
// tile of a unit) the row's reference m is set from these 32 scores (column 0 is the half's position 0, always a
// real one).  A chunk whose largest exponent argument leaves the headroom moves the reference up by a whole
// number of octaves and is written again from the scores still in the registers; what O_b holds so far
// (`have_o`; wait_prev() waits for the previous step's MMAs) and, for chunk 1, the weights of chunk 0 are
// multiplied by the same power of two.  Returns false if that wait ran out.
// `valid` counts the real positions of the half (1..64); column (c, e) of the half holds position
// pos_of_col(c, e) of the half.  TAIL = true (end of a history, at most once per unit and group) masks the
// columns beyond.
// VIS (visible lengths): `valid` differs from thread to thread and may be zero or negative (the row sees nothing
// of this half tile); a row's reference is then set by the first chunk in which it sees a position.
template <bool TAIL, bool VIS, typename WaitPrev>
__device__ __forceinline__ bool softmax_chunk(const uint32_t (&cur)[32], int c, uint32_t tS, uint32_t tO, float sc,
                                              int valid, bool first, bool have_o, float& m_ref, float& l, WaitPrev&& wait_prev)
{
    if ((c == 0 && first) || (VIS && m_ref == -CUDART_INF_F)) {
        float t0 = -CUDART_INF_F, t1 = -CUDART_INF_F;
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
            float x[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                x[i] = (TAIL && pos_of_col(c, e + i) >= valid) ? -CUDART_INF_F : __uint_as_float(cur[e + i]);
            t0 = max3(t0, x[0], x[1]);
            t1 = max3(t1, x[2], x[3]);
        }
        m_ref = fmaxf(t0, t1) * sc;
    }
    float nm = -m_ref;
    float ls0 = 0.f, ls1 = 0.f;  // this chunk's share of the row sum
    uint32_t p[16];
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        float x0, x1;
        fma2_scalar(x0, x1, __uint_as_float(cur[e]), __uint_as_float(cur[e + 1]), sc, nm);
        if (TAIL) {
            if (pos_of_col(c, e) >= valid) x0 = -CUDART_INF_F;
            if (pos_of_col(c, e + 1) >= valid) x1 = -CUDART_INF_F;
        }
        const float e0 = ex2(x0), e1 = ex2(x1);
        add2(ls0, ls1, e0, e1);
        p[e >> 1] = pack_bf16(e0, e1);
    }
    // Leaving the headroom shows in the chunk's sum: 32 weights of at most 2^64 add up to at most 2^69, so a sum
    // beyond kSumLimit = 2^70 (or one that is not a number) means some weight of this row is beyond 2^65.  That
    // costs one comparison here instead of a running maximum over the arguments.
    if (!__any_sync(0xffffffffu, !(ls0 + ls1 <= kSumLimit))) {
        tmem_st16(tS + 16 * c, p);
    } else {
        // rare: some row of this warp left the headroom and its weights may have overflowed.  Nothing of this
        // chunk has been written yet, so its scores are still in TMEM: move the reference, bring what was
        // accumulated and written before into the new scale, and work the chunk out again from there.
        uint32_t again[32];
        tmem_ld32(tS + 32 * c, again);
        tmem_wait_ld32(again);
        const float mx = chunk_max<TAIL>(again, sc, nm, valid, c);
        const float shift = mx > kHeadroom ? ceilf(mx) : 0.f;
        const float f = ex2(-shift);
        m_ref += shift;
        nm = -m_ref;
        tc_wait_st();
        l *= f;
        if (have_o) {
            if (!wait_prev()) return false;
            tc_fence_after();
            rescale_row(tO, f);
        }
        if (c == 1) rescale_weights(tS, f);
        ls0 = rewrite_weights<TAIL>(tS + 16 * c, again, sc, nm, valid, c);
        ls1 = 0.f;
        tc_wait_st();
    }
    l += ls0 + ls1;
    return true;
}

// p = silu(x) = x sigmoid(x) = h (1 + tanh(h)), h = x / 2, as bf16 pairs over the head of the scores like the
// softmax weights   (sc = scale / 2)
template <bool TAIL>
__device__ __forceinline__ void silu_chunk(const uint32_t (&cur)[32], int c, uint32_t tS, float sc, int valid)
{
    uint32_t p[16];
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        float h0, h1, w0, w1;
        mul2_scalar(h0, h1, __uint_as_float(cur[e]), __uint_as_float(cur[e + 1]), sc);
        fma2(w0, w1, h0, h1, tanh_fast(h0), tanh_fast(h1), h0, h1);
        if (TAIL) {
            if (pos_of_col(c, e) >= valid) w0 = 0.f;
            if (pos_of_col(c, e + 1) >= valid) w1 = 0.f;
        }
        p[e >> 1] = pack_bf16(w0, w1);
    }
    tmem_st16(tS + 16 * c, p);
}

// The user-specific leading elements of one row (DUB = 2 d_user bytes), as the producers carry
// them from the compressed cache to a shared-memory tile.
template <int DUB> struct UserPart;
template <> struct UserPart<0> {};
template <> struct UserPart<2> {
    uint16_t v;
    __device__ __forceinline__ void load(const char* p) { v = __ldg(reinterpret_cast<const uint16_t*>(p)); }
    __device__ __forceinline__ void store(unsigned char* p) const { *reinterpret_cast<uint16_t*>(p) = v; }
};
template <> struct UserPart<4> {
    uint32_t v;
    __device__ __forceinline__ void load(const char* p) { v = __ldg(reinterpret_cast<const uint32_t*>(p)); }
    __device__ __forceinline__ void store(unsigned char* p) const { *reinterpret_cast<uint32_t*>(p) = v; }
};
template <> struct UserPart<8> {
    uint2 v;
    __device__ __forceinline__ void load(const char* p) { v = __ldg(reinterpret_cast<const uint2*>(p)); }
    __device__ __forceinline__ void store(unsigned char* p) const { *reinterpret_cast<uint2*>(p) = v; }
};
template <> struct UserPart<16> {
    uint4 v;
    __device__ __forceinline__ void load(const char* p) { v = __ldg(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ void store(unsigned char* p) const { *reinterpret_cast<uint4*>(p) = v; }
};

// One work unit of the CTA's share, decoded from its Work record.
struct Unit {
    Work wk;
    int grp;
    int row0;        // first query row of the block
    int n_tiles;     // > 0: tiles to process; 0: empty history (zero output rows); < 0: nothing at all
    int last_valid;  // real positions in the last tile
};

// Which group takes a unit's first half (half p goes to group (p + rotation) mod NG).  A function of the unit
// alone -- not of its place in a CTA's stream -- so that results do not depend on what else a call processes.
__device__ __forceinline__ int unit_rotation(const Unit& u)
{
    return (int)((uint32_t)(u.grp + (u.row0 >> 7) + (u.wk.begin >> 6)) % (uint32_t)NG);
}

__device__ __forceinline__ Work load_work(const Work* p)
{
    static_assert(sizeof(Work) == 48, "Work is read as three 16-byte words");
    union {
        Work w;
        uint4 q[3];
    } u;
    const uint4* src = reinterpret_cast<const uint4*>(p);
    u.q[0] = __ldg(src);
    u.q[1] = __ldg(src + 1);
    u.q[2] = __ldg(src + 2);
    return u.w;
}

// The CTA's tile stream: units blockIdx.x, blockIdx.x + gridDim.x, ... tile by tile.  Every role
// walks an identical copy, so stage and buffer indices need no communication.  The record of
// the following unit is always in flight while the current one is processed.  Unit w stands for
// (item, group, query block) = (w / n_mb / G, w / n_mb % G, w % n_mb); the coordinates are
// stepped with carries instead of divided out each time.
// KEEP_EMPTY: also stop at units with an empty history (the role that writes their zero rows).
template <bool KEEP_EMPTY, bool VIS>
struct Stream {
    const Work* works;
    const int32_t* vmax;         // VIS: per (request, query block) the largest visible length of its rows
    uint32_t n_mb, n_groups;
    uint32_t w, n_work;          // the host keeps n_work + gridDim.x below 2^32
    uint32_t item, grp, mb;      // coordinates of unit w
    uint32_t d_item, d_grp, d_mb;  // gridDim.x in the same mixed radix
    Unit u;
    Work nxt;    // record of unit w + gridDim.x (valid if that is < n_work)
    int j;       // tile inside the unit
    int g;       // tiles before this one in the stream
    int useq;    // units with tiles before this one
    bool valid;
    __device__ __forceinline__ void step(uint32_t& it, uint32_t& gr, uint32_t& m) const
    {
        m += d_mb;
        gr += d_grp;
        it += d_item;
        if (m >= n_mb) {
            m -= n_mb;
            ++gr;
        }
        if (gr >= n_groups) {
            gr -= n_groups;
            ++it;
        }
    }
    __device__ __forceinline__ void take()
    {
        valid = false;
        while (w < n_work) {
            u.wk = nxt;
            u.grp = (int)grp;
            u.row0 = (int)mb * 128;
            const uint32_t wn = w + gridDim.x;
            uint32_t ni = item, ng = grp, nm = mb;
            step(ni, ng, nm);
            if (wn < n_work) nxt = load_work(works + ni);
            // with visible lengths nothing behind the block's largest limit is touched (every role decodes the same)
            int len = u.wk.len;
            if constexpr (VIS) {
                if (u.row0 < u.wk.M) len = min(len, max(__ldg(vmax + u.wk.pad[0] + mb) - u.wk.begin, 0));
            }
            u.n_tiles = u.row0 < u.wk.M ? (len + TK - 1) / TK : -1;
            u.last_valid = len - (u.n_tiles - 1) * TK;
            if (u.n_tiles > 0 || (KEEP_EMPTY && u.n_tiles == 0)) {
                valid = true;
                j = 0;
                return;
            }
            w = wn;
            item = ni;
            grp = ng;
            mb = nm;
        }
    }
    __device__ __forceinline__ void to_next_unit()
    {
        w += gridDim.x;
        step(item, grp, mb);
        take();
    }
    __device__ __forceinline__ void init(const AttendArgs& a, int n_mb_, int64_t n_work_)
    {
        works = a.works;
        if constexpr (VIS) vmax = a.vmax;
        n_mb = (uint32_t)n_mb_;
        n_groups = (uint32_t)a.cv.n_groups;
        n_work = (uint32_t)n_work_;
        w = blockIdx.x;
        mb = w % n_mb;
        grp = (w / n_mb) % n_groups;
        item = (w / n_mb) / n_groups;
        d_mb = gridDim.x % n_mb;
        d_grp = (gridDim.x / n_mb) % n_groups;
        d_item = (gridDim.x / n_mb) / n_groups;
        g = 0;
        useq = 0;
        if (w < n_work) nxt = load_work(works + item);
        take();
    }
    __device__ __forceinline__ void next_unit()
    {
        g += u.n_tiles > 0 ? u.n_tiles : 0;
        useq += u.n_tiles > 0;
        to_next_unit();
    }
    __device__ __forceinline__ void advance()
    {
        ++g;
        if (++j == u.n_tiles) {
            ++useq;
            to_next_unit();
        }
    }
    // n tiles on
    __device__ __forceinline__ void advance_by(int n)
    {
        g += n;
        j += n;
        while (valid && j >= u.n_tiles) {
            const int over = j - u.n_tiles;
            ++useq;
            to_next_unit();  // sets j = 0
            j = over;
        }
    }
};

// VIS: visible lengths (a.vis, a.vmax); the plain instantiations carry none of that code.
template <int MODE, int DUB, bool VIS>
__global__ void __launch_bounds__(kThreads, 1) attend_umma_kernel(const AttendArgs a, int n_mb, int64_t n_work, int* err_flag)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint32_t tmem_base_slot;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffAbort);
    const int G = a.cv.n_groups;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar(BAR_FULL + s), 1);   // lane 0 of the producer warp that owns the tile
            mbar_init(bar(BAR_EMPTY + s), 2);  // one arrival per half
        }
        for (int q = 0; q < NQ; ++q) {
            mbar_init(bar(BAR_QEMPTY + q), NG);  // every issuer
            mbar_init(bar(BAR_QFULL + q), 1);    // lane 0 of the producer warp that staged the unit's Q block
        }
        for (int bi = 0; bi < NG * NB; ++bi) {
            mbar_init(bar(BAR_SFULL + bi), 1);
            mbar_init(bar(BAR_PREADY + bi), kGroupThreads);
            mbar_init(bar(BAR_PFREE + bi), 1);
        }
        for (int b = 0; b < NG; ++b) {
            mbar_init(bar(BAR_OFULL + b), 1);
            mbar_init(bar(BAR_DRAIN + b), 1);
        }
        for (int b = 0; b < NG - 1; ++b) {
            mbar_init(bar(BAR_XFULL + b), kGroupThreads);
            mbar_init(bar(BAR_XEMPTY + b), kGroupThreads);
        }
        abort_flag[0] = 0;  // raised by the first role that gives up
        abort_flag[1] = 0;  // site of the first wait that ran out
        abort_flag[4] = 0;  // units whose Q block has a producer at work on it (see the producers)
        abort_flag[2] = 0;  // never raised: the flag of the teardown wait, which must not be cut short
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kIssueWarp0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;

    if (warp < kIssueWarp0) {
        // --------------------------------------------------------------- normalisation groups
        const int b = warp >> 2;                    // group
        const int row = tid & (kGroupThreads - 1);  // query row inside the block = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS0 = tmem + lane_base + kColGroup * b, tO = tS0 + 64u * NB;
        const float sc = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 0.5f);
        float* xch = reinterpret_cast<float*>(smem + kOffX);
        int cnt = 0;    // halves this group has normalised
        int ocnt = 0;   // units in which this group had halves
        int xcnt = 0;   // units exchanged between the groups
        bool ok = true;
        uint32_t sa[32];  // one 32-column chunk of a half's scores
        Stream<true, VIS> sn;
        sn.init(a, n_mb, n_work);
        for (; sn.valid && ok; sn.next_unit()) {
            const Unit& u = sn.u;
            const int r = u.row0 + row;
            if (r < u.wk.M) (void)CKV_CLAMP((int64_t)(u.wk.q0 + r), a.q_rows, err_flag);
            const int64_t out_base = ((int64_t)(u.wk.q0 + r) * G + u.grp) * D;
            if (u.n_tiles == 0) {  // empty history, or a chunk behind every row's visible length: zero rows
                if (b == 0 && r < u.wk.M) {
                    if (u.wk.part_row >= 0) {  // (only with visible lengths) an empty partial result
                        float* pr = a.partials + (CKV_CLAMP((int64_t)(u.wk.part_row + r), a.part_rows, err_flag) * G + u.grp) * (D + 2);
                        pr[0] = -CUDART_INF_F;
                        for (int e = 1; e < D + 2; ++e) pr[e] = 0.f;
                    } else if (a.out_dtype == CKV_BF16) {
                        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(a.out) + out_base);
                        for (int q4 = 0; q4 < 4; ++q4) dst[q4] = make_uint4(0, 0, 0, 0);
                    } else {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + out_base);
                        for (int q4 = 0; q4 < 8; ++q4) dst[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                continue;
            }
            // positions this thread's query row attends: [0, lim); rows beyond the user's queries take none
            int lim = u.wk.L;
            if constexpr (VIS) lim = r < u.wk.M ? min(max(__ldg(a.vis + u.wk.q0 + r), 0), u.wk.L) : 0;
            float m_ref = -CUDART_INF_F, l = 0.f;
            int mine = 0;  // halves of this unit normalised by this group
            // The unit's non-empty halves are p = 2 j + half < n_half (only the second half of the last tile can be
            // empty); half p goes to group (p + unit_rotation) mod NG.
            const int n_half = 2 * u.n_tiles - (u.last_valid <= TH ? 1 : 0);
            for (int p = (b + NG - unit_rotation(u)) % NG; p < n_half && ok; p += NG) {
                const int j = p >> 1, half = p & 1;
                const int valid = (j == u.n_tiles - 1 ? u.last_valid : TK) - TH * half;  // real positions of the half
                const int i = cnt % NB;                                                   // buffer of this step
                const uint32_t tS = tS0 + 64u * i;
                ok = mbar_wait_fast(bar(BAR_SFULL + NB * b + i), (cnt / NB) & 1, abort_flag, SITE_SFULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                // (softmax, only taken when a row leaves the headroom) the previous step's MMAs must have finished
                // before O_b is rescaled
                auto wait_prev = [&]() {
                    bool w = mbar_wait(bar(BAR_PFREE + NB * b + (cnt - 1) % NB), ((cnt - 1) / NB) & 1, abort_flag, SITE_PFREE);
                    return __all_sync(0xffffffffu, w);
                };
                // real (and, with visible lengths, attended) positions of this thread's row in the half
                int valid_r = valid;
                bool tail = valid < TH;
                if constexpr (VIS) {
                    valid_r = min(valid, lim - (u.wk.begin + j * TK + TH * half));
                    tail = __any_sync(0xffffffffu, valid_r < TH);
                }
                // One 32-column chunk at a time: the other groups' warps on this sub-partition cover the TMEM load.
                if (tail) {  // end of a history or of some row's visible positions: masked columns
#pragma unroll 1
                    for (int c = 0; c < 2 && ok; ++c) {
                        tmem_ld32(tS + 32 * c, sa);
                        tmem_wait_ld32(sa);
                        if constexpr (MODE == CKV_SOFTMAX)
                            ok = softmax_chunk<true, VIS>(sa, c, tS, tO, sc, valid_r, mine == 0, mine > 0, m_ref, l, wait_prev);
                        else
                            silu_chunk<true>(sa, c, tS, sc, valid_r);
                    }
                } else {
#pragma unroll 1
                    for (int c = 0; c < 2 && ok; ++c) {
                        tmem_ld32(tS + 32 * c, sa);
                        tmem_wait_ld32(sa);
                        if constexpr (MODE == CKV_SOFTMAX)
                            ok = softmax_chunk<false, VIS>(sa, c, tS, tO, sc, valid, mine == 0, mine > 0, m_ref, l, wait_prev);
                        else
                            silu_chunk<false>(sa, c, tS, sc, valid);
                    }
                }
                if (!ok) break;
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(BAR_PREADY + NB * b + i));
                ++cnt;
                ++mine;
            }
            if (!ok) break;

            // ---- the unit's epilogue: fetch O_b, merge the groups, store
            float o[32];
            if (mine > 0) {
                ok = mbar_wait(bar(BAR_OFULL + b), ocnt & 1, abort_flag, SITE_OFULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ++ocnt;
                tc_fence_after();
                uint32_t raw[32];
                tmem_ld32(tO, raw);
                tmem_wait_ld32(raw);
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __uint_as_float(raw[e]);
                tc_fence_before();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = 0.f;
            }
            // Group 0 merges and stores, always: a barrier of the hand-over is then waited on by the same threads use
            // after use.  (With the merging passed round -- to the group that has the unit's last half -- a group
            // could come to wait for a use while the one before was still open, and a parity wait cannot tell.)
            if (b != 0) {
                const int slot = b - 1;
                float* x = xch + slot * 34 * 128;
                if (xcnt > 0) ok = mbar_wait(bar(BAR_XEMPTY + slot), (xcnt - 1) & 1, abort_flag, SITE_XEMPTY);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                x[row] = m_ref;
                x[128 + row] = l;
#pragma unroll
                for (int e = 0; e < 32; ++e) x[(2 + e) * 128 + row] = o[e];
                mbar_arrive(bar(BAR_XFULL + slot));
                ++xcnt;
            } else {
#pragma unroll 1
                for (int slot = 0; slot < NG - 1 && ok; ++slot) {
                    const float* x = xch + slot * 34 * 128;
                    ok = mbar_wait(bar(BAR_XFULL + slot), xcnt & 1, abort_flag, SITE_XFULL);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const float m1 = x[row], l1 = x[128 + row];
                    if constexpr (MODE == CKV_SOFTMAX) {
                        const float mt = fmaxf(m_ref, m1);
                        const float ms = mt == -CUDART_INF_F ? 0.f : mt;
                        const float c0 = ex2(m_ref - ms), c1 = ex2(m1 - ms);
                        l = l * c0 + l1 * c1;
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = o[e] * c0 + x[(2 + e) * 128 + row] * c1;
                        m_ref = mt;
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] += x[(2 + e) * 128 + row];
                    }
                    mbar_arrive(bar(BAR_XEMPTY + slot));
                }
                if (!ok) break;
                ++xcnt;
                if (r < u.wk.M) {
                    if (u.wk.part_row < 0) {
                        float inv;
                        if constexpr (MODE == CKV_SOFTMAX) inv = l > 0.f ? 1.0f / l : 0.f;
                        else inv = 1.0f / (float)u.wk.L;
                        if (a.out_dtype == CKV_BF16) {
                            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(a.out) + out_base);
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                uint4 v;
                                v.x = pack_bf16(o[8 * q4 + 0] * inv, o[8 * q4 + 1] * inv);
                                v.y = pack_bf16(o[8 * q4 + 2] * inv, o[8 * q4 + 3] * inv);
                                v.z = pack_bf16(o[8 * q4 + 4] * inv, o[8 * q4 + 5] * inv);
                                v.w = pack_bf16(o[8 * q4 + 6] * inv, o[8 * q4 + 7] * inv);
                                dst[q4] = v;
                            }
                        } else {
                            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + out_base);
#pragma unroll
                            for (int q4 = 0; q4 < 8; ++q4)
                                dst[q4] = make_float4(o[4 * q4] * inv, o[4 * q4 + 1] * inv, o[4 * q4 + 2] * inv,
                                                      o[4 * q4 + 3] * inv);
                        }
                    } else {
                        float* pr = a.partials + (CKV_CLAMP((int64_t)(u.wk.part_row + r), a.part_rows, err_flag) * G + u.grp) * (D + 2);
                        pr[0] = m_ref;
                        pr[1] = l;
#pragma unroll
                        for (int e = 0; e < 32; ++e) pr[2 + e] = o[e];
                    }
                }
            }
        }
        tc_wait_ld();
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(err_flag, ERR_NORMALISE);
        }
    } else if (warp < kProducerWarp0) {
        // --------------------------------------------------------------------- MMA issue for one group
        // One thread per group, and its loop is the pipeline's pacemaker: it is a chain of dependent instructions
        // of a single thread, so everything that can be kept out of it is (descriptors are a constant plus an
        // offset, the two pending weighted sums live in named registers, waits poll once inline before they call).
        if (lane == 0) {
            const int b = warp - kIssueWarp0;
            constexpr uint32_t idesc_s = make_idesc(128, TH, false), idesc_pv = make_idesc(128, D, true);
            const uint32_t tS0 = tmem + kColGroup * b, tO = tS0 + 64u * NB;
            const uint64_t dq0 = smem_desc(sbase + kOffQ, 128, 512), dk0 = smem_desc(sbase + kOffK, 128, 512),
                           dv0 = smem_desc(sbase + kOffV, kVGroup, 128);
            auto at = [](uint64_t d, uint32_t byte_off) { return d + (uint64_t)(byte_off >> 4); };  // no carry out of the address field
            static_assert(NB == 2, "two pending weighted sums");
            Stream<false, VIS> ss;
            ss.init(a, n_mb, n_work);
            int cnt = 0;   // steps whose scores have been issued
            int done = 0;  // steps whose weighted sum has been issued
            // what the weighted sums of the (at most two) steps in flight need, oldest first: byte offset of the half V
            // tile, stage to release, flags (bit 0: O_b already holds the unit's earlier halves; bit 1: the group's
            // last half of the unit)
            uint32_t pv_off0 = 0, pv_off1 = 0;
            int pv_s0 = 0, pv_s1 = 0, pv_f0 = 0, pv_f1 = 0;
            int gs = 0, gp = 0;  // stage and phase parity of the unit's first tile: g % NS, (g / NS) & 1
            bool ok = true;
            // O_b += P_bi V_half for step `done`, whose group has written P_bi
            auto do_pv = [&]() {
                const int i = done & 1;
                tc_fence_after();
                const uint64_t dv = at(dv0, pv_off0);
#pragma unroll
                for (int kk = 0; kk < TH / 16; ++kk)  // sixteen positions per instruction
                    umma_ts(tO, tS0 + 64u * i + 8 * kk, at(dv, kk * 2 * kVGroup), idesc_pv, ((pv_f0 & 1) || kk > 0) ? 1u : 0u);
                tc_commit(bar(BAR_EMPTY + pv_s0));
                tc_commit(bar(BAR_PFREE + NB * b + i));
                if (pv_f0 & 2) tc_commit(bar(BAR_OFULL + b));
                pv_off0 = pv_off1;
                pv_s0 = pv_s1;
                pv_f0 = pv_f1;
                ++done;
            };
            // ... waiting for the weights first (used where the thread can do nothing else)
            auto issue_pv = [&]() {
                if (!mbar_wait_fast(bar(BAR_PREADY + NB * b + (done & 1)), (done >> 1) & 1, abort_flag, SITE_PREADY)) return false;
                do_pv();
                return true;
            };
            for (; ok && ss.valid; ss.next_unit()) {
                const Unit& u = ss.u;
                const int n_half = 2 * u.n_tiles - (u.last_valid <= TH ? 1 : 0);
                const int rot = unit_rotation(u);
                const uint32_t q_off = (uint32_t)(ss.useq % NQ) * kTileK;
                bool q_seen = false;  // this thread has seen the unit's Q block staged
                for (int p = (b + NG - rot) % NG; p < n_half; p += NG) {
                    const int t = gs + (p >> 1), half = p & 1;
                    const int s = t % NS, par = gp ^ ((t / NS) & 1);
                    // buffer i still holds the weights of step cnt - NB: its weighted sum goes first (and before the
                    // wait for the tile: at a unit's end the group is waiting for exactly this weighted sum).  The tensor
                    // core runs this thread's instructions in order, so the scores below need not wait for it to finish.
                    if (ok && cnt - done == NB) ok = issue_pv();
                    if (ok) ok = mbar_wait_fast(bar(BAR_FULL + s), par, abort_flag, SITE_TILE);
                    if (ok && !q_seen) {  // first scores of a unit: its Q block must have landed
                        ok = mbar_wait_fast(bar(BAR_QFULL + ss.useq % NQ), (ss.useq / NQ) & 1, abort_flag, SITE_Q);
                        q_seen = true;
                    }
                    if (!ok) break;
                    tc_fence_after();
                    const int i = cnt & 1;
                    const uint64_t dq = at(dq0, q_off), dk = at(dk0, (uint32_t)s * kTileK + half * (TH / 8) * 512);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        umma_ss(tS0 + 64u * i, at(dq, ks * 256), at(dk, ks * 256), idesc_s, ks > 0 ? 1u : 0u);
                    tc_commit(bar(BAR_SFULL + NB * b + i));
                    const uint32_t off = (uint32_t)s * kTileV + half * (TH / 8) * kVGroup;
                    const int f = (p >= NG ? 1 : 0) | (p + NG >= n_half ? 2 : 0);
                    if (cnt == done) {
                        pv_off0 = off;
                        pv_s0 = s;
                        pv_f0 = f;
                    } else {
                        pv_off1 = off;
                        pv_s1 = s;
                        pv_f1 = f;
                    }
                    ++cnt;
                }
                if (!ok) break;
                const int t_last = gs + u.n_tiles - 1;
                const bool empty_tail = u.last_valid <= TH && (2 * u.n_tiles - 1 + rot) % NG == b;
                // A weighted sum is normally issued when its buffer is wanted for the scores two steps on.  In a run of
                // short units whose halves go to the other groups that could be many units on -- while the other groups
                // wait, at the end of the unit it belongs to, for this group's accumulator, the issuing threads behind
                // them stop releasing Q blocks and stages, and the tile or Q block this thread is waiting for never comes.
                // So where this thread passes a unit in which it issued nothing (or has only the empty tail to release),
                // whatever it still holds is issued first; waiting for the weights there cannot block on anything this
                // thread does later.  Units in which the group has halves keep their lead of two steps.
                if (!q_seen || empty_tail)
                    while (ok && done < cnt) ok = issue_pv();
                if (!ok) break;
                if (empty_tail) {
                    // the empty second half of the unit's last tile is this group's: nothing to compute, but the
                    // stage needs this half's release
                    ok = mbar_wait_fast(bar(BAR_FULL + t_last % NS), gp ^ ((t_last / NS) & 1), abort_flag, SITE_TAIL_TILE);
                    if (!ok) break;
                    mbar_arrive(bar(BAR_EMPTY + t_last % NS));
                }
                // This issuer no longer reads the unit's Q buffer.  It observes every staging of a buffer,
                // whether it has halves in the unit or not: the buffer is staged again only after all
                // issuers have released it, so no issuer can run a use ahead of another on these barriers.
                if (!q_seen) ok = mbar_wait_fast(bar(BAR_QFULL + ss.useq % NQ), (ss.useq / NQ) & 1, abort_flag, SITE_Q);
                if (!ok) break;
                tc_commit(bar(BAR_QEMPTY + ss.useq % NQ));
                gp ^= ((t_last + 1) / NS) & 1;
                gs = (t_last + 1) % NS;
            }
            while (ok && done < cnt) ok = issue_pv();
            if (!ok) {
                *abort_flag = 1;
                atomicOr(err_flag, ERR_MMA);
            }
            // nothing of this CTA may still be running on the tensor core at teardown
            tc_commit(bar(BAR_DRAIN + b));
            if (!mbar_wait(bar(BAR_DRAIN + b), 0, abort_flag + 2, SITE_DRAIN)) atomicOr(err_flag, ERR_DRAIN);
        }
        __syncwarp();
    } else {
        // --------------------------------------------------------------------- producers
        // Producer warp pw owns every kProducerWarps-th tile of the stream and does all of its
        // copies, so the per-tile bookkeeping is paid by one warp while the others work on their own
        // tiles.  Lane (q = lane / 4, chunk = lane % 4) copies chunk `chunk` of the pool rows of
        // positions 32 rb + 4 q + i (rb, i < 4) into tile rows 32 rb + 8 i + q, and patches the
        // user-specific leading elements of tile rows 32 rb + lane.  A producer is one warp running a chain of
        // dependent instructions per tile: five of them keep the stage ring ahead of three groups only because a
        // tile's 32 copies per lane are issued back to back, with nothing that waits between them.
        const int pw = warp - kProducerWarp0, q = lane >> 2, chunk = lane & 3;
        const int patch_pos = 4 * (lane & 7) + (lane >> 3);  // position (inside a 32-block) held by row `lane`
        const uint32_t kv_lane = (uint32_t)(chunk * 128 + q * 16);
        const int64_t pool_stride = (int64_t)a.cv.n_entries * (D * 2);
        const char* poolK0 = reinterpret_cast<const char*>(a.cv.poolK) + chunk * 16;
        const char* poolV0 = reinterpret_cast<const char*>(a.cv.poolV) + chunk * 16;
        const uint16_t* Q = reinterpret_cast<const uint16_t*>(a.queries);
        // A side that is not shared (sharing only keys or only values): its rows are the tile's own units in the
        // arena, the position inside the tile stands in for the pool index, and nothing is patched.
        const bool full_k = a.cv.full_k != 0, full_v = a.cv.full_v != 0;
        const char* rowsK0 = reinterpret_cast<const char*>(a.cv.userK) + chunk * 16;
        const char* rowsV0 = reinterpret_cast<const char*>(a.cv.userV) + chunk * 16;
        Stream<false, VIS> st;
        st.init(a, n_mb, n_work);
        for (int i = 0; i < pw && st.valid; ++i) st.advance();
        bool ok = true;
        // Everything a tile needs from the compressed cache is requested one tile of this warp ahead:
        uint2 xk, xv;                     // pool rows of positions 4 lane .. 4 lane + 3
        UserPart<DUB> uk_n[4], uv_n[4];   // user-specific leading elements (Eq. K: dims [0, d_user)) of tile rows 32 rb + lane
        auto fetch = [&]() {
            if (!st.valid) return;
            const int pos0 = st.u.wk.begin + st.j * TK;
            const int64_t unit0 = st.u.wk.base + (int64_t)st.u.grp * st.u.wk.Lpad + pos0;  // arena unit of the tile's position 0
            (void)CKV_CLAMP(unit0, a.arena_units, err_flag);
            const int valid = st.j == st.u.n_tiles - 1 ? st.u.last_valid : TK;
            xk = xv = make_uint2(0, 0);
            if (pos0 + 4 * lane < st.u.wk.Lpad) {  // the arena is padded to 32 positions per user
                if (!full_k) xk = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(a.cv.idxK) + unit0 + 4 * lane));
                if (!full_v) xv = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(a.cv.idxV) + unit0 + 4 * lane));
            }
            if (full_k) xk = make_uint2((4 * lane) | ((4 * lane + 1) << 16), (4 * lane + 2) | ((4 * lane + 3) << 16));
            if (full_v) xv = make_uint2((4 * lane) | ((4 * lane + 1) << 16), (4 * lane + 2) | ((4 * lane + 3) << 16));
            if constexpr (DUB > 0) {
#pragma unroll
                for (int rb = 0; rb < 4; ++rb) {
                    if (32 * rb + patch_pos < valid) {
                        if (!full_k) uk_n[rb].load(reinterpret_cast<const char*>(a.cv.userK) + (unit0 + 32 * rb + patch_pos) * DUB);
                        if (!full_v) uv_n[rb].load(reinterpret_cast<const char*>(a.cv.userV) + (unit0 + 32 * rb + patch_pos) * DUB);
                    }
                }
            }
        };
        fetch();
        while (st.valid && ok) {
            const int s = st.g % NS;
            UserPart<DUB> uk[4], uv[4];
#pragma unroll
            for (int rb = 0; rb < 4; ++rb) {
                uk[rb] = uk_n[rb];
                uv[rb] = uv_n[rb];
            }
            const uint2 xk_cur = xk, xv_cur = xv;  // this tile's indices (fetch() below refills xk, xv for the next)
            if (st.g >= NS) {
                if (lane == 0) ok = mbar_wait(bar(BAR_EMPTY + s), ((st.g / NS) - 1) & 1, abort_flag, SITE_STAGE);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (!ok) break;
            const int q_slot = st.j == 0 ? st.useq % NQ : -1;
            if (st.j == 0) {  // a new unit: stage its Q block (rows beyond M are zero)
                // Q blocks are taken up in unit order.  A parity wait cannot tell "this buffer's previous use has been
                // released" from "not even the use before that has": with short units the producers work on five
                // consecutive units at once, so the warp staging unit u could otherwise overtake the one still
                // waiting to stage unit u - NQ.
                if (lane == 0) {
                    ok = false;
                    for (uint32_t it = 0; it < (kSpinLimit << 3); ++it) {
                        if (abort_flag[4] == st.useq) {
                            ok = true;
                            break;
                        }
                        if ((it & 63u) == 63u && *abort_flag) break;
                        __nanosleep(64);
                    }
                    if (!ok && !*abort_flag) note_site(abort_flag, SITE_QTURN);
                    if (ok && st.useq >= NQ)
                        ok = mbar_wait(bar(BAR_QEMPTY + st.useq % NQ), ((st.useq / NQ) - 1) & 1, abort_flag, SITE_QBUF);
                    if (ok) abort_flag[4] = st.useq + 1;
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t qdst = sbase + kOffQ + (st.useq % NQ) * kTileK + kv_lane;
                const int rows_in = st.u.wk.M - st.u.row0;
                const uint16_t* qsrc = Q + ((int64_t)(st.u.wk.q0 + st.u.row0 + q) * G + st.u.grp) * D + chunk * 8;
#pragma unroll 2
                for (int rr = 0; rr < 16; ++rr) {  // rows 8 rr + q
                    const bool in = 8 * rr + q < rows_in;
                    cp_async16_once(qdst + 512 * rr, in ? qsrc + (int64_t)8 * rr * G * D : Q, in ? 16u : 0u);
                }
            }
            const int64_t tile_unit0 = st.u.wk.base + (int64_t)st.u.grp * st.u.wk.Lpad + st.u.wk.begin + st.j * TK;
            const char* pk = full_k ? rowsK0 + tile_unit0 * (D * 2) : poolK0 + st.u.grp * pool_stride;
            const char* pv = full_v ? rowsV0 + tile_unit0 * (D * 2) : poolV0 + st.u.grp * pool_stride;
            const uint32_t kdst = sbase + kOffK + s * kTileK + kv_lane, vdst = sbase + kOffV + s * kTileV + kv_lane;
            const int valid = st.j == st.u.n_tiles - 1 ? st.u.last_valid : TK;
            // The indices of positions 32 rb + 4 q .. + 3 are with lane 8 rb + q (it fetched them as one 8-byte
            // word per side); all sixteen of a side come over by shuffles before the first copy is issued, so that
            // the copies are not strung out between dependent loads.
            uint32_t ik[8], iv[8];
#pragma unroll
            for (int rb = 0; rb < 4; ++rb) {
                ik[2 * rb] = __shfl_sync(0xffffffffu, xk_cur.x, 8 * rb + q);
                ik[2 * rb + 1] = __shfl_sync(0xffffffffu, xk_cur.y, 8 * rb + q);
                iv[2 * rb] = __shfl_sync(0xffffffffu, xv_cur.x, 8 * rb + q);
                iv[2 * rb + 1] = __shfl_sync(0xffffffffu, xv_cur.y, 8 * rb + q);
            }
#pragma unroll
            for (int it = 0; it < 16; ++it) {  // rb = it / 4, i = it % 4: position 32 rb + 4 q + i -> tile row 32 rb + 8 i + q
                const int pos = 32 * (it >> 2) + 4 * q + (it & 3);
                const uint32_t nb = pos < valid ? 16u : 0u;  // rows of positions beyond the history are zero
                const int jk = (int)((ik[it >> 1] >> (16 * (it & 1))) & 0xffffu), jv = (int)((iv[it >> 1] >> (16 * (it & 1))) & 0xffffu);
                // (range-checked build: pool indices below n_entries, destinations inside the stage)
                (void)CKV_CLAMP((int)(512 * it + kv_lane), kTileK - 15, err_flag);
                (void)CKV_CLAMP((int)(kVGroup * it + kv_lane), kTileV - 15, err_flag);
                cp_async16(kdst + 512 * it, pk + (size_t)CKV_CLAMP(jk, full_k ? TK : a.cv.n_entries, err_flag) * (D * 2), nb);
                cp_async16(vdst + kVGroup * it, pv + (size_t)CKV_CLAMP(jv, full_v ? TK : a.cv.n_entries, err_flag) * (D * 2), nb);
            }
            cp_async_commit();
            // what this warp's next tile needs travels while the copies land
            st.advance_by(kProducerWarps);
            fetch();
            cp_async_wait<0>();
            __syncwarp();  // a row's chunks were copied by four lanes of this warp
            if constexpr (DUB > 0) {
#pragma unroll
                for (int rb = 0; rb < 4; ++rb) {
                    if (32 * rb + patch_pos < valid) {  // zero rows beyond the history stay zero
                        if (!full_k) uk[rb].store(smem + kOffK + s * kTileK + k_off(32 * rb + lane, 0));
                        if (!full_v) uv[rb].store(smem + kOffV + s * kTileV + v_off(32 * rb + lane, 0));
                    }
                }
            }
            fence_proxy_async();  // by the writing threads themselves: a fence on the reading side alone is not enough
            __syncwarp();
            if (lane == 0) {
                if (q_slot >= 0) mbar_arrive(bar(BAR_QFULL + q_slot));
                mbar_arrive(bar(BAR_FULL + s));
            }
        }
        cp_async_wait<0>();
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(err_flag, ERR_PRODUCER);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && abort_flag[1] != 0) atomicOr(err_flag, abort_flag[1] << 8);
    if (warp == kIssueWarp0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

bool umma_supported(int dtype, int head_dim, int d_user, int idx_bytes)
{
    return dtype == CKV_BF16 && head_dim == D && idx_bytes == 2 &&
           (d_user == 0 || d_user == 1 || d_user == 2 || d_user == 4 || d_user == 8);
}

namespace {

// vmax[off(req) + mb] = largest visible length (clamped to the history) among the rows of query block mb of a
// request; off(req) is pad[0] of the request's work records.  One block per work item (its request's blocks are
// written once per item: the same values).
__global__ void vis_block_max_kernel(const Work* __restrict__ works, int n_items, const int32_t* __restrict__ vis,
                                     int32_t* __restrict__ vmax)
{
    const Work w = works[blockIdx.x];
    const int n_mb = (w.M + 127) / 128;
    for (int mb = threadIdx.x >> 5; mb < n_mb; mb += blockDim.x >> 5) {
        int m = 0;
        for (int r = 128 * mb + (threadIdx.x & 31); r < min(w.M, 128 * mb + 128); r += 32)
            m = max(m, min(max(__ldg(vis + w.q0 + r), 0), w.L));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        if ((threadIdx.x & 31) == 0) vmax[w.pad[0] + mb] = m;
    }
}

}  // namespace

cudaError_t launch_vis_block_max(const AttendArgs& a, int32_t* vmax, cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    vis_block_max_kernel<<<a.n_items, 128, 0, s>>>(a.works, a.n_items, a.vis, vmax);
    return cudaGetLastError();
}

cudaError_t launch_attend_umma(int max_M, const AttendArgs& a, int n_sms, int* err_flag, cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    const int n_mb = (max_M + 127) / 128;
    const int64_t n_work = (int64_t)a.n_items * n_mb * a.cv.n_groups;
    if (n_work + n_sms >= (int64_t)1 << 32) return cudaErrorInvalidValue;  // the kernel counts units in 32 bits
    const unsigned grid = (unsigned)(n_work < n_sms ? n_work : n_sms);
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, kSmemBytes, s>>>(a, n_mb, n_work, err_flag);
        return cudaGetLastError();
    };
    const bool sm = a.mode == CKV_SOFTMAX, vis = a.vis != nullptr;
    if (vis && a.vmax == nullptr) return cudaErrorInvalidValue;
#define CKV_UMMA_GO(DUB)                                                                                          \
    (vis ? (sm ? go(attend_umma_kernel<CKV_SOFTMAX, DUB, true>) : go(attend_umma_kernel<CKV_SILU_OVER_L, DUB, true>)) \
         : (sm ? go(attend_umma_kernel<CKV_SOFTMAX, DUB, false>) : go(attend_umma_kernel<CKV_SILU_OVER_L, DUB, false>)))
    switch (a.cv.full_k && a.cv.full_v ? 0 : a.cv.d_user) {  // the user-specific width of the shared side(s)
        case 0: return CKV_UMMA_GO(0);
        case 1: return CKV_UMMA_GO(2);
        case 2: return CKV_UMMA_GO(4);
        case 4: return CKV_UMMA_GO(8);
        case 8: return CKV_UMMA_GO(16);
    }
#undef CKV_UMMA_GO
    return cudaErrorInvalidValue;
}

}  // namespace ckv
