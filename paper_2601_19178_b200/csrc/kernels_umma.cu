// tcgen05 gather-concat-attention kernel (bf16, head_dim 32) for many queries per user.
//
// Persistent: one CTA per SM walks a static round-robin share of the work units, where a unit
// is (work item = history chunk of one user, group, block of up to 128 queries).  The history
// chunk is processed in tiles of 128 positions.  Roles (warp-specialised, 13 warps):
//   warps 0-3   normalisation group 0: thread i owns query row i = TMEM lane i, even tiles
//   warps 4-7   normalisation group 1: the same rows, odd tiles
//   warp  8     issues tcgen05.mma (one thread), owns the TMEM allocation
//   warps 9-12  producers: gather pool rows into shared memory with 16-byte cp.async, patch the
//               user-specific leading elements (Eq. K), publish the tile; also stage Q
//
// Tile t of the CTA's tile stream uses score buffer b = t mod 2:
//   S_b  = Q K_t^T                    UMMA 128 x 128 x 32, A = Q smem, B = K tile smem (K-major)
//   P_b  = exp2(S_b c - m) | silu     group b: tcgen05.ld -> math -> bf16 -> tcgen05.st
//   O_b += P_b [V_t | 1]              UMMA 128 x 48 x 128, A = P from TMEM, B = V tile (MN-major)
// While group b normalises tile t the tensor core already works on tile t+1 for the other
// group, and the producers gather tiles t+2...; nothing drains between work units.  The two
// groups keep separate accumulators O_0, O_1 with separate reference maxima and merge them
// through shared memory when a unit ends.
//
// Softmax bookkeeping.  The V tile carries sixteen extra columns of which the first is all
// ones, so column 32 of O_b accumulates the row sum l of exactly the bf16-rounded P that
// multiplies V.  The reference maximum m of a row is the exact maximum of the group's first
// tile of the unit and stays fixed: later scores may exceed it by up to 2^64 (fp32
// accumulators and bf16 P have the exponent range for that); only when a tile exceeds that
// bound is O_b rescaled (TMEM read-modify-write) and the tile redone.
//
// Shared-memory tiles use the no-swizzle UMMA canonical layout: groups of 8 rows, inside a
// group one 128-byte core matrix per 16-byte row chunk, inside a core matrix row r%8 at 16 r.
// K tiles and Q use 512-byte groups (4 chunks); V tiles 768-byte groups (4 data chunks + 2
// chunks holding the ones column).
//
// Every wait in this kernel is bounded: on time-out the CTA records an error code, raises a
// CTA-wide abort flag that ends every other wait, drains its own copies, frees its TMEM and
// returns.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int D = 32;
constexpr int TK = 128;                  // positions per tile
constexpr int NS = 6;                    // K/V stages
constexpr int LAG = 3;                   // tiles whose copies are in flight per producer thread
constexpr int NQ = 3;                    // Q buffers
// A producer publishes tile t - LAG before it issues tile t.  Q buffer reuse waits for the unit
// NQ units back, whose last tile is at most t - NQ: published already iff NQ >= LAG.
static_assert(NQ >= LAG, "Q buffer reuse would wait for a tile that is not published yet");
constexpr int kGroupThreads = 128;       // one normalisation group
constexpr int kMmaWarp = 8;
constexpr int kProducerWarp0 = 9;
constexpr int kProducerThreads = 128;
constexpr int kThreads = 2 * kGroupThreads + 32 + kProducerThreads;  // 416
constexpr int kTileK = TK * D * 2;       // 8 KB, also the Q tile
constexpr int kVGroup = 768;             // bytes of one 8-row group of a V tile
constexpr int kTileV = (TK / 8) * kVGroup;  // 12 KB
constexpr int kNV = 48;                  // columns of [V | 1 | 0...]
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColP = 256, kColO = 384;  // S_b at kColS + 128 b, P_b at kColP + 64 b, O_b at kColO + 48 b
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kHeadroom = 64.0f;       // log2 units a score may exceed the reference maximum
constexpr uint32_t kSpinLimit = 1u << 20;

// dynamic shared memory map
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + NQ * kTileK;
constexpr int kOffV = kOffK + NS * kTileK;
constexpr int kOffX = kOffV + NS * kTileV;          // exchange between the groups: [34][128] floats
constexpr int kOffBar = kOffX + 34 * 128 * 4;
constexpr int kOffAbort = kOffBar + 256;
constexpr int kSmemBytes = kOffAbort + 16;

// barrier slots (8 bytes each) behind kOffBar
enum {
    BAR_FULL = 0, BAR_EMPTY = NS, BAR_QEMPTY = 2 * NS, BAR_SFULL = 2 * NS + NQ, BAR_PREADY = BAR_SFULL + 2,
    BAR_PFREE = BAR_SFULL + 4, BAR_OFULL = BAR_SFULL + 6, BAR_XFULL = BAR_SFULL + 8, BAR_XEMPTY, BAR_DRAIN, BAR_COUNT
};
static_assert(BAR_COUNT * 8 <= 256, "barrier area");

// error codes OR-ed into the context's device error word
enum { ERR_NORMALISE = 1, ERR_MMA = 2, ERR_DRAIN = 4, ERR_PRODUCER = 8 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on a phase parity.  Returns false on time-out or when the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* abort_flag)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}
// 16-byte copy global -> shared; src_bytes = 0 fills the destination with zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes)
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

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float tanh_fast(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// byte offset of (row r, 16-byte chunk c) inside a K/Q tile and inside a V tile
__device__ __forceinline__ uint32_t k_off(int r, int c) { return (uint32_t)((r >> 3) * 512 + c * 128 + (r & 7) * 16); }
__device__ __forceinline__ uint32_t v_off(int r, int c) { return (uint32_t)((r >> 3) * kVGroup + c * 128 + (r & 7) * 16); }

// One work unit of the CTA's share.
struct Unit {
    Item it;
    Req rq;
    int grp;
    int row0;        // first query row of the block
    int n_tiles;     // > 0: tiles to process; 0: empty history (zero output rows); < 0: nothing at all
    int last_valid;  // real positions in the last tile
};

__device__ __forceinline__ void load_unit(const AttendArgs& a, int n_mb, int64_t w, Unit& u)
{
    const int G = a.cv.n_groups;
    const int mb = (int)(w % n_mb);
    const int64_t t = w / n_mb;
    u.grp = (int)(t % G);
    u.it = a.items[t / G];
    u.rq = a.reqs[u.it.req];
    u.row0 = mb * 128;
    u.n_tiles = u.row0 < u.rq.M ? (u.it.len + TK - 1) / TK : -1;
    u.last_valid = u.it.len - (u.n_tiles - 1) * TK;
}

// The CTA's tile stream: units blockIdx.x, blockIdx.x + gridDim.x, ... that have tiles, tile by
// tile.  Every role walks an identical copy, so stage and buffer indices need no communication.
struct Stream {
    const AttendArgs* a;
    int n_mb;
    int64_t w, n_work;
    Unit u;
    int j;       // tile inside the unit
    int g;       // tiles before this one in the stream
    int useq;    // units with tiles before this one
    bool valid;
    __device__ __forceinline__ void seek()
    {
        valid = false;
        while (w < n_work) {
            load_unit(*a, n_mb, w, u);
            if (u.n_tiles > 0) {
                valid = true;
                j = 0;
                return;
            }
            w += gridDim.x;
        }
    }
    __device__ __forceinline__ void init(const AttendArgs* args, int n_mb_, int64_t n_work_)
    {
        a = args;
        n_mb = n_mb_;
        n_work = n_work_;
        w = blockIdx.x;
        g = 0;
        useq = 0;
        seek();
    }
    __device__ __forceinline__ void advance()
    {
        ++g;
        if (++j == u.n_tiles) {
            w += gridDim.x;
            ++useq;
            seek();
        }
    }
};

template <int MODE, bool IDX16>
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
            mbar_init(bar(BAR_FULL + s), kProducerThreads);
            mbar_init(bar(BAR_EMPTY + s), 1);
        }
        for (int q = 0; q < NQ; ++q) mbar_init(bar(BAR_QEMPTY + q), 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(BAR_SFULL + b), 1);
            mbar_init(bar(BAR_PREADY + b), kGroupThreads);
            mbar_init(bar(BAR_PFREE + b), 1);
            mbar_init(bar(BAR_OFULL + b), 1);
        }
        mbar_init(bar(BAR_XFULL), kGroupThreads);
        mbar_init(bar(BAR_XEMPTY), kGroupThreads);
        mbar_init(bar(BAR_DRAIN), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the constant chunks 4 and 5 of every V stage: column 32 is one, columns 33..47 are zero
    for (int i = tid; i < NS * TK * 2; i += kThreads) {
        const int s = i / (TK * 2), r = (i >> 1) & (TK - 1), c = 4 + (i & 1);
        *reinterpret_cast<uint4*>(smem + kOffV + s * kTileV + v_off(r, c)) = make_uint4(c == 4 ? 0x3f80u : 0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;

    if (warp < 8) {
        // --------------------------------------------------------------- normalisation groups
        const int b = warp >> 2;                  // group = score buffer
        const int row = tid & (kGroupThreads - 1);  // query row inside the block = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + 128u * b, tP = tmem + lane_base + kColP + 64u * b,
                       tO = tmem + lane_base + kColO + (uint32_t)kNV * b;
        const float sc = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 0.5f);
        float* xch = reinterpret_cast<float*>(smem + kOffX);
        int cnt = 0;    // tiles this group has normalised
        int ocnt = 0;   // units in which this group had tiles
        int xcnt = 0;   // units exchanged between the groups
        int g = 0;      // tiles of the stream before the current unit
        bool ok = true;
        for (int64_t w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
            Unit u;
            load_unit(a, n_mb, w, u);
            if (u.n_tiles < 0) continue;
            const int r = u.row0 + row;
            const int64_t out_base = ((int64_t)(u.rq.q0 + r) * G + u.grp) * D;
            if (u.n_tiles == 0) {  // empty history: zero output rows
                if (b == 0 && r < u.rq.M && u.it.part_row < 0) {
                    if (a.out_dtype == CKV_BF16) {
                        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(a.out) + out_base);
                        for (int q4 = 0; q4 < 4; ++q4) dst[q4] = make_uint4(0, 0, 0, 0);
                    } else {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + out_base);
                        for (int q4 = 0; q4 < 8; ++q4) dst[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                continue;
            }
            float m_ref = -CUDART_INF_F;
            int mine = 0;  // tiles of this unit normalised by this group
            for (int j = 0; j < u.n_tiles && ok; ++j) {
                if (((g + j) & 1) != b) continue;
                ok = mbar_wait(bar(BAR_SFULL + b), cnt & 1, abort_flag);
                if (ok && cnt > 0) ok = mbar_wait(bar(BAR_PFREE + b), (cnt - 1) & 1, abort_flag);  // P_b and O_b are quiet
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int valid = j == u.n_tiles - 1 ? u.last_valid : TK;
                const bool tail = valid < TK;
                if constexpr (MODE == CKV_SOFTMAX) {
                    if (mine == 0) {  // the reference maximum: exact maximum of the first tile
                        float tmax = -CUDART_INF_F;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            uint32_t s[32];
                            tmem_ld32(tS + 32 * c, s);
                            tmem_wait_ld32(s);
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float x0 = __uint_as_float(s[e]), x1 = __uint_as_float(s[e + 1]);
                                if (tail) {
                                    if (32 * c + e >= valid) x0 = -CUDART_INF_F;
                                    if (32 * c + e + 1 >= valid) x1 = -CUDART_INF_F;
                                }
                                tmax = max3(tmax, x0, x1);
                            }
                        }
                        m_ref = tmax * sc;  // valid >= 1, so finite
                    }
                    for (int attempt = 0; attempt < 2; ++attempt) {
                        const float nm = -m_ref;
                        float mx = -CUDART_INF_F;
                        uint32_t sa[32], sb[32];
                        tmem_ld32(tS, sa);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t(&cur)[32] = (c & 1) ? sb : sa;
                            uint32_t(&nxt)[32] = (c & 1) ? sa : sb;
                            tmem_wait_ld32(cur);
                            if (c < 3) tmem_ld32(tS + 32 * (c + 1), nxt);
                            uint32_t p[16];
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float x0 = fmaf(__uint_as_float(cur[e]), sc, nm), x1 = fmaf(__uint_as_float(cur[e + 1]), sc, nm);
                                if (tail) {
                                    if (32 * c + e >= valid) x0 = -CUDART_INF_F;
                                    if (32 * c + e + 1 >= valid) x1 = -CUDART_INF_F;
                                }
                                mx = max3(mx, x0, x1);
                                p[e >> 1] = pack_bf16(ex2(x0), ex2(x1));
                            }
                            tmem_st16(tP + 16 * c, p);
                        }
                        if (!__any_sync(0xffffffffu, mx > kHeadroom)) break;
                        // some row of this warp left the headroom: move its reference, rescale what
                        // O_b holds so far (its MMAs have finished, see the PFREE wait) and redo the tile
                        const float shift = mx > kHeadroom ? mx : 0.f;
                        const float f = ex2(-shift);
                        m_ref += shift;
                        if (mine > 0) {
                            uint32_t o[32];
                            tmem_ld32(tO, o);
                            tmem_wait_ld32(o);
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
                            tmem_st32(tO, o);
                            const uint32_t l = tmem_ld1(tO + 32);
                            tmem_st1(tO + 32, __float_as_uint(__uint_as_float(l) * f));
                        }
                        tc_wait_st();
                    }
                } else {
                    // silu(x) = x sigmoid(x) = h (1 + tanh(h)), h = x / 2   (sc = scale / 2)
                    uint32_t sa[32], sb[32];
                    tmem_ld32(tS, sa);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t(&cur)[32] = (c & 1) ? sb : sa;
                        uint32_t(&nxt)[32] = (c & 1) ? sa : sb;
                        tmem_wait_ld32(cur);
                        if (c < 3) tmem_ld32(tS + 32 * (c + 1), nxt);
                        uint32_t p[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            const float h0 = __uint_as_float(cur[e]) * sc, h1 = __uint_as_float(cur[e + 1]) * sc;
                            float w0 = fmaf(h0, tanh_fast(h0), h0), w1 = fmaf(h1, tanh_fast(h1), h1);
                            if (tail) {
                                if (32 * c + e >= valid) w0 = 0.f;
                                if (32 * c + e + 1 >= valid) w1 = 0.f;
                            }
                            p[e >> 1] = pack_bf16(w0, w1);
                        }
                        tmem_st16(tP + 16 * c, p);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(BAR_PREADY + b));
                ++cnt;
                ++mine;
            }
            g += u.n_tiles;
            if (!ok) break;

            // ---- the unit's epilogue: fetch O_b, merge the two groups, store
            float o[32], l = 0.f;
            if (mine > 0) {
                ok = mbar_wait(bar(BAR_OFULL + b), ocnt & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ++ocnt;
                tc_fence_after();
                uint32_t raw[32];
                tmem_ld32(tO, raw);
                tmem_wait_ld32(raw);
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __uint_as_float(raw[e]);
                if constexpr (MODE == CKV_SOFTMAX) l = __uint_as_float(tmem_ld1(tO + 32));
                tc_fence_before();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = 0.f;
            }
            if (b == 1) {
                if (xcnt > 0) ok = mbar_wait(bar(BAR_XEMPTY), (xcnt - 1) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                xch[row] = m_ref;
                xch[128 + row] = l;
#pragma unroll
                for (int e = 0; e < 32; ++e) xch[(2 + e) * 128 + row] = o[e];
                mbar_arrive(bar(BAR_XFULL));
                ++xcnt;
            } else {
                ok = mbar_wait(bar(BAR_XFULL), xcnt & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ++xcnt;
                const float m1 = xch[row], l1 = xch[128 + row];
                if constexpr (MODE == CKV_SOFTMAX) {
                    const float mt = fmaxf(m_ref, m1);
                    const float ms = mt == -CUDART_INF_F ? 0.f : mt;
                    const float c0 = ex2(m_ref - ms), c1 = ex2(m1 - ms);
                    l = l * c0 + l1 * c1;
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = o[e] * c0 + xch[(2 + e) * 128 + row] * c1;
                    m_ref = mt;
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] += xch[(2 + e) * 128 + row];
                }
                mbar_arrive(bar(BAR_XEMPTY));
                if (r < u.rq.M) {
                    if (u.it.part_row < 0) {
                        float inv;
                        if constexpr (MODE == CKV_SOFTMAX) inv = l > 0.f ? 1.0f / l : 0.f;
                        else inv = 1.0f / (float)u.rq.L;
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
                        float* pr = a.partials + ((int64_t)(u.it.part_row + r) * G + u.grp) * (D + 2);
                        pr[0] = m_ref;
                        pr[1] = l;
#pragma unroll
                        for (int e = 0; e < 32; ++e) pr[2 + e] = o[e];
                    }
                }
            }
        }
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(err_flag, ERR_NORMALISE);
        }
    } else if (warp == kMmaWarp) {
        // --------------------------------------------------------------------- MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(128, TK, false);
            constexpr uint32_t idesc_pv = make_idesc(128, MODE == CKV_SOFTMAX ? kNV : D, true);
            Stream ss, sp;  // next tile whose S / whose PV is to be issued
            ss.init(&a, n_mb, n_work);
            sp = ss;
            int pcnt[2] = {0, 0};
            bool ok = true;
            auto issue_s = [&]() {
                const int s = ss.g % NS, b = ss.g & 1;
                if (!mbar_wait(bar(BAR_FULL + s), (ss.g / NS) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t q_addr = sbase + kOffQ + (ss.useq % NQ) * kTileK, k_addr = sbase + kOffK + s * kTileK;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    umma_ss(tmem + kColS + 128u * b, smem_desc(q_addr + ks * 256, 128, 512),
                            smem_desc(k_addr + ks * 256, 128, 512), idesc_s, ks > 0 ? 1u : 0u);
                tc_commit(bar(BAR_SFULL + b));
                if (ss.j == ss.u.n_tiles - 1) tc_commit(bar(BAR_QEMPTY + ss.useq % NQ));  // Q buffer no longer read
                ss.advance();
                return true;
            };
            auto issue_pv = [&]() {  // O_b += P_b [V | 1], sixteen positions per instruction
                const int s = sp.g % NS, b = sp.g & 1;
                if (!mbar_wait(bar(BAR_PREADY + b), pcnt[b] & 1, abort_flag)) return false;
                ++pcnt[b];
                tc_fence_after();
                const uint32_t v_addr = sbase + kOffV + s * kTileV;
#pragma unroll
                for (int kk = 0; kk < TK / 16; ++kk)
                    umma_ts(tmem + kColO + (uint32_t)kNV * b, tmem + kColP + 64u * b + 8 * kk,
                            smem_desc(v_addr + kk * 2 * kVGroup, kVGroup, 128), idesc_pv, (sp.j >= 2 || kk > 0) ? 1u : 0u);
                tc_commit(bar(BAR_EMPTY + s));
                tc_commit(bar(BAR_PFREE + b));
                if (sp.j >= sp.u.n_tiles - 2) tc_commit(bar(BAR_OFULL + b));  // last tile of its group in the unit
                sp.advance();
                return true;
            };
            if (ss.valid) ok = issue_s();
            if (ok && ss.valid) ok = issue_s();
            while (ok && sp.valid) {
                ok = issue_pv();
                if (ok && ss.valid) ok = issue_s();
            }
            if (!ok) {
                *abort_flag = 1;
                atomicOr(err_flag, ERR_MMA);
            }
            // nothing of this CTA may still be running on the tensor core at teardown
            tc_commit(bar(BAR_DRAIN));
            volatile int never = 0;
            if (!mbar_wait(bar(BAR_DRAIN), 0, &never)) atomicOr(err_flag, ERR_DRAIN);
        }
        __syncwarp();
    } else {
        // --------------------------------------------------------------------- producers
        const int p = tid - kProducerWarp0 * 32;  // 0..127 = the tile row this thread owns
        const int pw = p >> 5;
        const int du_bytes = a.cv.d_user * 2;
        const int src_lane0 = lane >> 2, chunk = lane & 3;
        Stream st;
        st.init(&a, n_mb, n_work);
        bool ok = true;
        // per tile in flight: where it went and this thread's user-specific leading elements
        uint4 uk[LAG], uv[LAG];
        int stage_of[LAG];
        bool patch[LAG], live[LAG];
#pragma unroll
        for (int u = 0; u < LAG; ++u) {
            live[u] = false;
            patch[u] = false;
            stage_of[u] = 0;
            uk[u] = uv[u] = make_uint4(0, 0, 0, 0);
        }
        // indices of the next tile to issue, loaded one iteration ahead
        int ik = 0, iv = 0;
        int64_t my_unit = 0;
        bool my_valid = false;
        auto prefetch = [&]() {
            if (!st.valid) return;
            const int valid = st.j == st.u.n_tiles - 1 ? st.u.last_valid : TK;
            my_valid = p < valid;
            my_unit = st.u.rq.base + (int64_t)st.u.grp * st.u.rq.Lpad + st.u.it.begin + (int64_t)st.j * TK + p;
            ik = iv = 0;
            if (my_valid) {
                if constexpr (IDX16) {
                    ik = __ldg(reinterpret_cast<const uint16_t*>(a.cv.idxK) + my_unit);
                    iv = __ldg(reinterpret_cast<const uint16_t*>(a.cv.idxV) + my_unit);
                } else {
                    ik = __ldg(reinterpret_cast<const int32_t*>(a.cv.idxK) + my_unit);
                    iv = __ldg(reinterpret_cast<const int32_t*>(a.cv.idxV) + my_unit);
                }
            }
        };
        prefetch();
        bool more = true;
        while (more) {
            more = false;
#pragma unroll
            for (int u = 0; u < LAG; ++u) {
                // (1) the tile issued LAG iterations ago has landed: patch and publish it
                if (live[u]) {
                    cp_async_wait<LAG - 1>();
                    __syncwarp();  // a row's chunks were copied by four other lanes of this warp
                    if (patch[u]) {  // Eq. K: dims [0, d_user) come from the user part
                        unsigned char* kd = smem + kOffK + stage_of[u] * kTileK + k_off(p, 0);
                        unsigned char* vd = smem + kOffV + stage_of[u] * kTileV + v_off(p, 0);
                        if (du_bytes == 4) {
                            *reinterpret_cast<uint32_t*>(kd) = uk[u].x;
                            *reinterpret_cast<uint32_t*>(vd) = uv[u].x;
                        } else if (du_bytes == 2) {
                            *reinterpret_cast<uint16_t*>(kd) = (uint16_t)uk[u].x;
                            *reinterpret_cast<uint16_t*>(vd) = (uint16_t)uv[u].x;
                        } else if (du_bytes == 8) {
                            *reinterpret_cast<uint2*>(kd) = make_uint2(uk[u].x, uk[u].y);
                            *reinterpret_cast<uint2*>(vd) = make_uint2(uv[u].x, uv[u].y);
                        } else {
                            *reinterpret_cast<uint4*>(kd) = uk[u];
                            *reinterpret_cast<uint4*>(vd) = uv[u];
                        }
                    }
                    fence_proxy_async();
                    mbar_arrive(bar(BAR_FULL + stage_of[u]));
                    live[u] = false;
                }
                // (2) issue the copies of the next tile of the stream
                if (st.valid && ok) {
                    const int s = st.g % NS;
                    if (st.g >= NS) ok = mbar_wait(bar(BAR_EMPTY + s), ((st.g / NS) - 1) & 1, abort_flag);
                    if (ok && st.j == 0) {  // a new unit: stage its Q block (rows beyond M are zero)
                        if (st.useq >= NQ) ok = mbar_wait(bar(BAR_QEMPTY + st.useq % NQ), ((st.useq / NQ) - 1) & 1, abort_flag);
                        if (ok) {
                            const uint32_t qdst = sbase + kOffQ + (st.useq % NQ) * kTileK;
                            const uint16_t* Q = reinterpret_cast<const uint16_t*>(a.queries);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int r = 32 * pw + 8 * i + src_lane0;
                                const bool in = st.u.row0 + r < st.u.rq.M;
                                const uint16_t* src = Q + ((int64_t)(st.u.rq.q0 + st.u.row0 + (in ? r : 0)) * G + st.u.grp) * D + chunk * 8;
                                cp_async16(qdst + k_off(r, chunk), src, in ? 16u : 0u);
                            }
                        }
                    }
                    if (ok) {
                        const char* poolK = reinterpret_cast<const char*>(a.cv.poolK) + (int64_t)st.u.grp * a.cv.n_entries * (D * 2);
                        const char* poolV = reinterpret_cast<const char*>(a.cv.poolV) + (int64_t)st.u.grp * a.cv.n_entries * (D * 2);
                        const uint32_t kdst = sbase + kOffK + s * kTileK, vdst = sbase + kOffV + s * kTileV;
                        const uint32_t vbits = __ballot_sync(0xffffffffu, my_valid);
                        // four lanes fetch the four 16-byte chunks of one row: 64 contiguous bytes per row
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int sl = 8 * i + src_lane0;
                            const int rk = __shfl_sync(0xffffffffu, ik, sl), rv = __shfl_sync(0xffffffffu, iv, sl);
                            const uint32_t nb = (vbits >> sl) & 1u ? 16u : 0u;  // rows beyond the history are zero
                            const int r = 32 * pw + sl;
                            cp_async16(kdst + k_off(r, chunk), poolK + (int64_t)rk * (D * 2) + chunk * 16, nb);
                            cp_async16(vdst + v_off(r, chunk), poolV + (int64_t)rv * (D * 2) + chunk * 16, nb);
                        }
                        patch[u] = my_valid && du_bytes > 0;
                        if (patch[u]) {
                            const char* ku = reinterpret_cast<const char*>(a.cv.userK) + my_unit * du_bytes;
                            const char* vu = reinterpret_cast<const char*>(a.cv.userV) + my_unit * du_bytes;
                            if (du_bytes == 4) {
                                uk[u].x = __ldg(reinterpret_cast<const uint32_t*>(ku));
                                uv[u].x = __ldg(reinterpret_cast<const uint32_t*>(vu));
                            } else if (du_bytes == 2) {
                                uk[u].x = __ldg(reinterpret_cast<const uint16_t*>(ku));
                                uv[u].x = __ldg(reinterpret_cast<const uint16_t*>(vu));
                            } else if (du_bytes == 8) {
                                const uint2 x = __ldg(reinterpret_cast<const uint2*>(ku)), y = __ldg(reinterpret_cast<const uint2*>(vu));
                                uk[u] = make_uint4(x.x, x.y, 0, 0);
                                uv[u] = make_uint4(y.x, y.y, 0, 0);
                            } else {
                                uk[u] = __ldg(reinterpret_cast<const uint4*>(ku));
                                uv[u] = __ldg(reinterpret_cast<const uint4*>(vu));
                            }
                        }
                        stage_of[u] = s;
                        live[u] = true;
                        st.advance();
                        prefetch();
                    }
                }
                cp_async_commit();  // one group per iteration, also when nothing was issued
                more = more || live[u];
            }
            more = more || (st.valid && ok);
        }
        cp_async_wait<0>();
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(err_flag, ERR_PRODUCER);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

bool umma_supported(int dtype, int head_dim, int d_user)
{
    return dtype == CKV_BF16 && head_dim == D && (d_user == 0 || d_user == 1 || d_user == 2 || d_user == 4 || d_user == 8);
}

cudaError_t launch_attend_umma(int max_M, const AttendArgs& a, int n_sms, int* err_flag, cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    const int n_mb = (max_M + 127) / 128;
    const int64_t n_work = (int64_t)a.n_items * n_mb * a.cv.n_groups;
    const unsigned grid = (unsigned)(n_work < n_sms ? n_work : n_sms);
    const bool i16 = a.cv.idx_bytes == 2;
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, kSmemBytes, s>>>(a, n_mb, n_work, err_flag);
        return cudaGetLastError();
    };
    if (a.mode == CKV_SOFTMAX)
        return i16 ? go(attend_umma_kernel<CKV_SOFTMAX, true>) : go(attend_umma_kernel<CKV_SOFTMAX, false>);
    return i16 ? go(attend_umma_kernel<CKV_SILU_OVER_L, true>) : go(attend_umma_kernel<CKV_SILU_OVER_L, false>);
}

}  // namespace ckv
