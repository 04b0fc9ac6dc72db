// tcgen05 gather-concat-attention kernel (bf16, head_dim 32) for many queries per user.
//
// One CTA owns (work item, group, block of up to 128 queries) and walks the history chunk
// in tiles of 128 positions.  Roles (warp-specialised, 7 warps):
//   warps 0-3  softmax / SiLU: thread i owns query row i = TMEM lane i
//   warp  4    issues tcgen05.mma (one elected thread), owns the TMEM allocation
//   warps 5-6  producers: gather pool rows into shared memory with 16-byte cp.async,
//              patch the user-specific leading elements (Eq. K), publish the tile
//
// Per tile j:   S_j = Q K_j^T   (UMMA 128 x 128 x 32, A = Q smem, B = K tile smem, K-major)
//               P_j = exp2(S_j c - m) or silu(S_j c)    (softmax warps: tcgen05.ld -> math ->
//                                                         bf16 -> tcgen05.st)
//               O  += P_j V_j   (UMMA 128 x 32 x 128, A = P from TMEM, B = V tile smem, MN-major)
// O stays in TMEM for the whole chunk.  The softmax keeps a reference maximum m per row and
// only rescales O (a TMEM read-modify-write) when a tile raises the maximum by more than 2^8;
// otherwise p may exceed 1 by at most that factor, which fp32/bf16 hold easily.
//
// Shared-memory tiles use the no-swizzle UMMA canonical layout: 8-row groups of 512 bytes,
// inside a group four 128-byte core matrices (one per 16-byte row chunk), inside a core
// matrix row r%8 at 16 r.  A gathered 64-byte row therefore lands as four 16-byte pieces;
// the same physical layout serves K (K-major B operand) and V (MN-major B operand).
//
// Every wait in this kernel is bounded: on time-out the CTA records an error code, drains its
// own copies, frees its TMEM and returns.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int D = 32;
constexpr int TK = 128;                 // positions per tile
constexpr int NS = 4;                   // shared-memory stages
constexpr int kSoftmaxThreads = 128;
constexpr int kProducerThreads = 64;
constexpr int kThreads = kSoftmaxThreads + 32 + kProducerThreads;  // 224
constexpr int kMmaWarp = 4;
constexpr int kTileBytes = TK * D * 2;  // 8 KB
constexpr int kMaxDu = 8;
constexpr int kSideBytes = TK * kMaxDu * 2;  // user part of one tile, K or V: up to 2 KB
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColP = 128, kColO = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr uint32_t kSpinLimit = 1u << 20;

// dynamic shared memory map
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kTileBytes;
constexpr int kOffV = kOffK + NS * kTileBytes;
constexpr int kOffSideK = kOffV + NS * kTileBytes;
constexpr int kOffSideV = kOffSideK + NS * kSideBytes;
constexpr int kOffBar = kOffSideV + NS * kSideBytes;
constexpr int kSmemBytes = kOffBar + 256;  // 8 KB + 64 KB + 16 KB + barriers

// barrier slots (8 bytes each) behind kOffBar
enum { BAR_FULL = 0, BAR_EMPTY = NS, BAR_S = 2 * NS, BAR_P, BAR_PV, BAR_DRAIN, BAR_COUNT };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on a phase parity.  Returns false on time-out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
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
    }
    return false;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
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
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
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

// byte offset of (row r, 16-byte chunk c) inside a tile
__device__ __forceinline__ uint32_t tile_off(int r, int c) { return (uint32_t)((r >> 3) * 512 + c * 128 + (r & 7) * 16); }

template <int MODE, bool IDX16>
__global__ void __launch_bounds__(kThreads, 2) attend_umma_kernel(const AttendArgs a, int n_mb, int* err_flag)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint32_t tmem_base_slot;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Item it = a.items[blockIdx.x / n_mb];
    const int mb = blockIdx.x % n_mb;
    const Req rq = a.reqs[it.req];
    const int row0 = mb * 128;
    if (row0 >= rq.M) return;  // uniform per CTA
    const int grp = blockIdx.y, G = a.cv.n_groups, d_user = a.cv.d_user;
    const int n_tiles = (it.len + TK - 1) / TK;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar(BAR_FULL + s), kProducerThreads);
            mbar_init(bar(BAR_EMPTY + s), 1);
        }
        mbar_init(bar(BAR_S), 1);
        mbar_init(bar(BAR_P), kSoftmaxThreads);
        mbar_init(bar(BAR_PV), 1);
        mbar_init(bar(BAR_DRAIN), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Q tile: rows row0 .. row0+127 of this (user, group), zero beyond M
    {
        const uint16_t* Q = reinterpret_cast<const uint16_t*>(a.queries);
        for (int i = tid; i < 128 * 4; i += kThreads) {
            const int r = i >> 2, c = i & 3;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (row0 + r < rq.M)
                v = __ldg(reinterpret_cast<const uint4*>(Q + ((int64_t)(rq.q0 + row0 + r) * G + grp) * D + c * 8));
            *reinterpret_cast<uint4*>(smem + kOffQ + tile_off(r, c)) = v;
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;

    if (n_tiles > 0) {
        if (warp < 4) {
            // ------------------------------------------------------------- softmax / SiLU
            const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
            const float sc = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 0.5f);
            float m_ref = -CUDART_INF_F, l_run = 0.f;
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                ok = mbar_wait(bar(BAR_S), j & 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int valid = min(TK, it.len - j * TK);  // columns of this tile that are real positions
                bool waited_pv = false;
                if constexpr (MODE == CKV_SOFTMAX) {
                    float tmax = -CUDART_INF_F;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tmem_ld32(tmem + lane_base + kColS + 32 * c, r);
                        tc_wait_ld();
                        if (valid >= 32 * (c + 1)) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) tmax = fmaxf(tmax, __uint_as_float(r[e]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (32 * c + e < valid) tmax = fmaxf(tmax, __uint_as_float(r[e]));
                        }
                    }
                    const float m_new = fmaxf(m_ref, tmax * sc);  // valid >= 1, so finite
                    if (__any_sync(0xffffffffu, m_new > m_ref + kRescaleThreshold)) {
                        if (j > 0) {
                            ok = mbar_wait(bar(BAR_PV), (j - 1) & 1);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            waited_pv = true;
                            tc_fence_after();
                            const float f = ex2(m_ref - m_new);
                            uint32_t o[32];
                            tmem_ld32(tmem + lane_base + kColO, o);
                            tc_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
                            tmem_st32(tmem + lane_base + kColO, o);
                            l_run *= f;
                        }
                        m_ref = m_new;
                    }
                }
                if (j > 0 && !waited_pv) {  // P buffer is free once PV of the previous tile has finished
                    ok = mbar_wait(bar(BAR_PV), (j - 1) & 1);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + kColS + 32 * c, r);
                    tc_wait_ld();
                    uint32_t p[16];
                    const bool full = valid >= 32 * (c + 1);
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float w0, w1;
                        if constexpr (MODE == CKV_SOFTMAX) {
                            w0 = ex2(fmaf(__uint_as_float(r[e]), sc, -m_ref));
                            w1 = ex2(fmaf(__uint_as_float(r[e + 1]), sc, -m_ref));
                        } else {
                            const float h0 = __uint_as_float(r[e]) * sc, h1 = __uint_as_float(r[e + 1]) * sc;
                            w0 = fmaf(h0, tanh_fast(h0), h0);
                            w1 = fmaf(h1, tanh_fast(h1), h1);
                        }
                        if (!full) {
                            if (32 * c + e >= valid) w0 = 0.f;
                            if (32 * c + e + 1 >= valid) w1 = 0.f;
                        }
                        if constexpr (MODE == CKV_SOFTMAX) l_run += w0 + w1;
                        p[e >> 1] = pack_bf16(w0, w1);
                    }
                    tmem_st16(tmem + lane_base + kColP + 16 * c, p);
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(BAR_P));
            }
            // epilogue: O is final once the last PV has finished
            if (ok) {
                ok = mbar_wait(bar(BAR_PV), (n_tiles - 1) & 1);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (ok) {
                tc_fence_after();
                uint32_t o[32];
                tmem_ld32(tmem + lane_base + kColO, o);
                tc_wait_ld();
                const int r = row0 + tid;
                if (r < rq.M) {
                    if (it.part_row < 0) {
                        float inv;
                        if constexpr (MODE == CKV_SOFTMAX) inv = l_run > 0.f ? 1.0f / l_run : 0.f;
                        else inv = 1.0f / (float)rq.L;
                        const int64_t base = ((int64_t)(rq.q0 + r) * G + grp) * D;
                        if (a.out_dtype == CKV_BF16) {
                            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(a.out) + base);
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                uint4 v;
                                v.x = pack_bf16(__uint_as_float(o[8 * q4 + 0]) * inv, __uint_as_float(o[8 * q4 + 1]) * inv);
                                v.y = pack_bf16(__uint_as_float(o[8 * q4 + 2]) * inv, __uint_as_float(o[8 * q4 + 3]) * inv);
                                v.z = pack_bf16(__uint_as_float(o[8 * q4 + 4]) * inv, __uint_as_float(o[8 * q4 + 5]) * inv);
                                v.w = pack_bf16(__uint_as_float(o[8 * q4 + 6]) * inv, __uint_as_float(o[8 * q4 + 7]) * inv);
                                dst[q4] = v;
                            }
                        } else {
                            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + base);
#pragma unroll
                            for (int q4 = 0; q4 < 8; ++q4)
                                dst[q4] = make_float4(__uint_as_float(o[4 * q4]) * inv, __uint_as_float(o[4 * q4 + 1]) * inv,
                                                      __uint_as_float(o[4 * q4 + 2]) * inv, __uint_as_float(o[4 * q4 + 3]) * inv);
                        }
                    } else {
                        float* pr = a.partials + ((int64_t)(it.part_row + r) * G + grp) * (D + 2);
                        pr[0] = m_ref;
                        pr[1] = l_run;
#pragma unroll
                        for (int e = 0; e < 32; ++e) pr[2 + e] = __uint_as_float(o[e]);
                    }
                }
            }
            if (!ok && lane == 0) atomicOr(err_flag, 1);
        } else if (warp == kMmaWarp) {
            // ------------------------------------------------------------- MMA issue
            if (lane == 0) {
                constexpr uint32_t idesc_s = make_idesc(128, TK, false);
                constexpr uint32_t idesc_pv = make_idesc(128, D, true);
                const uint32_t q_addr = sbase + kOffQ;
                bool ok = true;
                auto issue_pv = [&](int j) {  // O += P_j V_j, sixteen positions per instruction
                    const uint32_t v_addr = sbase + kOffV + (j % NS) * kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < TK / 16; ++kk)
                        umma_ts(tmem + kColO, tmem + kColP + 8 * kk, smem_desc(v_addr + kk * 1024, 512, 128), idesc_pv,
                                (j > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar(BAR_PV));
                    tc_commit(bar(BAR_EMPTY + j % NS));
                };
                for (int j = 0; j < n_tiles; ++j) {
                    ok = mbar_wait(bar(BAR_FULL + j % NS), (j / NS) & 1);
                    if (ok && j > 0) ok = mbar_wait(bar(BAR_P), (j - 1) & 1);  // S free, P_{j-1} written
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t k_addr = sbase + kOffK + (j % NS) * kTileBytes;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        umma_ss(tmem + kColS, smem_desc(q_addr + ks * 256, 128, 512), smem_desc(k_addr + ks * 256, 128, 512),
                                idesc_s, ks > 0 ? 1u : 0u);
                    tc_commit(bar(BAR_S));
                    if (j > 0) issue_pv(j - 1);
                }
                if (ok) ok = mbar_wait(bar(BAR_P), (n_tiles - 1) & 1);
                if (ok) {
                    tc_fence_after();
                    issue_pv(n_tiles - 1);
                } else {
                    atomicOr(err_flag, 2);
                }
                // nothing of this CTA may still be running on the tensor core at teardown
                tc_commit(bar(BAR_DRAIN));
                if (!mbar_wait(bar(BAR_DRAIN), 0)) atomicOr(err_flag, 4);
            }
            __syncwarp();
        } else {
            // ------------------------------------------------------------- producers
            const int p = tid - (kSoftmaxThreads + 32);  // 0..63
            const char* poolK = reinterpret_cast<const char*>(a.cv.poolK) + (int64_t)grp * a.cv.n_entries * (D * 2);
            const char* poolV = reinterpret_cast<const char*>(a.cv.poolV) + (int64_t)grp * a.cv.n_entries * (D * 2);
            const int64_t unit0 = rq.base + (int64_t)grp * rq.Lpad + it.begin;
            const int side_granules = (TK * d_user * 2) / 16;  // 16-byte pieces of one tile's user part
            bool ok = true;
            constexpr int LAG = 2;
            for (int j = 0; j < n_tiles + LAG; ++j) {
                // after a time-out nothing more is copied, but the loop keeps its shape so that
                // every producer thread meets the same named barriers
                if (j < n_tiles && ok && j >= NS) ok = mbar_wait(bar(BAR_EMPTY + (j % NS)), ((j / NS) - 1) & 1);
                if (j < n_tiles && ok) {
                    const int s = j % NS;
                    const int valid = min(TK, it.len - j * TK);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int r = p + 64 * h;
                        int ik = 0, iv = 0;
                        if (r < valid) {
                            const int64_t u = unit0 + (int64_t)j * TK + r;
                            if constexpr (IDX16) {
                                ik = __ldg(reinterpret_cast<const uint16_t*>(a.cv.idxK) + u);
                                iv = __ldg(reinterpret_cast<const uint16_t*>(a.cv.idxV) + u);
                            } else {
                                ik = __ldg(reinterpret_cast<const int32_t*>(a.cv.idxK) + u);
                                iv = __ldg(reinterpret_cast<const int32_t*>(a.cv.idxV) + u);
                            }
                        }
                        const char* ksrc = poolK + (int64_t)ik * (D * 2);
                        const char* vsrc = poolV + (int64_t)iv * (D * 2);
                        const uint32_t kdst = sbase + kOffK + s * kTileBytes, vdst = sbase + kOffV + s * kTileBytes;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            cp_async16(kdst + tile_off(r, c), ksrc + 16 * c);
                            cp_async16(vdst + tile_off(r, c), vsrc + 16 * c);
                        }
                    }
                    // the tile's user-specific parts: contiguous in the cache, copied as they are
                    const int64_t pos0 = (int64_t)it.begin + (int64_t)j * TK;
                    for (int gr = p; gr < side_granules; gr += kProducerThreads) {
                        const int64_t first_pos = pos0 + (int64_t)gr * 8 / d_user;
                        if (first_pos < rq.Lpad) {
                            const int64_t byte = ((unit0 + (int64_t)j * TK) * d_user) * 2 + (int64_t)gr * 16;
                            cp_async16(sbase + kOffSideK + s * kSideBytes + gr * 16, reinterpret_cast<const char*>(a.cv.userK) + byte);
                            cp_async16(sbase + kOffSideV + s * kSideBytes + gr * 16, reinterpret_cast<const char*>(a.cv.userV) + byte);
                        }
                    }
                }
                cp_async_commit();
                if (j >= LAG) {
                    const int jj = j - LAG, s = jj % NS;
                    cp_async_wait<LAG>();
                    asm volatile("bar.sync 1, %0;" ::"n"(kProducerThreads) : "memory");  // side buffers are shared work
                    if (d_user > 0) {
                        const int valid = min(TK, it.len - jj * TK);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int r = p + 64 * h;
                            if (r < valid) {  // Eq. K: dims [0, d_user) come from the user part
                                const uint16_t* sk = reinterpret_cast<const uint16_t*>(smem + kOffSideK + s * kSideBytes) + r * d_user;
                                const uint16_t* sv = reinterpret_cast<const uint16_t*>(smem + kOffSideV + s * kSideBytes) + r * d_user;
                                uint16_t* kd = reinterpret_cast<uint16_t*>(smem + kOffK + s * kTileBytes + tile_off(r, 0));
                                uint16_t* vd = reinterpret_cast<uint16_t*>(smem + kOffV + s * kTileBytes + tile_off(r, 0));
                                for (int e = 0; e < d_user; ++e) {
                                    kd[e] = sk[e];
                                    vd[e] = sv[e];
                                }
                            }
                        }
                    }
                    fence_proxy_async();
                    mbar_arrive(bar(BAR_FULL + s));
                }
            }
            if (!ok) atomicOr(err_flag, 8);
            cp_async_wait<0>();
        }
    }

    if (n_tiles == 0 && warp < 4 && row0 + tid < rq.M && it.part_row < 0) {  // empty history: zero output row
        const int64_t base = ((int64_t)(rq.q0 + row0 + tid) * G + grp) * D;
        if (a.out_dtype == CKV_BF16) {
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(a.out) + base);
            for (int q4 = 0; q4 < 4; ++q4) dst[q4] = make_uint4(0, 0, 0, 0);
        } else {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + base);
            for (int q4 = 0; q4 < 8; ++q4) dst[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
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
    return dtype == CKV_BF16 && head_dim == D && d_user <= kMaxDu && (d_user == 0 || 8 % d_user == 0);
}

cudaError_t launch_attend_umma(int max_M, const AttendArgs& a, int* err_flag, cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    const int n_mb = (max_M + 127) / 128;
    const dim3 grid((unsigned)((int64_t)a.n_items * n_mb), a.cv.n_groups);
    const bool i16 = a.cv.idx_bytes == 2;
    auto go = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, kSmemBytes, s>>>(a, n_mb, err_flag);
        return cudaGetLastError();
    };
    if (a.mode == CKV_SOFTMAX)
        return i16 ? go(attend_umma_kernel<CKV_SOFTMAX, true>) : go(attend_umma_kernel<CKV_SOFTMAX, false>);
    return i16 ? go(attend_umma_kernel<CKV_SILU_OVER_L, true>) : go(attend_umma_kernel<CKV_SILU_OVER_L, false>);
}

}  // namespace ckv
