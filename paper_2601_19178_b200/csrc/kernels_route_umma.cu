// Prefill router (Sec. 4.3) on the tcgen05 tensor cores: I[i][g] = lowest j maximising x_i . W_g[j] + b_g[j].
//
// One CTA owns 256 positions of one group, as two blocks of 128.  Their inputs sit in shared memory once (A operand,
// K-major core-matrix layout); the group's weight rows stream through a four-stage ring in tiles of 128 entries
// (B operand, same layout, 16-byte cp.async by four producer warps, each bound to one stage), and every tile is
// multiplied with both blocks, which halves the weight traffic out of L2 per product.  One thread issues the two
// 128 x 128 x d_in products of a tile into the tile's two TMEM accumulators (two per block, alternating: all 512
// columns); two groups of four warps, one per block (thread = position = TMEM lane), read their accumulator, add
// the bias, and keep a running (best score, entry) in registers, so the score matrix never leaves the SM.
// Every wait is bounded: a time-out raises the CTA's abort flag, the CTA drains, frees its TMEM, reports through
// the error word and writes nothing.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"

namespace ckv {
namespace {

constexpr int kRows = 256, kTileN = 128, kMaxStages = 4, kBiasSlots = 8;
constexpr int kEpiWarps = 8, kIssueWarp = 8, kProdWarp0 = 9, kProdWarps = 4;
constexpr int kThreadsRU = (kProdWarp0 + kProdWarps) * 32;
constexpr uint32_t kSpin = 1u << 18, kSuspend = 4000;
enum { ERR_ROUTE = 64 };

// B_AFULL / B_AEMPTY: [2 * block + buffer]
enum Bar { B_FULL = 0, B_EMPTY = kMaxStages, B_AFULL = 2 * kMaxStages, B_AEMPTY = 2 * kMaxStages + 4, B_DRAIN = 2 * kMaxStages + 8, B_COUNT };

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __noinline__ bool bar_wait(uint32_t bar, uint32_t parity, const volatile int* abort_flag)
{
    for (uint32_t i = 0; i < kSpin; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kSuspend)
            : "memory");
        if (ok) return true;
        if ((i & 31u) == 31u && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ void fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit_to(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
// shared-memory matrix descriptor, no swizzle: start address, leading / stride byte offsets (16-byte units), version 1
__device__ __forceinline__ uint64_t mat_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46);
}
// instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, both K-major
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void ld32(uint32_t taddr, uint32_t (&r)[32])
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
__device__ __forceinline__ void wait_ld32(uint32_t (&r)[32])
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
__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// 16-byte copy global -> shared; src_bytes = 0 fills the destination with zeros instead
__device__ __forceinline__ void cp16(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

template <int DIN>
struct RU {
    static constexpr int CPR = DIN / 8;              // 16-byte chunks per row
    static constexpr int SBO = CPR * 128;            // bytes per group of 8 rows
    static constexpr int XTILE = kRows * DIN * 2;    // bytes of the positions' tile
    static constexpr int TILE = kTileN * DIN * 2;    // bytes of a weight tile
    static constexpr int STAGES = 4;
    static constexpr int PPT = kProdWarps / STAGES;  // producer warps that share one tile (each stage has its own warps)
    static constexpr int OFF_X = 0, OFF_W = XTILE, OFF_BIAS = OFF_W + STAGES * TILE,
                         OFF_BAR = OFF_BIAS + kBiasSlots * kTileN * 4,
                         OFF_ABORT = OFF_BAR + 24 * 8, SMEM = OFF_ABORT + 16;
};
// byte offset of (row r, 16-byte chunk c) in the K-major core-matrix layout: 8 x 16-byte core matrices, chunks of a
// row group 128 bytes apart, row groups SBO apart
template <int DIN>
__device__ __forceinline__ uint32_t tile_off(int r, int c)
{
    return (uint32_t)((r >> 3) * RU<DIN>::SBO + c * 128 + (r & 7) * 16);
}

template <int DIN>
__global__ void __launch_bounds__(kThreadsRU, 1)
    route_umma_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ W, const float* __restrict__ bias, int n,
                      int m, int G, int32_t* __restrict__ out, int* __restrict__ err_flag)
{
    using L = RU<DIN>;
    extern __shared__ __align__(1024) unsigned char usm[];
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sb = s_u32(usm);
    auto bar = [&](int i) { return sb + L::OFF_BAR + 8u * (uint32_t)i; };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(usm + L::OFF_ABORT);
    const int grp = blockIdx.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const uint16_t* Wg = W + (int64_t)grp * m * DIN;
    const float* bg = bias ? bias + (int64_t)grp * m : nullptr;
    const int n_tiles = (m + kTileN - 1) / kTileN;

    if (tid == 0) {
        for (int s = 0; s < L::STAGES; ++s) {
            bar_init(bar(B_FULL + s), L::PPT);
            bar_init(bar(B_EMPTY + s), 1);
        }
        for (int e = 0; e < 4; ++e) {
            bar_init(bar(B_AFULL + e), 1);
            bar_init(bar(B_AEMPTY + e), 128);
        }
        bar_init(bar(B_DRAIN), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kIssueWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_u32(&tmem_slot)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the positions' inputs, once: row r of the tile is position row0 + r (zero rows past the end)
    for (int q = tid; q < kRows * L::CPR; q += kThreadsRU) {
        const int r = (q & 7) + 8 * (q / (8 * L::CPR)), c = (q >> 3) % L::CPR;
        const bool in = row0 + r < n;
        cp16(sb + L::OFF_X + tile_off<DIN>(r, c), x + (in ? (row0 + r) * DIN + c * 8 : 0), in ? 16u : 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_async();
    tc_before();
    __syncthreads();
    tc_after();
    const uint32_t tmem = tmem_slot;
    bool ok = true;

    if (warp < kEpiWarps) {
        // ------------------------------------------------------------ running arg-max, thread = position
        const int e = warp >> 2, row = 128 * e + (warp & 3) * 32 + lane;  // block e, position row of the CTA
        const uint32_t tacc0 = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(2 * kTileN * e);
        float best = -CUDART_INF_F;
        int arg = 0;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int a = t & 1;
            ok = bar_wait(bar(B_AFULL + 2 * e + a), (t >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_after();
            const uint32_t tacc = tacc0 + (uint32_t)(kTileN * a);
            const float4* bs = reinterpret_cast<const float4*>(usm + L::OFF_BIAS) + (t % kBiasSlots) * (kTileN / 4);
            const int j0 = t * kTileN;
            // 32 columns at a time, the next 32 already on their way out of TMEM.  Only the maximum of a block is
            // compared with the running best (a new best gets rare quickly); the block is searched for its first
            // maximal column only then.  Entries come in increasing order and the comparison is strict, so the
            // lowest entry wins among equals; past the last entry the bias slot holds -inf.
            uint32_t va[32], vb[32];
            ld32(tacc, va);
            auto block = [&](uint32_t (&v)[32], int c4) {
                float f[32];
#pragma unroll
                for (int k = 0; k < 32; k += 4) {
                    const float4 b4 = bs[8 * c4 + (k >> 2)];
                    f[k] = __uint_as_float(v[k]) + b4.x;
                    f[k + 1] = __uint_as_float(v[k + 1]) + b4.y;
                    f[k + 2] = __uint_as_float(v[k + 2]) + b4.z;
                    f[k + 3] = __uint_as_float(v[k + 3]) + b4.w;
                }
                float mx = f[0];
#pragma unroll
                for (int k = 1; k + 1 < 32; k += 2) mx = max3f(mx, f[k], f[k + 1]);
                mx = fmaxf(mx, f[31]);
                if (mx > best) {
                    best = mx;
                    int first = 31;
#pragma unroll
                    for (int k = 30; k >= 0; --k) first = f[k] == mx ? k : first;
                    arg = j0 + 32 * c4 + first;
                }
            };
#pragma unroll 1
            for (int c4 = 0; c4 < kTileN / 32; c4 += 2) {
                wait_ld32(va);
                ld32(tacc + 32 * (c4 + 1), vb);
                block(va, c4);
                wait_ld32(vb);
                if (c4 + 2 < kTileN / 32) ld32(tacc + 32 * (c4 + 2), va);
                block(vb, c4 + 1);
            }
            tc_before();
            bar_arrive(bar(B_AEMPTY + 2 * e + a));
        }
        if (ok && !*abort_flag && row0 + row < n) out[(row0 + row) * G + grp] = arg;
        if (!ok) *abort_flag = 1;
    } else if (warp == kIssueWarp) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, kTileN);
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int s = t % L::STAGES, a = t & 1;
                ok = bar_wait(bar(B_FULL + s), (t / L::STAGES) & 1, abort_flag);
                for (int e = 0; e < 2 && ok; ++e) {
                    if (t >= 2) ok = bar_wait(bar(B_AEMPTY + 2 * e + a), ((t >> 1) - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_after();
#pragma unroll
                    for (int ks = 0; ks < DIN / 16; ++ks)
                        mma_ss(tmem + (uint32_t)(kTileN * (2 * e + a)),
                               mat_desc(sb + L::OFF_X + e * 16 * L::SBO + ks * 256, 128, L::SBO),
                               mat_desc(sb + L::OFF_W + s * L::TILE + ks * 256, 128, L::SBO), idesc, ks > 0 ? 1u : 0u);
                    tc_commit_to(bar(B_AFULL + 2 * e + a));
                }
                if (!ok) break;
                tc_commit_to(bar(B_EMPTY + s));
            }
            if (!ok) *abort_flag = 1;
            // nothing of this CTA may still run on the tensor core at teardown
            tc_commit_to(bar(B_DRAIN));
            volatile int never = 0;
            if (!bar_wait(bar(B_DRAIN), 0, &never)) *abort_flag = 1;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ producers
        // warp p works for stage p % STAGES only (its waits on that stage's barriers are then in phase order) and
        // copies part p / STAGES of each of that stage's tiles
        const int p = warp - kProdWarp0, part = p / L::STAGES;
        constexpr int kPartRows = kTileN / L::PPT;
        float* bias_s = reinterpret_cast<float*>(usm + L::OFF_BIAS);
        for (int t = p % L::STAGES; t < n_tiles && ok; t += L::STAGES) {
            const int s = t % L::STAGES, j0 = t * kTileN;
            if (t >= L::STAGES) ok = bar_wait(bar(B_EMPTY + s), ((t / L::STAGES) - 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t dst = sb + L::OFF_W + s * L::TILE;
            for (int q = lane; q < kPartRows * L::CPR; q += 32) {
                const int r = part * kPartRows + (q & 7) + 8 * (q / (8 * L::CPR)), c = (q >> 3) % L::CPR;
                const int j = min(j0 + r, m - 1);
                cp16(dst + tile_off<DIN>(r, c), Wg + (int64_t)j * DIN + c * 8, 16u);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            for (int k = part * kPartRows + lane; k < (part + 1) * kPartRows; k += 32) {
                const int j = j0 + k;
                bias_s[(t % kBiasSlots) * kTileN + k] = j < m ? (bg ? __ldg(bg + j) : 0.f) : -CUDART_INF_F;
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            fence_async();  // the copies of this lane are visible to the tensor core's proxy
            __syncwarp();
            if (lane == 0) bar_arrive(bar(B_FULL + s));
        }
        if (!ok) *abort_flag = 1;
    }
    tc_before();
    __syncthreads();
    tc_after();
    if (warp == kIssueWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    if (tid == 0 && *abort_flag) atomicOr(err_flag, ERR_ROUTE);
}

template <int DIN>
cudaError_t launch_t(const void* x, const void* W, const float* bias, int n, int m, int G, int32_t* out, int* err_flag,
                     cudaStream_t s)
{
    cudaError_t e = cudaFuncSetAttribute(route_umma_kernel<DIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, RU<DIN>::SMEM);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((n + kRows - 1) / kRows), (unsigned)G);
    route_umma_kernel<DIN><<<grid, kThreadsRU, RU<DIN>::SMEM, s>>>((const uint16_t*)x, (const uint16_t*)W, bias, n, m, G,
                                                                   out, err_flag);
    return cudaGetLastError();
}

}  // namespace

// err_flag: device int, OR-ed with a non-zero code if a bounded wait inside the kernel ran out (nothing is written then).
cudaError_t launch_route_umma(int d_in, const void* x, const void* W, const float* bias, int n, int n_entries, int G,
                              int32_t* out, int* err_flag, cudaStream_t s)
{
    if (n == 0) return cudaSuccess;
    switch (d_in) {
        case 32: return launch_t<32>(x, W, bias, n, n_entries, G, out, err_flag, s);
        case 64: return launch_t<64>(x, W, bias, n, n_entries, G, out, err_flag, s);
        default: return launch_t<128>(x, W, bias, n, n_entries, G, out, err_flag, s);
    }
}

}  // namespace ckv
