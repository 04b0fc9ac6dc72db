// Prefill router (Sec. 4.3): which global-pool entry a history position selects,
//     I[i][g] = argmin { j : M_ij maximal },   M = X W_g^T + b_g,
// for n positions with d_in-wide inputs X (bf16), per group g a weight matrix W_g stored entry-major
// ([n_entries][d_in] bf16: an entry's weights are contiguous, like a pool row) and an optional fp32 bias.
// The score matrix M (n x n_entries) is never written: every warp keeps the running best (value, entry) of its
// rows in registers while the entries stream through shared memory.
//
// One CTA = 8 warps x 32 positions; the positions' inputs stay in registers as m16n8k16 A fragments.  The group's
// weight rows go through a two-slot shared-memory ring in chunks of 64 entries (cp.async by the whole CTA, rows
// swizzled for ldmatrix), each chunk used by all eight warps.  Products are exact (bf16 x bf16), sums fp32.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"
#include "ptx_helpers.cuh"

namespace ckv {
namespace {

constexpr int kRouteWarps = 8, kRouteChunk = 64;
// 16-position tiles per warp: every weight fragment read from shared memory serves that many MMAs
__host__ __device__ constexpr int route_mt(int) { return 2; }  // (four measured no faster: 334 against 342 TFLOP/s)
__host__ __device__ constexpr int route_rows(int d_in) { return kRouteWarps * 16 * route_mt(d_in); }  // positions per CTA

// 16-byte chunk c of ring row r sits at chunk c ^ swz(r): the eight rows of an ldmatrix block (consecutive
// entries) fall into eight different bank groups
template <int DIN>
__device__ __forceinline__ int swz(int r)
{
    return DIN == 32 ? ((r >> 1) & 3) : (r & 7);
}

template <int DIN>
__global__ void __launch_bounds__(kRouteWarps * 32)
    route_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ W, const float* __restrict__ bias, int n,
                 int m, int G, int32_t* __restrict__ out)
{
    constexpr int KS = DIN / 16, MT = route_mt(DIN), ROWB = DIN * 2, CPR = ROWB / 16, CH = kRouteChunk;
    constexpr int SLOT_B = CH * ROWB;
    extern __shared__ __align__(128) unsigned char rsm[];
    float* bias_s = reinterpret_cast<float*>(rsm + 2 * SLOT_B);  // [2][CH]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gl = lane >> 2, t = lane & 3;
    const int grp = blockIdx.y;
    const int64_t row0 = (int64_t)blockIdx.x * route_rows(DIN) + warp * (16 * MT);
    const uint16_t* Wg = W + (int64_t)grp * m * DIN;
    const float* bg = bias ? bias + (int64_t)grp * m : nullptr;

    uint32_t qa[MT][KS][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int64_t r_lo = row0 + 16 * mt + gl, r_hi = r_lo + 8;
        const uint16_t* p_lo = x + r_lo * DIN;
        const uint16_t* p_hi = x + r_hi * DIN;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int c = 16 * ks + 2 * t;
            qa[mt][ks][0] = r_lo < n ? __ldg(reinterpret_cast<const uint32_t*>(p_lo + c)) : 0u;
            qa[mt][ks][1] = r_hi < n ? __ldg(reinterpret_cast<const uint32_t*>(p_hi + c)) : 0u;
            qa[mt][ks][2] = r_lo < n ? __ldg(reinterpret_cast<const uint32_t*>(p_lo + c + 8)) : 0u;
            qa[mt][ks][3] = r_hi < n ? __ldg(reinterpret_cast<const uint32_t*>(p_hi + c + 8)) : 0u;
        }
    }
    float bv[MT][2];
    int bi[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        bv[mt][0] = bv[mt][1] = -CUDART_INF_F;
        bi[mt][0] = bi[mt][1] = 0;
    }

    const uint32_t ring = smem_u32(rsm);
    auto stage = [&](int c) {  // entries 64 c .. 64 c + 63 into slot c & 1 (past the last entry: the last row, bias -inf)
        const int slot = c & 1, j0 = c * CH;
        for (int q = tid; q < CH * CPR; q += kRouteWarps * 32) {
            const int r = q / CPR, cc = q - r * CPR;
            const int j = min(j0 + r, m - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring + slot * SLOT_B + r * ROWB +
                                                                          ((cc ^ swz<DIN>(r)) << 4)),
                         "l"(Wg + (int64_t)j * DIN + cc * 8)
                         : "memory");
        }
        if (tid < CH) {
            const int j = j0 + tid;
            bias_s[slot * CH + tid] = j < m ? (bg ? __ldg(bg + j) : 0.f) : -CUDART_INF_F;
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // ldmatrix row addresses of this lane: matrix lane >> 3 = 16-byte chunk within a k-step pair, row lane & 7
    const int lr = lane & 7, lm = lane >> 3;
    uint32_t offB[KS / 2];
#pragma unroll
    for (int kp = 0; kp < KS / 2; ++kp) offB[kp] = lr * ROWB + ((((4 * kp + lm) ^ swz<DIN>(lr)) & (CPR - 1)) << 4);

    const int nch = (m + CH - 1) / CH;
    stage(0);
    for (int c = 0; c < nch; ++c) {
        if (c + 1 < nch) {
            stage(c + 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const uint32_t wt = ring + (c & 1) * SLOT_B;
        const float* bs = bias_s + (c & 1) * CH;
#pragma unroll 2
        for (int nt = 0; nt < CH / 8; ++nt) {
            uint32_t b[KS][2];
#pragma unroll
            for (int kp = 0; kp < KS / 2; ++kp)
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b[2 * kp][0]), "=r"(b[2 * kp][1]), "=r"(b[2 * kp + 1][0]), "=r"(b[2 * kp + 1][1])
                             : "r"(wt + nt * (8 * ROWB) + offB[kp])
                             : "memory");
            const int j = c * CH + 8 * nt + 2 * t;  // entries of this lane's two accumulator columns
            const float b0 = bs[8 * nt + 2 * t], b1 = bs[8 * nt + 2 * t + 1];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) mma_bf16(acc, qa[mt][ks], b[ks][0], b[ks][1]);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float v0 = acc[2 * h] + b0, v1 = acc[2 * h + 1] + b1;
                    // entries arrive in increasing order: a strict comparison keeps the lowest entry among equals;
                    // a new best gets rare quickly, so one test of the pair's maximum guards the update
                    if (fmaxf(v0, v1) > bv[mt][h]) {
                        const bool first = v0 >= v1;
                        bv[mt][h] = first ? v0 : v1;
                        bi[mt][h] = first ? j : j + 1;
                    }
                }
            }
        }
        __syncthreads();  // everyone is done with this slot before the chunk after next is staged into it
    }
    // the four lanes of a row hold disjoint entries: best of them, lowest entry among equals
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float v = bv[mt][h];
            int i = bi[mt][h];
#pragma unroll
            for (int o = 1; o <= 2; o <<= 1) {
                const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
                const int i2 = __shfl_xor_sync(0xffffffffu, i, o);
                if (v2 > v || (v2 == v && i2 < i)) {
                    v = v2;
                    i = i2;
                }
            }
            const int64_t r = row0 + 16 * mt + gl + 8 * h;
            if (t == 0 && r < n) out[r * G + grp] = i;
        }
}

template <int DIN>
cudaError_t launch_route_t(const void* x, const void* W, const float* bias, int n, int m, int G, int32_t* out,
                           cudaStream_t s)
{
    const size_t smem = 2 * (size_t)kRouteChunk * DIN * 2 + 2 * kRouteChunk * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(route_kernel<DIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((n + route_rows(DIN) - 1) / route_rows(DIN)), (unsigned)G);
    route_kernel<DIN><<<grid, kRouteWarps * 32, smem, s>>>((const uint16_t*)x, (const uint16_t*)W, bias, n, m, G, out);
    return cudaGetLastError();
}

// User-specific low-dimensional projection of the prefill (Sec. 4.2): y[i][g][c] = x_i . W[g][c] + b[g][c],
// d_out <= 16 outputs per group.  Memory-bound: one thread per output element, the weights in shared memory
// (rows padded by 16 bytes against bank conflicts), 16-byte loads of the input row, fp32 sums, bf16 result.
__global__ void __launch_bounds__(256) project_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ W,
                                                      const float* __restrict__ bias, int64_t total, int d_in, int gd,
                                                      uint16_t* __restrict__ out)
{
    extern __shared__ __align__(16) unsigned char psm[];
    const int wrow = d_in * 2 + 16;  // bytes per padded weight row
    for (int q = threadIdx.x; q < gd * (d_in / 8); q += blockDim.x) {
        const int r = q / (d_in / 8), c = q - r * (d_in / 8);
        *reinterpret_cast<uint4*>(psm + r * wrow + c * 16) = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)r * d_in) + c);
    }
    __syncthreads();
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / gd;
        const int r = (int)(e - i * gd);  // (group, output) row of W
        const uint4* xr = reinterpret_cast<const uint4*>(x + i * d_in);
        const unsigned char* wr = psm + r * wrow;
        float acc = bias ? __ldg(bias + r) : 0.f;
        for (int c = 0; c < d_in / 8; ++c) {
            const uint4 a = __ldg(xr + c), b = *reinterpret_cast<const uint4*>(wr + c * 16);
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc = fmaf(__uint_as_float(aw[k] << 16), __uint_as_float(bw[k] << 16), acc);
                acc = fmaf(__uint_as_float(aw[k] & 0xffff0000u), __uint_as_float(bw[k] & 0xffff0000u), acc);
            }
        }
        out[e] = __bfloat16_as_ushort(__float2bfloat16_rn(acc));
    }
}

}  // namespace

bool route_supported(int d_in) { return d_in == 32 || d_in == 64 || d_in == 128; }

cudaError_t launch_route(int d_in, const void* x, const void* W, const float* bias, int n, int n_entries, int G,
                         int32_t* out, cudaStream_t s)
{
    if (n == 0) return cudaSuccess;
    switch (d_in) {
        case 32: return launch_route_t<32>(x, W, bias, n, n_entries, G, out, s);
        case 64: return launch_route_t<64>(x, W, bias, n, n_entries, G, out, s);
        default: return launch_route_t<128>(x, W, bias, n, n_entries, G, out, s);
    }
}

bool project_supported(int d_in, int d_out, int n_groups)
{
    return d_in >= 8 && d_in <= 256 && d_in % 8 == 0 && d_out >= 1 && d_out <= 16 &&
           (size_t)n_groups * d_out * (d_in * 2 + 16) <= 96 * 1024;
}

cudaError_t launch_project(int d_in, int d_out, int G, const void* x, const void* W, const float* bias, int64_t n,
                           void* out, cudaStream_t s)
{
    if (n == 0) return cudaSuccess;
    const int gd = G * d_out;
    const size_t smem = (size_t)gd * (d_in * 2 + 16);
    cudaError_t e = cudaFuncSetAttribute(project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total = n * gd;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    project_kernel<<<(unsigned)blocks, 256, smem, s>>>((const uint16_t*)x, (const uint16_t*)W, bias, total, d_in, gd,
                                                       (uint16_t*)out);
    return cudaGetLastError();
}

}  // namespace ckv
