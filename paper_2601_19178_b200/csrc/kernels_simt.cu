// CUDA-core gather-concat-attention kernel (few queries per user) and the
// split-along-history combine.
//
// One thread block per (work item, group).  A pool row (head_dim elements, 64-256 B) is
// read by LPR adjacent lanes, 16 bytes each, so one warp-wide load instruction fetches
// 32/LPR whole rows with every sector fully used.  The user-specific leading d_user
// elements (Eq. K: user part first) are patched into the lane that owns them; K and V
// rows therefore only ever exist in registers.  Scores are reduced over the LPR lanes
// with shuffles, the softmax is the running-max form, and partial results of the
// sub-warps / warps / history chunks are merged with the usual (m, l, acc) rule.
// A side that is not shared (sharing only keys or only values) has its full-width rows in the
// arena: they are read in place of the pool rows, coalesced, and nothing is patched.  With
// visible lengths a query row only takes the positions before its own limit.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"
#include "ptx_helpers.cuh"

namespace ckv {
namespace {

constexpr int kWarps = 4;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint4 ldg16(const void* p)
{
    return __ldg(reinterpret_cast<const uint4*>(p));
}

template <bool BF16>
__device__ __forceinline__ void unpack16(const uint4& r, float* f)
{
    if constexpr (BF16) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else {
        f[0] = __uint_as_float(r.x);
        f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z);
        f[3] = __uint_as_float(r.w);
    }
}

template <bool BF16>
__device__ __forceinline__ float load_elem(const void* base, int64_t i)
{
    if constexpr (BF16)
        return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(base) + i) << 16);
    else
        return __ldg(reinterpret_cast<const float*>(base) + i);
}

// the user part of one unit (2, 4 or 8 bytes, naturally aligned) into the low end of 8 bytes
__device__ __forceinline__ uint2 load_user(const void* base, int64_t unit, int bytes)
{
    const char* p = reinterpret_cast<const char*>(base) + unit * bytes;
    uint2 r = make_uint2(0, 0);
    if (bytes == 8) r = __ldg(reinterpret_cast<const uint2*>(p));
    else if (bytes == 4) r.x = __ldg(reinterpret_cast<const uint32_t*>(p));
    else r.x = __ldg(reinterpret_cast<const uint16_t*>(p));
    return r;
}

__device__ __forceinline__ int load_idx(const void* base, int64_t unit, int idx_bytes)
{
    return idx_bytes == 2 ? (int)__ldg(reinterpret_cast<const uint16_t*>(base) + unit)
                          : __ldg(reinterpret_cast<const int32_t*>(base) + unit);
}

__device__ __forceinline__ void store_out(void* out, int64_t i, float v, int out_dtype)
{
    if (out_dtype == CKV_BF16)
        reinterpret_cast<__nv_bfloat16*>(out)[i] = __float2bfloat16_rn(v);
    else
        reinterpret_cast<float*>(out)[i] = v;
}

template <bool BF16, int D, int QB, int MODE>
__global__ void __launch_bounds__(kWarps * 32, QB == 1 ? 5 : 1) attend_simt_kernel(const AttendArgs a)
{
    constexpr int ES = BF16 ? 2 : 4;
    constexpr int EPL = 16 / ES;         // elements per lane
    constexpr int LPR = D / EPL;         // lanes per row
    constexpr int PPW = 32 / LPR;        // positions per warp-wide load
    constexpr int UNR = LPR >= 16 ? 2 : 4;
    static_assert(LPR >= 1 && LPR <= 32, "row must fit a warp");

    __shared__ float sm_m[kWarps][QB], sm_l[kWarps][QB];
    __shared__ float sm_acc[kWarps][QB][D];

    const Item it = a.items[blockIdx.x];
    const int g = blockIdx.y;
    const Req rq = a.reqs[it.req];
    const CacheView& cv = a.cv;
    const int G = cv.n_groups, d_user = cv.d_user, idx_bytes = cv.idx_bytes;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LPR, ch = lane % LPR;
    const int64_t unit0 = rq.base + (int64_t)g * rq.Lpad;
    const char* poolK = (const char*)cv.poolK + (int64_t)g * cv.n_entries * D * ES + ch * 16;
    const char* poolV = (const char*)cv.poolV + (int64_t)g * cv.n_entries * D * ES + ch * 16;
    const bool full_k = cv.full_k != 0, full_v = cv.full_v != 0;  // the side's rows are cached full width
    const char* rowsK = (const char*)cv.userK + ch * 16;
    const char* rowsV = (const char*)cv.userV + ch * 16;
    const bool owns_user = ch * EPL < d_user && !(full_k && full_v);
    // user part of a position in one load of at most 8 bytes: it fits the row's first lane and its size is a power of two
    const int user_bytes = d_user * ES;
    const bool wide_user = d_user <= EPL && (user_bytes == 2 || user_bytes == 4 || user_bytes == 8);
    const int chunk_end = it.begin + it.len;
    const float qscale = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 1.0f);

    for (int qb = 0; qb < rq.M; qb += QB) {
        float q[QB][EPL];
#pragma unroll
        for (int r = 0; r < QB; ++r) {
            if (qb + r < rq.M) {
                const int64_t row = (CKV_CLAMP((int64_t)(rq.q0 + qb + r), a.q_rows, a.err) * G + g) * D;
                unpack16<BF16>(ldg16((const char*)a.queries + (row + ch * EPL) * ES), q[r]);
#pragma unroll
                for (int e = 0; e < EPL; ++e) q[r][e] *= qscale;
            } else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) q[r][e] = 0.f;
            }
        }
        // positions query row r attends: [0, lim[r]); the block of rows stops at the largest limit
        int lim[QB], end = 0;
#pragma unroll
        for (int r = 0; r < QB; ++r) {
            lim[r] = 0;
            if (qb + r < rq.M) lim[r] = a.vis ? min(max(__ldg(a.vis + rq.q0 + qb + r), 0), rq.L) : rq.L;
            end = max(end, lim[r]);
        }
        end = min(end, chunk_end);
        float m_run[QB], l_run[QB], acc[QB][EPL];
#pragma unroll
        for (int r = 0; r < QB; ++r) {
            m_run[r] = -CUDART_INF_F;
            l_run[r] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[r][e] = 0.f;
        }

        // Coalesced loads of the compressed cache for the PPW * UNR positions of a step (lane l takes
        // positions l, l + 32, ...): the indices and, where a user part is one 2..16-byte word, the user
        // parts.  They are requested one step ahead: all of it streams from HBM, which takes several
        // times longer than a pool row takes from L2.
        constexpr int NL = (PPW * UNR + 31) / 32;
        int my_ik[NL], my_iv[NL];
        uint2 my_uk[NL], my_uv[NL];
        auto request_indices = [&](int p0) {
#pragma unroll
            for (int l = 0; l < NL; ++l) {
                const int my_p = p0 + l * 32 + lane;
                const int64_t my_unit = CKV_CLAMP(unit0 + ((l * 32 + lane < PPW * UNR && my_p < end) ? my_p : it.begin),
                                                  a.arena_units, a.err);
                my_ik[l] = full_k ? 0 : load_idx(cv.idxK, my_unit, idx_bytes);
                my_iv[l] = full_v ? 0 : load_idx(cv.idxV, my_unit, idx_bytes);
                my_uk[l] = my_uv[l] = make_uint2(0, 0);
                if (wide_user) {
                    if (!full_k) my_uk[l] = load_user(cv.userK, my_unit, user_bytes);
                    if (!full_v) my_uv[l] = load_user(cv.userV, my_unit, user_bytes);
                }
            }
        };
        if (it.begin + warp * (PPW * UNR) < end) request_indices(it.begin + warp * (PPW * UNR));
        for (int p0 = it.begin + warp * (PPW * UNR); p0 < end; p0 += kWarps * PPW * UNR) {
            int pos[UNR];
            uint4 kraw[UNR], vraw[UNR];
            int64_t unit[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                pos[j] = p0 + j * PPW + sub;
                unit[j] = CKV_CLAMP(unit0 + (pos[j] < end ? pos[j] : it.begin), a.arena_units, a.err);
            }
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const int src = (j * PPW) % 32 + sub;
                const int ik = CKV_CLAMP(__shfl_sync(0xffffffffu, my_ik[(j * PPW) / 32], src), cv.n_entries, a.err),
                          iv = CKV_CLAMP(__shfl_sync(0xffffffffu, my_iv[(j * PPW) / 32], src), cv.n_entries, a.err);
                kraw[j] = full_k ? ldg16(rowsK + unit[j] * (D * ES)) : ldg16(poolK + (int64_t)ik * (D * ES));
                vraw[j] = full_v ? ldg16(rowsV + unit[j] * (D * ES)) : ldg16(poolV + (int64_t)iv * (D * ES));
            }
            uint2 cur_uk[NL], cur_uv[NL];  // this step's user parts: the next request overwrites my_uk, my_uv
#pragma unroll
            for (int l = 0; l < NL; ++l) {
                cur_uk[l] = my_uk[l];
                cur_uv[l] = my_uv[l];
            }
            if (p0 + kWarps * PPW * UNR < end) request_indices(p0 + kWarps * PPW * UNR);
            float s[UNR][QB];
            float v[UNR][EPL];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                float k[EPL];
                unpack16<BF16>(kraw[j], k);
                unpack16<BF16>(vraw[j], v[j]);
                if (wide_user) {  // Eq. K: the first d_user dims come from the user part
                    // hand the position's user part to the lanes of its row (the first of them uses it)
                    const int src = (j * PPW) % 32 + sub;
                    uint4 ukj = make_uint4(0, 0, 0, 0), uvj = make_uint4(0, 0, 0, 0);
                    ukj.x = __shfl_sync(0xffffffffu, cur_uk[(j * PPW) / 32].x, src);
                    uvj.x = __shfl_sync(0xffffffffu, cur_uv[(j * PPW) / 32].x, src);
                    if (user_bytes > 4) {
                        ukj.y = __shfl_sync(0xffffffffu, cur_uk[(j * PPW) / 32].y, src);
                        uvj.y = __shfl_sync(0xffffffffu, cur_uv[(j * PPW) / 32].y, src);
                    }
                    if (owns_user) {
                        float ku[EPL], vu[EPL];
                        unpack16<BF16>(ukj, ku);
                        unpack16<BF16>(uvj, vu);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) {
                            if (e < d_user) {
                                if (!full_k) k[e] = ku[e];
                                if (!full_v) v[j][e] = vu[e];
                            }
                        }
                    }
                } else if (owns_user) {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) {
                        if (ch * EPL + e < d_user) {
                            const int64_t ui = unit[j] * d_user + ch * EPL + e;
                            if (!full_k) k[e] = load_elem<BF16>(cv.userK, ui);
                            if (!full_v) v[j][e] = load_elem<BF16>(cv.userV, ui);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < QB; ++r) {
                    float d = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) d = fmaf(q[r][e], k[e], d);
                    s[j][r] = d;
                }
            }
#pragma unroll
            for (int off = LPR / 2; off >= 1; off >>= 1)
#pragma unroll
                for (int j = 0; j < UNR; ++j)
#pragma unroll
                    for (int r = 0; r < QB; ++r)
                        s[j][r] += __shfl_xor_sync(0xffffffffu, s[j][r], off);

#pragma unroll
            for (int r = 0; r < QB; ++r) {
                if constexpr (MODE == CKV_SOFTMAX) {
                    float mn = m_run[r];
#pragma unroll
                    for (int j = 0; j < UNR; ++j)
                        if (pos[j] < min(end, lim[r])) mn = fmaxf(mn, s[j][r]);
                    const float ms = mn == -CUDART_INF_F ? 0.f : mn;
                    const float corr = exp2f(m_run[r] - ms);
                    m_run[r] = mn;
                    l_run[r] *= corr;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[r][e] *= corr;
#pragma unroll
                    for (int j = 0; j < UNR; ++j) {
                        const float p = pos[j] < min(end, lim[r]) ? exp2f(s[j][r] - ms) : 0.f;
                        l_run[r] += p;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) acc[r][e] = fmaf(p, v[j][e], acc[r][e]);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < UNR; ++j) {
                        const float x = s[j][r];
                        const float w = pos[j] < min(end, lim[r]) ? x / (1.0f + expf(-x)) : 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) acc[r][e] = fmaf(w, v[j][e], acc[r][e]);
                    }
                }
            }
        }

        // merge the sub-warps of this warp
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
            for (int r = 0; r < QB; ++r) {
                if constexpr (MODE == CKV_SOFTMAX) {
                    const float mo = __shfl_xor_sync(0xffffffffu, m_run[r], off);
                    const float lo = __shfl_xor_sync(0xffffffffu, l_run[r], off);
                    const float mn = fmaxf(m_run[r], mo);
                    const float ms = mn == -CUDART_INF_F ? 0.f : mn;
                    const float ca = exp2f(m_run[r] - ms), cb = exp2f(mo - ms);
                    l_run[r] = l_run[r] * ca + lo * cb;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) {
                        const float ao = __shfl_xor_sync(0xffffffffu, acc[r][e], off);
                        acc[r][e] = acc[r][e] * ca + ao * cb;
                    }
                    m_run[r] = mn;
                } else {
#pragma unroll
                    for (int e = 0; e < EPL; ++e)
                        acc[r][e] += __shfl_xor_sync(0xffffffffu, acc[r][e], off);
                }
            }
        }
        if (sub == 0) {
#pragma unroll
            for (int r = 0; r < QB; ++r) {
                if (ch == 0) {
                    sm_m[warp][r] = m_run[r];
                    sm_l[warp][r] = l_run[r];
                }
#pragma unroll
                for (int e = 0; e < EPL; ++e) sm_acc[warp][r][ch * EPL + e] = acc[r][e];
            }
        }
        __syncthreads();
        for (int t = threadIdx.x; t < QB * D; t += kWarps * 32) {
            const int r = t / D, c = t - r * D;
            if (qb + r >= rq.M) continue;
            float mt = -CUDART_INF_F, lt = 0.f, o = 0.f;
            if constexpr (MODE == CKV_SOFTMAX) {
#pragma unroll
                for (int w = 0; w < kWarps; ++w) mt = fmaxf(mt, sm_m[w][r]);
                const float ms = mt == -CUDART_INF_F ? 0.f : mt;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) {
                    const float cw = exp2f(sm_m[w][r] - ms);
                    lt += sm_l[w][r] * cw;
                    o += sm_acc[w][r][c] * cw;
                }
            } else {
#pragma unroll
                for (int w = 0; w < kWarps; ++w) o += sm_acc[w][r][c];
            }
            if (it.part_row < 0) {
                float res;
                if constexpr (MODE == CKV_SOFTMAX) res = lt > 0.f ? o / lt : 0.f;
                else res = rq.L > 0 ? o / (float)rq.L : 0.f;
                store_out(a.out, (CKV_CLAMP((int64_t)(rq.q0 + qb + r), a.q_rows, a.err) * G + g) * D + c, res, a.out_dtype);
            } else {
                float* pr = a.partials + (CKV_CLAMP((int64_t)(it.part_row + qb + r), a.part_rows, a.err) * G + g) * (D + 2);
                if (c == 0) {
                    pr[0] = mt;
                    pr[1] = lt;
                }
                pr[2 + c] = o;
            }
        }
        __syncthreads();
    }
}

// One block per (split request, group): out = merge over the request's chunks.
template <int MODE>
__global__ void __launch_bounds__(128) combine_kernel(const AttendArgs a, const int32_t* split_reqs,
                                                      int D)
{
    const Req rq = a.reqs[split_reqs[blockIdx.x]];
    const int g = blockIdx.y, G = a.cv.n_groups;
    const int W = D + 2;
    for (int t = threadIdx.x; t < rq.M * D; t += blockDim.x) {
        const int r = t / D, c = t - r * D;
        float res;
        if constexpr (MODE == CKV_SOFTMAX) {
            float mt = -CUDART_INF_F;
            for (int k = 0; k < rq.n_chunks; ++k)
                mt = fmaxf(mt, a.partials[(CKV_CLAMP((int64_t)(rq.part0 + k * rq.M + r), a.part_rows, a.err) * G + g) * W]);
            const float ms = mt == -CUDART_INF_F ? 0.f : mt;
            float lt = 0.f, o = 0.f;
            for (int k = 0; k < rq.n_chunks; ++k) {
                const float* pr = a.partials + ((int64_t)(rq.part0 + k * rq.M + r) * G + g) * W;
                const float ck = exp2f(pr[0] - ms);
                lt += pr[1] * ck;
                o += pr[2 + c] * ck;
            }
            res = lt > 0.f ? o / lt : 0.f;
        } else {
            float o = 0.f;
            for (int k = 0; k < rq.n_chunks; ++k)
                o += a.partials[((int64_t)(rq.part0 + k * rq.M + r) * G + g) * W + 2 + c];
            res = rq.L > 0 ? o / (float)rq.L : 0.f;
        }
        store_out(a.out, (CKV_CLAMP((int64_t)(rq.q0 + r), a.q_rows, a.err) * G + g) * D + c, res, a.out_dtype);
    }
}

template <bool BF16, int D>
cudaError_t launch_simt_d(const AttendArgs& a, int max_M, cudaStream_t s)
{
    const dim3 grid(a.n_items, a.cv.n_groups), block(kWarps * 32);
    const bool sm = a.mode == CKV_SOFTMAX;
    if (max_M <= 1) {
        if (sm) attend_simt_kernel<BF16, D, 1, CKV_SOFTMAX><<<grid, block, 0, s>>>(a);
        else attend_simt_kernel<BF16, D, 1, CKV_SILU_OVER_L><<<grid, block, 0, s>>>(a);
    } else {
        if (sm) attend_simt_kernel<BF16, D, 4, CKV_SOFTMAX><<<grid, block, 0, s>>>(a);
        else attend_simt_kernel<BF16, D, 4, CKV_SILU_OVER_L><<<grid, block, 0, s>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attend_simt(int dtype, int D, int max_M, const AttendArgs& a, cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    const bool bf = dtype == CKV_BF16;
    switch (D) {
        case 16: return bf ? launch_simt_d<true, 16>(a, max_M, s) : launch_simt_d<false, 16>(a, max_M, s);
        case 32: return bf ? launch_simt_d<true, 32>(a, max_M, s) : launch_simt_d<false, 32>(a, max_M, s);
        case 64: return bf ? launch_simt_d<true, 64>(a, max_M, s) : launch_simt_d<false, 64>(a, max_M, s);
        case 128: return bf ? launch_simt_d<true, 128>(a, max_M, s) : launch_simt_d<false, 128>(a, max_M, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_combine(int D, const AttendArgs& a, const int32_t* split_reqs, int n_split,
                           cudaStream_t s)
{
    if (n_split == 0) return cudaSuccess;
    const dim3 grid(n_split, a.cv.n_groups);
    if (a.mode == CKV_SOFTMAX) combine_kernel<CKV_SOFTMAX><<<grid, 128, 0, s>>>(a, split_reqs, D);
    else combine_kernel<CKV_SILU_OVER_L><<<grid, 128, 0, s>>>(a, split_reqs, D);
    return cudaGetLastError();
}

}  // namespace ckv
