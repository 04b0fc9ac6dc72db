// Pool-side factorisation of the gather for one query per user (bf16, head_dim 32 or 64).
//
// With a single query q per (user, group) the gathered rows are only ever used in two sums:
//     score_i  = q_u . K_u[i] + q_g . P_k[I_k[i]]            = q_u . K_u[i] + T[I_k[i]],  T = P_k q_g
//     out_g    = sum_i p_i P_v[I_v[i]]                       = sum_j w[j] P_v[j],       w[j] = sum_{i: I_v[i] = j} p_i
// (Eq. K / Eq. Kc with the user part first; q_u, q_g the user and shared slices of q).  T for all users is
// one dense product with the K pool, the output one dense product of the weight histograms w with the V pool;
// per position only two 4-byte table accesses remain instead of two gathered pool rows.  Same mathematics as
// the gathering kernels, another summation order.  It pays when histories are long compared with the pool
// (tables cost 2 x n_entries x 4 bytes per (user, group) to HBM and back) -- the caller decides.
//
// Three launches:
//   fact_table_kernel  T[r][g][j] = q_r . P_k[g][j]          m16n8k16 MMAs, fp32 out
//   fact_main_kernel   persistent CTAs over the (user, group) pairs: T row into shared memory, scores, max, weights, histogram w,
//                      user-part output and row sum; w takes T's place in shared memory and in HBM
//   fact_out_kernel    out[r][g][:] = (w[r][g] P_v[g] + user part) / l          MMAs, w in bf16
#include <cuda_bf16.h>
#include <math_constants.h>

#include <algorithm>

#include "ckv_internal.h"
#include "ptx_helpers.cuh"

namespace ckv {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMainThreads = 1024;
constexpr int kOutWarps = 16;

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }
// ------------------------------------------------------------------------------------------------ T = P_k q
// T / w rows in HBM are this many floats apart: 32-byte aligned rows, room for zero-filled bf16 pairs up to a
// multiple of 8 entries
__host__ __device__ __forceinline__ int row_floats(int n_entries) { return (n_entries + 7) & ~7; }

constexpr int kTableMT = 4;  // 16-request tiles per warp: every pool row fetched serves 64 requests

template <int D>
__global__ void __launch_bounds__(128) fact_table_kernel(const AttendArgs a, int n_req, float* __restrict__ tw)
{
    constexpr int KS = D / 16, MT = kTableMT;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gl = lane >> 2, t = lane & 3;
    const int m = a.cv.n_entries, G = a.cv.n_groups, grp = blockIdx.z;
    const int j0 = blockIdx.x * 256 + warp * 64, r0 = blockIdx.y * (16 * MT);
    if (j0 >= m) return;
    // Which feature sits in which k-slot of the MMA is free as long as Q and the pool rows agree: a lane reads
    // D / 4 contiguous bytes of "its" rows, and k-step ks, slots (2t, 2t+1, 2t+8, 2t+9) hold features
    // (D / 4) t + 4 ks + (0, 1, 2, 3).
    constexpr int W = D / 8;  // 32-bit words per lane and row
    const uint16_t* Q = reinterpret_cast<const uint16_t*>(a.queries);
    uint32_t qa[MT][KS][4];
    bool v_lo[MT], v_hi[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int r_lo = r0 + 16 * mt + gl, r_hi = r_lo + 8;
        v_lo[mt] = r_lo < n_req && a.reqs[r_lo].M > 0;
        v_hi[mt] = r_hi < n_req && a.reqs[r_hi].M > 0;
        uint32_t q_lo[W], q_hi[W];
#pragma unroll
        for (int h = 0; h < W / 4; ++h) {
            uint4 x = make_uint4(0, 0, 0, 0), y = x;
            if (v_lo[mt])
                x = __ldg(reinterpret_cast<const uint4*>(Q + ((int64_t)a.reqs[r_lo].q0 * G + grp) * D + 2 * W * t) + h);
            if (v_hi[mt])
                y = __ldg(reinterpret_cast<const uint4*>(Q + ((int64_t)a.reqs[r_hi].q0 * G + grp) * D + 2 * W * t) + h);
            q_lo[4 * h] = x.x; q_lo[4 * h + 1] = x.y; q_lo[4 * h + 2] = x.z; q_lo[4 * h + 3] = x.w;
            q_hi[4 * h] = y.x; q_hi[4 * h + 1] = y.y; q_hi[4 * h + 2] = y.z; q_hi[4 * h + 3] = y.w;
        }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[mt][ks][0] = q_lo[2 * ks];
            qa[mt][ks][1] = q_hi[2 * ks];
            qa[mt][ks][2] = q_lo[2 * ks + 1];
            qa[mt][ks][3] = q_hi[2 * ks + 1];
        }
    }
    const uint16_t* P = reinterpret_cast<const uint16_t*>(a.cv.poolK) + (int64_t)grp * m * D;
    const int ms = row_floats(m);
#pragma unroll 2
    for (int nt = 0; nt < 8; ++nt) {
        const int jb = j0 + 8 * nt + gl;  // pool entry whose row is this lane's B column
        const uint4* row = reinterpret_cast<const uint4*>(P + (int64_t)(jb < m ? jb : m - 1) * D + 2 * W * t);
        uint32_t pw[W];
#pragma unroll
        for (int h = 0; h < W / 4; ++h) {
            const uint4 x = __ldg(row + h);
            pw[4 * h] = x.x; pw[4 * h + 1] = x.y; pw[4 * h + 2] = x.z; pw[4 * h + 3] = x.w;
        }
        const int jc = j0 + 8 * nt + 2 * t;  // columns of the accumulator fragment
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) mma_bf16(c, qa[mt][ks], pw[2 * ks], pw[2 * ks + 1]);
            float* t_lo = tw + ((int64_t)(r0 + 16 * mt + gl) * G + grp) * ms;
            float* t_hi = t_lo + (int64_t)8 * G * ms;
            // the two columns of a lane are one aligned 8-byte store (a column past the last entry lands in the row's padding)
            if (v_lo[mt] && jc < m) *reinterpret_cast<float2*>(t_lo + jc) = make_float2(c[0], c[1]);
            if (v_hi[mt] && jc < m) *reinterpret_cast<float2*>(t_hi + jc) = make_float2(c[2], c[3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------ main
template <bool IDX16>
__device__ __forceinline__ int load_index(const void* base, int64_t unit)
{
    if constexpr (IDX16) return __ldg(reinterpret_cast<const uint16_t*>(base) + unit);
    else return __ldg(reinterpret_cast<const int32_t*>(base) + unit);
}

// user part of one position (d_user <= 8 bf16 elements) as raw bits, two elements per word
__device__ __forceinline__ uint4 load_user(const uint16_t* u, int64_t unit, int d_user)
{
    uint4 r = make_uint4(0, 0, 0, 0);
    switch (d_user) {
        case 0: break;
        case 1: r.x = __ldg(u + unit); break;
        case 2: r.x = __ldg(reinterpret_cast<const uint32_t*>(u + unit * 2)); break;
        case 4: {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(u + unit * 4));
            r.x = w.x;
            r.y = w.y;
            break;
        }
        case 8: r = __ldg(reinterpret_cast<const uint4*>(u + unit * 8)); break;
        default: {
            uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e < d_user) w[e >> 1] |= (uint32_t)__ldg(u + unit * d_user + e) << (16 * (e & 1));
            r = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    return r;
}
// acc + sum_e c[e] * x[e]
__device__ __forceinline__ float dot_user(const float (&c)[8], const uint4& x, float acc)
{
    acc = fmaf(c[0], bf16_bits_to_float(x.x & 0xffffu), acc); acc = fmaf(c[1], __uint_as_float(x.x & 0xffff0000u), acc);
    acc = fmaf(c[2], bf16_bits_to_float(x.y & 0xffffu), acc); acc = fmaf(c[3], __uint_as_float(x.y & 0xffff0000u), acc);
    acc = fmaf(c[4], bf16_bits_to_float(x.z & 0xffffu), acc); acc = fmaf(c[5], __uint_as_float(x.z & 0xffff0000u), acc);
    acc = fmaf(c[6], bf16_bits_to_float(x.w & 0xffffu), acc); acc = fmaf(c[7], __uint_as_float(x.w & 0xffff0000u), acc);
    return acc;
}
// acc[e] += p * x[e]
__device__ __forceinline__ void axpy_user(float (&acc)[8], float p, const uint4& x)
{
    acc[0] = fmaf(p, bf16_bits_to_float(x.x & 0xffffu), acc[0]); acc[1] = fmaf(p, __uint_as_float(x.x & 0xffff0000u), acc[1]);
    acc[2] = fmaf(p, bf16_bits_to_float(x.y & 0xffffu), acc[2]); acc[3] = fmaf(p, __uint_as_float(x.y & 0xffff0000u), acc[3]);
    acc[4] = fmaf(p, bf16_bits_to_float(x.z & 0xffffu), acc[4]); acc[5] = fmaf(p, __uint_as_float(x.z & 0xffff0000u), acc[5]);
    acc[6] = fmaf(p, bf16_bits_to_float(x.w & 0xffffu), acc[6]); acc[7] = fmaf(p, __uint_as_float(x.w & 0xffff0000u), acc[7]);
}

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float x = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, x) : v + x;
    }
    __syncthreads();  // red may still be read from the previous reduction
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < kMainThreads / 32; ++w) r = is_max ? fmaxf(r, red[w]) : r + red[w];  // fixed order
    return r;
}

constexpr int kAux = 16;  // floats per (request, group): [0] row sum l, [1..8] user-part output (not normalised)

// Persistent: CTA c takes (item, group) pairs c, c + gridDim.x, ... of the list ordered longest history first
// (pair = item * G + group, so neighbours in the list weigh about the same).  While a pair is processed, the T row
// of the CTA's next pair is already on its way into the other table buffer.
template <int D, int MODE, bool IDX16>
__global__ void __launch_bounds__(kMainThreads, 1)
    fact_main_kernel(const AttendArgs a, float* __restrict__ tw, float* __restrict__ aux, int s_cap)
{
    extern __shared__ __align__(16) float fsm[];
    const int m = a.cv.n_entries, G = a.cv.n_groups, d_user = a.cv.d_user, tid = threadIdx.x;
    const int n_pairs = a.n_items * G;
    // fsm[0 .. 2m): two table buffers; a pair's T row, dead after the scores, then its weight histogram
    float* Sb = fsm + 2 * (size_t)m;     // [s_cap] scores (softmax), half scores (SiLU); at the end the warps' sums
    float* red = Sb + s_cap;             // [32]
    const uint16_t* uK = reinterpret_cast<const uint16_t*>(a.cv.userK);
    const uint16_t* uV = reinterpret_cast<const uint16_t*>(a.cv.userV);
    const float sc = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 0.5f);
    constexpr int B = 4;  // positions per thread whose loads are in flight together
    int ix[B];
    uint4 x[B];

    struct Pair {
        int req, grp, L, q0;
        int64_t unit0;
    };
    auto get_pair = [&](int p) {
        Pair r;
        const Item it = a.items[p / G];
        const Req rq = a.reqs[it.req];
        r.req = it.req;
        r.grp = p - (p / G) * G;
        r.L = rq.L;
        r.q0 = rq.q0;
        r.unit0 = rq.base + (int64_t)r.grp * rq.Lpad;
        return r;
    };
    auto table_row = [&](const Pair& pr) { return tw + ((int64_t)pr.req * G + pr.grp) * row_floats(m); };
    auto fetch_table = [&](const Pair& pr, float* dstp) {  // all of the row in flight at once
        const float* row = table_row(pr);
        if ((m & 3) == 0) {
            const uint32_t dst = smem_u32(dstp);
            for (int j = 4 * tid; j < m; j += 4 * kMainThreads)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 4 * j), "l"(row + j) : "memory");
        } else {
            for (int j = tid; j < m; j += kMainThreads) dstp[j] = row[j];
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto load_batch = [&](const void* idx, const uint16_t* u, const Pair& pr, int i0) {
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const int i = i0 + b * kMainThreads;
            ix[b] = 0;
            x[b] = make_uint4(0, 0, 0, 0);
            if (i < pr.L) {
                ix[b] = load_index<IDX16>(idx, CKV_CLAMP(pr.unit0 + i, a.arena_units, a.err));
                x[b] = load_user(u, pr.unit0 + i, d_user);
            }
        }
    };

    int p = blockIdx.x, k = 0;
    if (p >= n_pairs) return;
    Pair cur = get_pair(p);
    fetch_table(cur, fsm);
    load_batch(a.cv.idxK, uK, cur, tid);
    for (;;) {
        float* Ts = fsm + (size_t)k * m;
        float* Ws = Ts;
        const int L = cur.L;
        float qu[8], ou[8];
        {
            const uint16_t* q = reinterpret_cast<const uint16_t*>(a.queries) + ((int64_t)cur.q0 * G + cur.grp) * D;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                qu[e] = e < d_user ? bf16_bits_to_float(__ldg(q + e)) : 0.f;
                ou[e] = 0.f;
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();  // T of this pair is in place; the other buffer's histogram has been written out
        const int p_next = p + gridDim.x;
        const bool more = p_next < n_pairs;
        Pair nxt = cur;
        if (more) {
            nxt = get_pair(p_next);
            fetch_table(nxt, fsm + (size_t)(k ^ 1) * m);
        }

        // scores: Sb[i] = scale * (q_u . K_u[i] + T[I_k[i]])   (softmax: in log2 units; SiLU: half the score)
        float mx = -CUDART_INF_F, lsum = 0.f;
        for (int i0 = tid; i0 < L;) {
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int i = i0 + b * kMainThreads;
                if (i < L) {
                    const float sv = dot_user(qu, x[b], Ts[CKV_CLAMP(ix[b], m, a.err)]) * sc;
                    Sb[i] = sv;
                    mx = fmaxf(mx, sv);
                }
            }
            i0 += B * kMainThreads;
            if (i0 < L) load_batch(a.cv.idxK, uK, cur, i0);
        }
        load_batch(a.cv.idxV, uV, cur, tid);  // the first V-side batch travels during the reduction
        if constexpr (MODE == CKV_SOFTMAX) mx = block_reduce(mx, true, red);
        else __syncthreads();
        // T is dead: the same memory becomes the histogram
        for (int j = tid; j < m; j += kMainThreads) Ws[j] = 0.f;
        __syncthreads();
        // weights: p_i into w[I_v[i]], p_i V_u[i] into the user-part output (every thread reads back its own scores)
        for (int i0 = tid; i0 < L;) {
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int i = i0 + b * kMainThreads;
                if (i < L) {
                    float pw;
                    if constexpr (MODE == CKV_SOFTMAX) {
                        pw = ex2(Sb[i] - mx);
                        lsum += pw;
                    } else {
                        const float h = Sb[i];  // silu(x) = x sigmoid(x) = h (1 + tanh(h)), h = x / 2
                        pw = fmaf(h, tanh_fast(h), h);
                    }
                    atomicAdd(&Ws[CKV_CLAMP(ix[b], m, a.err)], pw);
                    axpy_user(ou, pw, x[b]);
                }
            }
            i0 += B * kMainThreads;
            if (i0 < L) load_batch(a.cv.idxV, uV, cur, i0);
        }
        if (more) load_batch(a.cv.idxK, uK, nxt, tid);  // the next pair's first K-side batch travels during the write-out
        // row sum and user-part output: warp sums, then one thread per value adds the warps' sums in fixed order
        float vals[9] = {lsum, ou[0], ou[1], ou[2], ou[3], ou[4], ou[5], ou[6], ou[7]};
#pragma unroll
        for (int q9 = 0; q9 < 9; ++q9)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) vals[q9] += __shfl_xor_sync(0xffffffffu, vals[q9], o);
        __syncthreads();  // the histogram is complete; Sb is free
        if ((tid & 31) == 0) {
#pragma unroll
            for (int q9 = 0; q9 < 9; ++q9) Sb[(tid >> 5) * 9 + q9] = vals[q9];
        }
        // w goes back to HBM rounded to bf16 (the precision the output product takes it in), two entries per word,
        // over the head of the T row, zero-filled up to a multiple of 8 entries
        {
            uint32_t* wrow = reinterpret_cast<uint32_t*>(table_row(cur));
            for (int j2 = tid; 2 * j2 < row_floats(m); j2 += kMainThreads)
                wrow[j2] = pack_bf16(2 * j2 < m ? Ws[2 * j2] : 0.f, 2 * j2 + 1 < m ? Ws[2 * j2 + 1] : 0.f);
        }
        __syncthreads();
        if (tid < 9) {
            float v = 0.f;
            for (int w = 0; w < kMainThreads / 32; ++w) v += Sb[w * 9 + tid];
            aux[((int64_t)cur.req * G + cur.grp) * kAux + tid] = v;
        }
        if (!more) break;
        __syncthreads();  // Sb (the warps' sums) is read before the next pair's scores overwrite it
        cur = nxt;
        p = p_next;
        k ^= 1;
    }
}

// ------------------------------------------------------------------------------------------------ out = w P_v
// One CTA per (16 requests, group); warp w covers pool entries [w, w + 1) * ceil32(m / 16).  P_v rows are
// contiguous here: 32-row tiles through a two-slot cp.async ring per warp, fragments by transposing ldmatrix.
// 16-byte chunk c of tile row r sits at chunk c ^ swz(r).  The eight rows of one ldmatrix block are rows
// 8 t' + const + e (t' < 4, e < 2) here, see the k-slot order below: they must fall into eight different bank groups.
template <int D>
__device__ __forceinline__ int swz(int r)
{
    return D == 64 ? ((((r >> 3) & 3) << 1) | (r & 1)) : ((r >> 3) & 3);
}

template <int D>
__global__ void __launch_bounds__(kOutWarps * 32, 1)
    fact_out_kernel(const AttendArgs a, int n_req, const float* __restrict__ tw, const float* __restrict__ aux)
{
    constexpr int NTD = D / 8, ROWB = D * 2, CPR = ROWB / 16, RPI = 32 / CPR, TILE_B = 32 * ROWB;
    extern __shared__ __align__(128) unsigned char osm[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gl = lane >> 2, t = lane & 3;
    const int m = a.cv.n_entries, G = a.cv.n_groups, grp = blockIdx.y, r0 = blockIdx.x * 16;
    const int span = ((m + kOutWarps - 1) / kOutWarps + 31) / 32 * 32;
    const int jbeg = warp * span, jend = min(m, jbeg + span);
    const int r_lo = r0 + gl, r_hi = r_lo + 8;
    const bool v_lo = r_lo < n_req && a.reqs[r_lo].M > 0, v_hi = r_hi < n_req && a.reqs[r_hi].M > 0;
    const float* w_lo = tw + ((int64_t)(v_lo ? r_lo : 0) * G + grp) * row_floats(m);
    const float* w_hi = tw + ((int64_t)(v_hi ? r_hi : 0) * G + grp) * row_floats(m);
    const char* pV = reinterpret_cast<const char*>(a.cv.poolV) + (int64_t)grp * m * ROWB;
    const uint32_t ring = smem_u32(osm) + warp * (2 * TILE_B);
    const int cr = lane / CPR, cc = lane % CPR, lr = lane & 7, lm = lane >> 3;
    // Which pool entry sits in which k-slot is free as long as w and the V rows agree: a lane reads 8 consecutive
    // weights of its two requests with one 16-byte load each, and k-step b, slots (2t, 2t+1, 2t+8, 2t+9) hold
    // entries 8t + 4b + (0, 1, 2, 3) of the 32-entry chunk; the ldmatrix row addresses follow.
    uint32_t offV[2][NTD / 2];
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        const int r = 8 * (lr >> 1) + 4 * b + 2 * (lm & 1) + (lr & 1);  // chunk row of matrix row lr, matrix half lm & 1
#pragma unroll
        for (int jp = 0; jp < NTD / 2; ++jp) offV[b][jp] = r * ROWB + (((2 * jp + (lm >> 1)) ^ swz<D>(r)) << 4);
    }

    auto issue = [&](int jc, int slot) {  // rows jc .. jc+31 of the V pool (clamped: their weights are zero)
#pragma unroll
        for (int i = 0; i < 32 / RPI; ++i) {
            const int r = i * RPI + cr;
            const int j = min(jc + r, m - 1);
            const uint32_t dst = ring + slot * TILE_B + r * ROWB + ((cc ^ swz<D>(r)) << 4);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(pV + (int64_t)j * ROWB + cc * 16)
                         : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // weights of one 32-entry chunk: entries 8t .. 8t+7 of both requests, the bf16 pairs the main kernel stored
    // (rows start at multiples of 32 bytes and are zero-filled behind the last entry up to a multiple of 8 entries)
    auto load_w = [&](int jc, uint4 (&x)[2]) {
        const int j = jc + 8 * t;
        const bool in = j < jend;
        x[0] = (in && v_lo) ? __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(w_lo) + (j >> 1)))
                            : make_uint4(0, 0, 0, 0);
        x[1] = (in && v_hi) ? __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(w_hi) + (j >> 1)))
                            : make_uint4(0, 0, 0, 0);
    };

    float o[NTD][4];
#pragma unroll
    for (int j = 0; j < NTD; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    const int nch = jbeg < jend ? (jend - jbeg + 31) / 32 : 0;
    uint4 wa[2], wb[2];
    if (nch > 0) {
        issue(jbeg, 0);
        load_w(jbeg, wa);
    }
    for (int c = 0; c < nch; ++c) {
        const int jc = jbeg + 32 * c;
        if (c + 1 < nch) {
            issue(jc + 32, (c + 1) & 1);
            load_w(jc + 32, wb);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncwarp();
        const uint32_t vt = ring + (c & 1) * TILE_B;
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            const uint32_t pa[4] = {b ? wa[0].z : wa[0].x, b ? wa[1].z : wa[1].x, b ? wa[0].w : wa[0].y,
                                    b ? wa[1].w : wa[1].y};
#pragma unroll
            for (int jp = 0; jp < NTD / 2; ++jp) {
                uint32_t v0, v1, v2, v3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3)
                             : "r"(vt + offV[b][jp])
                             : "memory");
                mma_bf16(o[2 * jp], pa, v0, v1);
                mma_bf16(o[2 * jp + 1], pa, v2, v3);
            }
        }
        __syncwarp();  // every lane is done reading the slot that the next iteration refills
#pragma unroll
        for (int i = 0; i < 2; ++i) wa[i] = wb[i];
    }

    // sum the warps' partial outputs in fixed order, add the user part, normalise, store
    __syncthreads();
    float* red = reinterpret_cast<float*>(osm);  // [kOutWarps][16][D]
#pragma unroll
    for (int j = 0; j < NTD; ++j) {
        float* p = red + ((size_t)warp * 16 + gl) * D + 8 * j + 2 * t;
        p[0] = o[j][0];
        p[1] = o[j][1];
        p[8 * D] = o[j][2];
        p[8 * D + 1] = o[j][3];
    }
    __syncthreads();
    for (int x = threadIdx.x; x < 16 * D; x += kOutWarps * 32) {
        const int rr = x / D, f = x - rr * D, r = r0 + rr;
        if (r >= n_req || a.reqs[r].M <= 0) continue;
        float v = 0.f;
        for (int w = 0; w < kOutWarps; ++w) v += red[((size_t)w * 16 + rr) * D + f];
        const float* ax = aux + ((int64_t)r * G + grp) * kAux;
        if (f < a.cv.d_user) v += ax[1 + f];
        float inv;
        if (a.mode == CKV_SOFTMAX) inv = ax[0] > 0.f ? 1.0f / ax[0] : 0.f;
        else inv = a.reqs[r].L > 0 ? 1.0f / (float)a.reqs[r].L : 0.f;
        v *= inv;
        const int64_t oi = ((int64_t)a.reqs[r].q0 * G + grp) * D + f;
        if (a.out_dtype == CKV_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16_rn(v);
        else reinterpret_cast<float*>(a.out)[oi] = v;
    }
}

// Opt-in to large dynamic shared memory (per launch: the attribute belongs to the current device).
template <typename K>
cudaError_t set_smem(K kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <int D>
cudaError_t launch_fact(const AttendArgs& a, int n_req, int max_L, int n_sms, float* tw, float* aux, cudaStream_t s)
{
    const int m = a.cv.n_entries, G = a.cv.n_groups;
    const bool i16 = a.cv.idx_bytes == 2, soft = a.mode == CKV_SOFTMAX;
    fact_table_kernel<D><<<dim3((m + 255) / 256, (n_req + 16 * kTableMT - 1) / (16 * kTableMT), G), 128, 0, s>>>(
        a, n_req, tw);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int s_cap = std::max((max_L + 31) / 32 * 32, 9 * (kMainThreads / 32));  // scores; later the warps' sums
    const size_t smem_main = (2 * (size_t)m + s_cap + 32) * sizeof(float);
    const int n_pairs = a.n_items * G;
    const dim3 grid(n_pairs < n_sms ? n_pairs : n_sms);
#define CKV_FACT_MAIN(MODE, I16)                                                       \
    do {                                                                               \
        e = set_smem(fact_main_kernel<D, MODE, I16>, smem_main);                       \
        if (e != cudaSuccess) return e;                                                \
        fact_main_kernel<D, MODE, I16><<<grid, kMainThreads, smem_main, s>>>(a, tw, aux, s_cap); \
    } while (0)
    if (soft) {
        if (i16) CKV_FACT_MAIN(CKV_SOFTMAX, true); else CKV_FACT_MAIN(CKV_SOFTMAX, false);
    } else {
        if (i16) CKV_FACT_MAIN(CKV_SILU_OVER_L, true); else CKV_FACT_MAIN(CKV_SILU_OVER_L, false);
    }
#undef CKV_FACT_MAIN
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t smem_out = std::max((size_t)kOutWarps * 2 * 32 * D * 2, (size_t)kOutWarps * 16 * D * sizeof(float));
    e = set_smem(fact_out_kernel<D>, smem_out);
    if (e != cudaSuccess) return e;
    fact_out_kernel<D><<<dim3((n_req + 15) / 16, G), kOutWarps * 32, smem_out, s>>>(a, n_req, tw, aux);
    return cudaGetLastError();
}

}  // namespace

// Largest history (positions) the main kernel can hold next to its two tables, or -1 if the shape is not supported.
int fact_max_history(int dtype, int head_dim, int d_user, int n_entries)
{
    if (dtype != CKV_BF16 || (head_dim != 32 && head_dim != 64) || d_user > 8) return -1;
    const int64_t floats = 220 * 1024 / 4 - 32 - 2 * (int64_t)n_entries;  // two table buffers + one score per position
    if (floats < 9 * (kMainThreads / 32)) return -1;
    return (int)(floats / 32 * 32);
}

int fact_aux_floats() { return kAux; }
int fact_row_floats(int n_entries) { return row_floats(n_entries); }

// Three launches; a.items holds one unsplit item per request with a query; tw: [n_req][G][fact_row_floats()] floats,
// aux: [n_req][G][fact_aux_floats()] floats.
cudaError_t launch_attend_fact(int D, const AttendArgs& a, int n_req, int max_L, int n_sms, float* tw, float* aux,
                               cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    return D == 64 ? launch_fact<64>(a, n_req, max_L, n_sms, tw, aux, s)
                   : launch_fact<32>(a, n_req, max_L, n_sms, tw, aux, s);
}

}  // namespace ckv
