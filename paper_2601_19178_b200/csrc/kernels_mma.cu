// Warp-level tensor-core gather-concat-attention kernel (bf16, head_dim 32 or 64) for a moderate
// number of queries per user (head_dim 64: also for a single query).
//
// One warp owns (work item, group, block of 16*MT queries) and walks the history chunk 32
// positions at a time with m16n8k16 MMAs: S = Q K^T, weights in registers, O += P V.
// K and V rows go from the pool into a per-warp ring of shared-memory tiles with 16-byte
// asynchronous copies, NST tiles deep, and reach the MMA register layouts through ldmatrix
// (transposing for V).  A whole row is fetched by adjacent lanes, so the L1 sees one line per
// row, and the copies in flight cost no registers: a warp keeps NST - 1 tiles outstanding
// while it computes.  The user-specific leading elements (Eq. K) are written over the head
// of each staged row.  Positions keep their order: tile row r is position p0 + r.
// A side that is not shared (sharing only keys or only values) has its full-width rows in the
// arena; they are copied into the ring in place of pool rows (cp.async loader only) and nothing is
// patched.  With visible lengths a query row only takes the positions before its own limit.
//
// Two ways to fill the ring (template parameter TMA), same results bit for bit:
//   - 16-byte cp.async copies through L1 (hot rows of skewed index distributions stay in L1, but every
//     row crosses the L1 / shared-memory data pipe on the way in and again on the way out);
//   - TMA tile::gather4 loads, four pool rows per instruction, completion on an mbarrier: the rows
//     bypass L1 and that pipe; the hardware swizzle modes are the chunk order ldmatrix wants.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "ckv_internal.h"
#include "ptx_helpers.cuh"

namespace ckv {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldsm4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}
__device__ __forceinline__ void ldsm4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}

template <bool IDX16>
__device__ __forceinline__ int load_index(const void* base, int64_t unit)
{
    if constexpr (IDX16) return __ldg(reinterpret_cast<const uint16_t*>(base) + unit);
    else return __ldg(reinterpret_cast<const int32_t*>(base) + unit);
}

// user part of one position (d_user in {1, 2, 4, 8}: 2 to 16 bytes)
__device__ __forceinline__ uint4 load_user_part(const uint16_t* u, int64_t unit, int d_user)
{
    uint4 r = make_uint4(0, 0, 0, 0);
    switch (d_user) {
        case 1: r.x = __ldg(u + unit); break;
        case 2: r.x = __ldg(reinterpret_cast<const uint32_t*>(u + unit * 2)); break;
        case 4: {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(u + unit * 4));
            r.x = w.x;
            r.y = w.y;
            break;
        }
        case 8: r = __ldg(reinterpret_cast<const uint4*>(u + unit * 8)); break;
        default: break;
    }
    return r;
}
__device__ __forceinline__ void store_user_part(uint32_t addr, const uint4& r, int d_user)
{
    switch (d_user) {
        case 1: asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((uint16_t)r.x) : "memory"); break;
        case 2: asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(r.x) : "memory"); break;
        case 4: asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(addr), "r"(r.x), "r"(r.y) : "memory"); break;
        case 8:
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w)
                         : "memory");
            break;
        default: break;
    }
}

template <int D, int MT, bool TMA>
struct MmaCfg {
    static constexpr int ROWB = D * 2;            // bytes per row
    static constexpr int CPR = ROWB / 16;         // 16-byte chunks per row
    static constexpr int RPI = 32 / CPR;          // rows one warp-wide copy instruction covers
    static constexpr int TILE_B = 32 * ROWB;      // one K or V tile of 32 positions
    // ring depth (more resident warps beat a deeper ring, except for cp.async with 128-byte rows)
    static constexpr int NST = (D == 64 && !TMA) ? 3 : 2;
    static constexpr int WARPS = 4;
    // TMA: tiles on 1024-byte boundaries (the swizzle pattern follows the address), then one mbarrier per slot
    static constexpr int SMEM = WARPS * NST * 2 * TILE_B + (TMA ? 1024 + WARPS * NST * 8 : 0);
    static constexpr int MIN_BLOCKS = MT == 1 ? (D == 64 ? (TMA ? 3 : 2) : 4) : 1;
};

enum { ERR_MMA_LOAD = 16 };  // a bounded wait for a TMA tile ran out
constexpr int kTmaSpinLimit = 1 << 22;

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// chunk c of tile row r sits at chunk c ^ swz(r): the eight rows of an 8x8 ldmatrix block fall into
// eight different 16-byte bank groups
template <int D>
__device__ __forceinline__ int swz(int r)
{
    return D == 64 ? (r & 7) : ((r >> 1) & 3);
}

// VAR = false: both sides shared and no visible lengths (the hot configurations); the code for the variants is
// compiled out.
template <int D, int MT, int MODE, bool IDX16, bool TMA, bool VAR>
__global__ void __launch_bounds__(128, MmaCfg<D, MT, TMA>::MIN_BLOCKS)
    attend_mma_kernel(const AttendArgs a, int n_mb, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, int* err_flag)
{
    using C = MmaCfg<D, MT, TMA>;
    constexpr int NTD = D / 8, KS = D / 16, ROWB = C::ROWB, CPR = C::CPR, RPI = C::RPI, NST = C::NST;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int64_t wid = (int64_t)blockIdx.x * C::WARPS + warp;
    if (wid >= (int64_t)a.n_items * n_mb) return;
    const Item it = a.items[wid / n_mb];
    const int mb = (int)(wid % n_mb);
    const Req rq = a.reqs[it.req];
    const int row0 = mb * 16 * MT;
    if (row0 >= rq.M) return;
    const int grp = blockIdx.y, G = a.cv.n_groups, d_user = a.cv.d_user;
    const bool full_k = VAR && a.cv.full_k != 0, full_v = VAR && a.cv.full_v != 0;  // the side's rows are cached full width
    const bool wide_user = d_user == 1 || d_user == 2 || d_user == 4 || d_user == 8;

    uint32_t qa[MT][KS][4];
    const uint16_t* Q = reinterpret_cast<const uint16_t*>(a.queries);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int r_lo = row0 + 16 * mt + g, r_hi = r_lo + 8;
        const uint16_t* q_lo = Q + ((int64_t)(rq.q0 + r_lo) * G + grp) * D;
        const uint16_t* q_hi = Q + ((int64_t)(rq.q0 + r_hi) * G + grp) * D;
        if (r_lo < rq.M) (void)CKV_CLAMP((int64_t)(rq.q0 + r_lo), a.q_rows, err_flag);
        if (r_hi < rq.M) (void)CKV_CLAMP((int64_t)(rq.q0 + r_hi), a.q_rows, err_flag);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int c = 16 * ks + 2 * t;
            qa[mt][ks][0] = r_lo < rq.M ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + c)) : 0u;
            qa[mt][ks][1] = r_hi < rq.M ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + c)) : 0u;
            qa[mt][ks][2] = r_lo < rq.M ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + c + 8)) : 0u;
            qa[mt][ks][3] = r_hi < rq.M ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + c + 8)) : 0u;
        }
    }
    // rows 8..15 of the only query tile are all padding when the user has at most 8 queries
    const bool has_hi = MT > 1 || row0 + 8 < rq.M;
    // positions a query row attends: [0, lim); rows beyond the user's queries take none
    int lim[MT][2], lim_max = rq.L, lim_min = rq.L;
    if constexpr (VAR) {
        lim_max = 0;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = row0 + 16 * mt + g + 8 * h;
                int v = 0;
                if (r < rq.M) {
                    v = a.vis ? min(max(__ldg(a.vis + rq.q0 + r), 0), rq.L) : rq.L;
                    lim_min = min(lim_min, v);
                }
                lim[mt][h] = v;
                lim_max = max(lim_max, v);
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lim_max = max(lim_max, __shfl_xor_sync(0xffffffffu, lim_max, o));
            lim_min = min(lim_min, __shfl_xor_sync(0xffffffffu, lim_min, o));
        }
    }

    float o[MT][NTD][4];
    float m_run[MT][2], l_run[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        m_run[mt][0] = m_run[mt][1] = -CUDART_INF_F;
        l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
        for (int j = 0; j < NTD; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[mt][j][e] = 0.f;
    }

    const int cr = lane / CPR, cc = lane % CPR;  // this lane's row within a copy instruction and its chunk
    const char* pK = reinterpret_cast<const char*>(a.cv.poolK) + (int64_t)grp * a.cv.n_entries * ROWB + cc * 16;
    const char* pV = reinterpret_cast<const char*>(a.cv.poolV) + (int64_t)grp * a.cv.n_entries * ROWB + cc * 16;
    const int64_t unit0 = rq.base + (int64_t)grp * rq.Lpad + it.begin + lane;  // this lane's position of step 0
    (void)CKV_CLAMP(unit0 - lane + ((it.len + 31) & ~31) - 1, a.arena_units, err_flag);  // the chunk's last (padded) unit
    const uint16_t* uK = reinterpret_cast<const uint16_t*>(a.cv.userK);
    const uint16_t* uV = reinterpret_cast<const uint16_t*>(a.cv.userV);
    const int end = VAR ? min(it.begin + it.len, lim_max) : it.begin + it.len;  // nothing behind the last visible position is touched
    const int nsteps = VAR ? (end > it.begin ? (end - it.begin + 31) >> 5 : 0) : (it.len + 31) >> 5;
    const int full_end = VAR ? min(end, lim_min) : end;  // up to here every row of this warp sees every position
    // A side that is not shared: its rows are the chunk's own units in the arena, and what stands in for the pool
    // index of the position in lane l of tile `step` is its offset 32 step + l from the chunk's first unit.
    if (full_k) pK = reinterpret_cast<const char*>(a.cv.userK) + (unit0 - lane) * ROWB + cc * 16;
    if (full_v) pV = reinterpret_cast<const char*>(a.cv.userV) + (unit0 - lane) * ROWB + cc * 16;
    const float sc = a.scale * (MODE == CKV_SOFTMAX ? kLog2e : 0.5f);

    uint32_t smem0 = smem_u32(smem_raw);
    if constexpr (TMA) smem0 = (smem0 + 1023u) & ~1023u;
    const uint32_t ring = smem0 + warp * (NST * 2 * C::TILE_B);
    const uint32_t bars = smem0 + C::WARPS * (NST * 2 * C::TILE_B) + warp * (NST * 8);  // TMA only
    if constexpr (TMA) {
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < NST; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bars + 8 * i));
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
    }
    const int row_base = grp * a.cv.n_entries;  // TMA row coordinate of pool row 0 of this group
    // ldmatrix row addresses of this lane (matrix lane >> 3, row lane & 7)
    const int lr = lane & 7, lm = lane >> 3;
    uint32_t offK[KS / 2 > 0 ? KS / 2 : 1], offV[NTD / 2];
#pragma unroll
    for (int kp = 0; kp < KS / 2; ++kp) offK[kp] = lr * ROWB + (((4 * kp + lm) ^ swz<D>(lr)) << 4);
#pragma unroll
    for (int jp = 0; jp < NTD / 2; ++jp)
        offV[jp] = ((lm & 1) * 8 + lr) * ROWB + (((2 * jp + (lm >> 1)) ^ swz<D>(lr)) << 4);
    const uint32_t offU = lane * ROWB + (swz<D>(lane) << 4);  // head of this lane's row (chunk 0)

    // copies of one tile: the indices of its 32 positions sit one per lane
    auto issue = [&](int step, int idx_k, int idx_v) {
        const uint32_t kt = ring + (step % NST) * (2 * C::TILE_B), vt = kt + C::TILE_B;
        if constexpr (TMA) {
            // lanes 0..7 fetch the K tile, lanes 8..15 the V tile, four rows (positions 4j .. 4j+3) each
            const uint32_t bar = bars + 8 * (step % NST);
            if (lane == 0)
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * C::TILE_B)
                             : "memory");
            __syncwarp();
            int r[4];
            const int j4 = 4 * (lane & 7);
            if constexpr (IDX16) {
                const int both = idx_k | (idx_v << 16);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int x = __shfl_sync(0xffffffffu, both, j4 + j);
                    r[j] = row_base + (lane < 8 ? (x & 0xffff) : (int)((uint32_t)x >> 16));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int xk = __shfl_sync(0xffffffffu, idx_k, j4 + j), xv = __shfl_sync(0xffffffffu, idx_v, j4 + j);
                    r[j] = row_base + (lane < 8 ? xk : xv);
                }
            }
            if (lane < 16) {
                const CUtensorMap* tm = lane < 8 ? &tmK : &tmV;
                const uint32_t dst = (lane < 8 ? kt : vt) + j4 * ROWB;
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
                    "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
                    "l"(tm), "r"(0), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(bar)
                    : "memory");
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32 / RPI; ++i) {
                const int r = i * RPI + cr;
                const uint32_t off = r * ROWB + ((cc ^ swz<D>(r)) << 4);
                // (range-checked build: a pool index below n_entries, or, for a side that is not shared, an offset
                // inside the user's padded history; the ring slot inside this block's shared memory)
                const int rk = CKV_CLAMP(__shfl_sync(0xffffffffu, idx_k, r), full_k ? rq.Lpad - it.begin : a.cv.n_entries, err_flag),
                          rv = CKV_CLAMP(__shfl_sync(0xffffffffu, idx_v, r), full_v ? rq.Lpad - it.begin : a.cv.n_entries, err_flag);
                (void)CKV_CLAMP((int)(vt + off - smem_u32(smem_raw)), C::SMEM - 15, err_flag);
                cp_async16(kt + off, pK + (int64_t)rk * ROWB);
                cp_async16(vt + off, pV + (int64_t)rv * ROWB);
            }
        }
    };
    auto fetch_idx = [&](int step, int& idx_k, int& idx_v) {
        if (step < nsteps) {
            idx_k = full_k ? 32 * step + lane : load_index<IDX16>(a.cv.idxK, unit0 + 32 * step);
            idx_v = full_v ? 32 * step + lane : load_index<IDX16>(a.cv.idxV, unit0 + 32 * step);
        } else {
            idx_k = idx_v = 0;
        }
    };
    auto fetch_user = [&](int step, uint4& k, uint4& v) {
        if (wide_user && step < nsteps) {
            if (!full_k) k = load_user_part(uK, unit0 + 32 * step, d_user);
            if (!full_v) v = load_user_part(uV, unit0 + 32 * step, d_user);
        }
    };

    // prologue: tiles 0 .. NST-2 in flight, indices two tiles further, user parts two tiles ahead
    int ikA, ivA, ikB, ivB, ikC, ivC;
#pragma unroll
    for (int s0 = 0; s0 < NST - 1; ++s0) {
        fetch_idx(s0, ikA, ivA);
        if (s0 < nsteps) issue(s0, ikA, ivA);
        if constexpr (!TMA) cp_async_commit();
    }
    fetch_idx(NST - 1, ikA, ivA);
    fetch_idx(NST, ikB, ivB);
    fetch_idx(NST + 1, ikC, ivC);
    uint4 ukA, uvA, ukB, uvB;
    ukA = uvA = ukB = uvB = make_uint4(0, 0, 0, 0);
    fetch_user(0, ukA, uvA);
    fetch_user(1, ukB, uvB);

    bool ok = true;
    for (int step = 0; step < nsteps; ++step) {
        const int p0 = it.begin + 32 * step;
        if (step + NST - 1 < nsteps) issue(step + NST - 1, ikA, ivA);
        if constexpr (!TMA) cp_async_commit();
        ikA = ikB; ivA = ivB; ikB = ikC; ivB = ivC;
        fetch_idx(step + NST + 2, ikC, ivC);
        if constexpr (TMA) {
            const uint32_t bar = bars + 8 * (step % NST), parity = (step / NST) & 1;
            int spins = 0;
            while (!mbar_try_wait(bar, parity)) {
                if (++spins > kTmaSpinLimit) {
                    ok = false;
                    break;
                }
            }
            if (!__all_sync(0xffffffffu, ok)) {  // give up: nothing more is issued, nothing is stored
                ok = false;
                break;
            }
        } else {
            cp_async_wait<NST - 1>();
        }
        __syncwarp();
        const uint32_t kt = ring + (step % NST) * (2 * C::TILE_B), vt = kt + C::TILE_B;
        // Eq. K: dims [0, d_user) of every row come from the user-specific part
        if (wide_user) {
            if (!full_k) store_user_part(kt + offU, ukA, d_user);
            if (!full_v) store_user_part(vt + offU, uvA, d_user);
            ukA = ukB; uvA = uvB;
            fetch_user(step + 2, ukB, uvB);
        } else if (d_user > 0 && !(full_k && full_v)) {
            for (int e = 0; e < d_user; ++e) {
                if (!full_k) {
                    const uint16_t xk = __ldg(uK + (unit0 + 32 * step) * d_user + e);
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(kt + offU + 2 * e), "h"(xk) : "memory");
                }
                if (!full_v) {
                    const uint16_t xv = __ldg(uV + (unit0 + 32 * step) * d_user + e);
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(vt + offU + 2 * e), "h"(xv) : "memory");
                }
            }
        }
        __syncwarp();
        const bool tail = p0 + 32 > full_end;  // some (row, position) pair of this tile is not attended

        uint32_t kf[4][2 * KS];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            if constexpr (D == 64) {
#pragma unroll
                for (int kp = 0; kp < 2; ++kp)
                    ldsm4(kf[nt][4 * kp], kf[nt][4 * kp + 1], kf[nt][4 * kp + 2], kf[nt][4 * kp + 3],
                          kt + nt * (8 * ROWB) + offK[kp]);
            } else {
                ldsm4(kf[nt][0], kf[nt][1], kf[nt][2], kf[nt][3], kt + nt * (8 * ROWB) + offK[0]);
            }
        }
        uint32_t vb[2][NTD][2];
#pragma unroll
        for (int b = 0; b < 2; ++b)
#pragma unroll
            for (int jp = 0; jp < NTD / 2; ++jp)
                ldsm4_trans(vb[b][2 * jp][0], vb[b][2 * jp][1], vb[b][2 * jp + 1][0], vb[b][2 * jp + 1][1],
                            vt + b * (16 * ROWB) + offV[jp]);

#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            float s[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) mma_bf16(s[nt], qa[mt][ks], kf[nt][2 * ks], kf[nt][2 * ks + 1]);
            }
            // element (nt, e): position p0 + 8 nt + 2t + (e & 1), query row g (e < 2) or g + 8
            uint32_t pa[2][4];
            if constexpr (MODE == CKV_SOFTMAX) {
                if (tail) {
                    const int e_lo = VAR ? min(end, lim[mt][0]) : end, e_hi = VAR ? min(end, lim[mt][1]) : end;
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        const int pc = p0 + 8 * nt + 2 * t;
                        if (pc >= e_lo) s[nt][0] = -CUDART_INF_F;
                        if (pc + 1 >= e_lo) s[nt][1] = -CUDART_INF_F;
                        if (pc >= e_hi) s[nt][2] = -CUDART_INF_F;
                        if (pc + 1 >= e_hi) s[nt][3] = -CUDART_INF_F;
                    }
                }
                float mx0 = s[0][0], mx1 = s[0][2];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
                    mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
                }
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                if (has_hi) {
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                }
                // a row may not see any position of this tile (or of any tile so far): its maximum is then -inf
                // and must not enter the exponent arguments
                const float mn0 = fmaxf(m_run[mt][0], mx0 * sc);
                const float mn1 = has_hi ? fmaxf(m_run[mt][1], mx1 * sc) : 0.f;
                // (without visible lengths the first position of a tile is always attended and the maxima are finite)
                const float ms0 = VAR && mn0 == -CUDART_INF_F ? 0.f : mn0, ms1 = VAR && mn1 == -CUDART_INF_F ? 0.f : mn1;
                // the running maxima settle after a few tiles: rescale only when one of them moved
                const bool moved = mn0 != m_run[mt][0] || (has_hi && mn1 != m_run[mt][1]);
                if (__any_sync(0xffffffffu, moved)) {
                    const float c0 = ex2(m_run[mt][0] - ms0), c1 = has_hi ? ex2(m_run[mt][1] - ms1) : 1.f;
                    m_run[mt][0] = mn0;
                    if (has_hi) m_run[mt][1] = mn1;
                    l_run[mt][0] *= c0;
                    l_run[mt][1] *= c1;
#pragma unroll
                    for (int j = 0; j < NTD; ++j) {
                        o[mt][j][0] *= c0; o[mt][j][1] *= c0;
                        o[mt][j][2] *= c1; o[mt][j][3] *= c1;
                    }
                }
                float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    const float p0v = ex2(fmaf(s[nt][0], sc, -ms0)), p1v = ex2(fmaf(s[nt][1], sc, -ms0));
                    ps0 += p0v + p1v;
                    pa[nt >> 1][(nt & 1) * 2] = pack_bf16(p0v, p1v);
                    if (has_hi) {
                        const float p2v = ex2(fmaf(s[nt][2], sc, -ms1)), p3v = ex2(fmaf(s[nt][3], sc, -ms1));
                        ps1 += p2v + p3v;
                        pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2v, p3v);
                    } else {
                        pa[nt >> 1][(nt & 1) * 2 + 1] = 0u;
                    }
                }
                l_run[mt][0] += ps0;
                l_run[mt][1] += ps1;
            } else {
                // silu(x) = x sigmoid(x) = h (1 + tanh(h)), h = x / 2   (sc = scale / 2)
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    float w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float h = s[nt][e] * sc;
                        w[e] = (e < 2 || has_hi) ? fmaf(h, tanh_fast(h), h) : 0.f;
                    }
                    if (tail) {
                        const int e_lo = VAR ? min(end, lim[mt][0]) : end, e_hi = VAR ? min(end, lim[mt][1]) : end,
                                  pc = p0 + 8 * nt + 2 * t;
                        if (pc >= e_lo) w[0] = 0.f;
                        if (pc + 1 >= e_lo) w[1] = 0.f;
                        if (pc >= e_hi) w[2] = 0.f;
                        if (pc + 1 >= e_hi) w[3] = 0.f;
                    }
                    pa[nt >> 1][(nt & 1) * 2] = pack_bf16(w[0], w[1]);
                    pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(w[2], w[3]);
                }
            }
#pragma unroll
            for (int b = 0; b < 2; ++b)
#pragma unroll
                for (int j = 0; j < NTD; ++j) mma_bf16(o[mt][j], pa[b], vb[b][j][0], vb[b][j][1]);
        }
        // every lane is done with this tile before the ring slot is refilled (TMA: its ordinary stores
        // and loads are ordered before the asynchronous-proxy writes of the refill)
        if constexpr (TMA) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
    }
    if constexpr (TMA) {
        if (!ok) {
            if (lane == 0) atomicOr(err_flag, ERR_MMA_LOAD);
            return;
        }
    } else {
        cp_async_wait<0>();
    }

    // epilogue: finish the row sums over the quad, then store outputs or partials
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float l = l_run[mt][h];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int r = row0 + 16 * mt + g + 8 * h;
            if (r >= rq.M) continue;
            if (it.part_row < 0) {
                float inv;
                if constexpr (MODE == CKV_SOFTMAX) inv = l > 0.f ? 1.0f / l : 0.f;
                else inv = rq.L > 0 ? 1.0f / (float)rq.L : 0.f;
                const int64_t base = ((int64_t)(rq.q0 + r) * G + grp) * D;
#pragma unroll
                for (int j = 0; j < NTD; ++j) {
                    const float x = o[mt][j][2 * h] * inv, y = o[mt][j][2 * h + 1] * inv;
                    if (a.out_dtype == CKV_BF16)
                        *reinterpret_cast<uint32_t*>(reinterpret_cast<uint16_t*>(a.out) + base + 8 * j + 2 * t) =
                            pack_bf16(x, y);
                    else
                        *reinterpret_cast<float2*>(reinterpret_cast<float*>(a.out) + base + 8 * j + 2 * t) =
                            make_float2(x, y);
                }
            } else {
                float* pr = a.partials + (CKV_CLAMP((int64_t)(it.part_row + r), a.part_rows, err_flag) * G + grp) * (D + 2);
                if (t == 0) {
                    pr[0] = m_run[mt][h];
                    pr[1] = l;
                }
#pragma unroll
                for (int j = 0; j < NTD; ++j)
                    *reinterpret_cast<float2*>(pr + 2 + 8 * j + 2 * t) =
                        make_float2(o[mt][j][2 * h], o[mt][j][2 * h + 1]);
            }
        }
    }
}

template <int D, int MT, int MODE, bool IDX16, bool TMA, bool VAR>
cudaError_t launch_mma_one(const AttendArgs& a, int n_mb, dim3 grid, const CUtensorMap* maps, int* err_flag,
                           cudaStream_t s)
{
    using C = MmaCfg<D, MT, TMA>;
    // per launch: the attribute belongs to the current device, and a context may sit on any of them
    cudaError_t e = cudaFuncSetAttribute(attend_mma_kernel<D, MT, MODE, IDX16, TMA, VAR>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    static const CUtensorMap none{};
    attend_mma_kernel<D, MT, MODE, IDX16, TMA, VAR>
        <<<grid, 128, C::SMEM, s>>>(a, n_mb, TMA ? maps[0] : none, TMA ? maps[1] : none, err_flag);
    return cudaGetLastError();
}

template <int D, int MT>
cudaError_t launch_mma(const AttendArgs& a, int n_mb, const CUtensorMap* maps, int* err_flag, cudaStream_t s)
{
    const int64_t warps = (int64_t)a.n_items * n_mb;
    const dim3 grid((unsigned)((warps + 3) / 4), a.cv.n_groups);
    const bool i16 = a.cv.idx_bytes == 2;
    const bool var = a.vis != nullptr || a.cv.full_k || a.cv.full_v;  // the TMA loader is never asked for with these
#define CKV_MMA_GO(MODE, I16)                                                                        \
    (maps  ? launch_mma_one<D, MT, MODE, I16, true, false>(a, n_mb, grid, maps, err_flag, s)         \
     : var ? launch_mma_one<D, MT, MODE, I16, false, true>(a, n_mb, grid, maps, err_flag, s)         \
           : launch_mma_one<D, MT, MODE, I16, false, false>(a, n_mb, grid, maps, err_flag, s))
    if (a.mode == CKV_SOFTMAX) return i16 ? CKV_MMA_GO(CKV_SOFTMAX, true) : CKV_MMA_GO(CKV_SOFTMAX, false);
    return i16 ? CKV_MMA_GO(CKV_SILU_OVER_L, true) : CKV_MMA_GO(CKV_SILU_OVER_L, false);
#undef CKV_MMA_GO
}

}  // namespace

bool mma_supported(int dtype, int head_dim, int d_user)
{
    return dtype == CKV_BF16 && (head_dim == 32 || head_dim == 64) && d_user <= 8;
}

// head_dim 64 rows keep a warp busy with one 16-query tile; 32-wide heads take up to four
int mma_queries_per_warp(int D, int max_M) { return (D == 64 || max_M <= 16) ? 16 : (max_M <= 32 ? 32 : 64); }

cudaError_t launch_attend_mma(int D, int max_M, const AttendArgs& a, const void* tensor_maps, int* err_flag,
                              cudaStream_t s)
{
    if (a.n_items == 0) return cudaSuccess;
    const CUtensorMap* maps = reinterpret_cast<const CUtensorMap*>(tensor_maps);
    const int qpw = mma_queries_per_warp(D, max_M);
    const int n_mb = (max_M + qpw - 1) / qpw;
    if (D == 64) return launch_mma<64, 1>(a, n_mb, maps, err_flag, s);
    switch (qpw) {
        case 16: return launch_mma<32, 1>(a, n_mb, maps, err_flag, s);
        case 32: return launch_mma<32, 2>(a, n_mb, maps, err_flag, s);
        default: return launch_mma<32, 4>(a, n_mb, maps, err_flag, s);
    }
}

// Tensor maps of the K and the V pool ([n_groups * n_entries] rows of head_dim bf16) for tile::gather4: a box of
// one row, hardware swizzle of the row's 16-byte chunks (128-byte rows: chunk ^ (row & 7); 64-byte rows:
// chunk ^ ((row >> 1) & 3)).  maps_out: 2 x 128 bytes, 64-byte aligned.  false if the driver cannot encode them.
bool make_pool_tensor_maps(int D, int64_t rows, const void* poolK, const void* poolV, void* maps_out)
{
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    if ((D != 32 && D != 64) || rows < 1 || rows > INT32_MAX) return false;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return false;
    }
    CUtensorMap* maps = reinterpret_cast<CUtensorMap*>(maps_out);
    const void* src[2] = {poolK, poolV};
    for (int i = 0; i < 2; ++i) {
        const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
        const cuuint32_t box[2] = {(cuuint32_t)D, 1};
        const cuuint32_t estr[2] = {1, 1};
        const CUresult r = reinterpret_cast<EncodeFn>(fn)(
            &maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(src[i]), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, D == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return false;
    }
    return true;
}

}  // namespace ckv
