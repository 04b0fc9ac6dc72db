// Data-movement kernels: pool row layout, compressed-cache packing with index
// validation, and the test-only full-width materialisation (Eq. Kc + Eq. K).
// All of them copy bits; none does arithmetic on values.
#include "ckv_internal.h"

namespace ckv {
namespace {

// dst[g][j][c] = c < d_user ? 0 : src[g][j][c - d_user]      (rows padded to the head width)
template <typename E>
__global__ void pool_layout_kernel(const E* __restrict__ src, E* __restrict__ dst, int64_t rows,
                                   int d_shared, int D)
{
    const int d_user = D - d_shared;
    const int64_t total = rows * D;
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = t / D;
        const int c = (int)(t - r * D);
        dst[t] = c < d_user ? E(0) : src[r * d_shared + (c - d_user)];
    }
}

// The two sides of a cache entry (K and V) are stored alike but may differ in width: a shared side keeps a pool
// index and d_user user-specific elements per unit, a side that is not shared (sharing only keys or only values)
// keeps the whole head_dim-wide row and no index.
struct SideDst {
    void* idx;     // arena indices, null for a side that is not shared
    void* user;    // arena user parts / full rows
    int width;     // elements per unit in `user`
};

template <typename E, typename I>
__device__ __forceinline__ void store_unit(const SideDst& d, int64_t dst, const int32_t* idx_src, const E* user_src,
                                           int64_t src, bool real, int n_entries, int* bad_flag)
{
    E* du = reinterpret_cast<E*>(d.user);
    if (real) {
        for (int c = 0; c < d.width; ++c) du[dst * d.width + c] = user_src[src * d.width + c];
    } else {  // padding: a valid row index and zeros
        for (int c = 0; c < d.width; ++c) du[dst * d.width + c] = E(0);
    }
    if (d.idx) {
        int32_t j = real ? idx_src[src] : 0;
        if (j < 0 || j >= n_entries) {
            atomicOr(bad_flag, 1);
            j = 0;
        }
        reinterpret_cast<I*>(d.idx)[dst] = (I)j;
    }
}

// One thread per arena unit of the batch.  unit_off[u] = sum over earlier users of
// G * Lpad; the unit of (user u, group g, position i) is unit_off[u] + g * Lpad_u + i.
template <typename E, typename I>
__global__ void pack_kernel(int G, int n_entries, int n_users,
                            const int64_t* __restrict__ hist_off,
                            const int64_t* __restrict__ unit_off, int64_t total_units,
                            int64_t arena_base, const int32_t* __restrict__ idxK,
                            const int32_t* __restrict__ idxV, const E* __restrict__ userK,
                            const E* __restrict__ userV, SideDst dK, SideDst dV, int* __restrict__ bad_flag)
{
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total_units;
         t += (int64_t)gridDim.x * blockDim.x) {
        int lo = 0, hi = n_users;  // last u with unit_off[u] <= t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (unit_off[mid] <= t) lo = mid; else hi = mid;
        }
        const int u = lo;
        const int64_t local = t - unit_off[u];
        const int64_t Lpad = (unit_off[u + 1] - unit_off[u]) / G;
        const int g = (int)(local / Lpad);
        const int64_t i = local - g * Lpad;
        const int64_t L = hist_off[u + 1] - hist_off[u];
        const int64_t dst = arena_base + t;
        const int64_t src = (hist_off[u] + i) * G + g;
        store_unit<E, I>(dK, dst, idxK, userK, src, i < L, n_entries, bad_flag);
        store_unit<E, I>(dV, dst, idxV, userV, src, i < L, n_entries, bad_flag);
    }
}

template <typename E, typename I>
__device__ __forceinline__ void copy_unit(const SideDst& d, int64_t dst, int64_t src)
{
    E* du = reinterpret_cast<E*>(d.user);
    for (int c = 0; c < d.width; ++c) du[dst * d.width + c] = du[src * d.width + c];
    if (d.idx) reinterpret_cast<I*>(d.idx)[dst] = reinterpret_cast<I*>(d.idx)[src];
}

// Append: units of one user with L_old + L_new positions at arena unit `dst_base`; position i < L_old is copied
// from the user's old units, the rest comes from the new [L_new][G] inputs (range-checked like pack_kernel).
template <typename E, typename I>
__global__ void append_kernel(int G, int n_entries, int64_t old_base, int L_old, int Lpad_old,
                              int64_t dst_base, int L_new, int Lpad_tot, const int32_t* __restrict__ idxK,
                              const int32_t* __restrict__ idxV, const E* __restrict__ userK,
                              const E* __restrict__ userV, SideDst dK, SideDst dV, int* __restrict__ bad_flag)
{
    const int64_t total = (int64_t)G * Lpad_tot;
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(t / Lpad_tot);
        const int i = (int)(t - (int64_t)g * Lpad_tot);
        const int64_t dst = dst_base + t;
        if (i < L_old) {
            const int64_t src = old_base + (int64_t)g * Lpad_old + i;
            copy_unit<E, I>(dK, dst, src);
            copy_unit<E, I>(dV, dst, src);
        } else {
            const int64_t src = (int64_t)(i - L_old) * G + g;
            const bool real = i < L_old + L_new;
            store_unit<E, I>(dK, dst, idxK, userK, src, real, n_entries, bad_flag);
            store_unit<E, I>(dV, dst, idxV, userV, src, real, n_entries, bad_flag);
        }
    }
}

template <typename E, typename I>
__global__ void materialize_kernel(int G, int n_entries, int D, CacheView cv, int64_t base, int L, int Lpad,
                                   E* __restrict__ K_out, E* __restrict__ V_out)
{
    const E* poolK = reinterpret_cast<const E*>(cv.poolK);
    const E* poolV = reinterpret_cast<const E*>(cv.poolV);
    const I* idxK = reinterpret_cast<const I*>(cv.idxK);
    const I* idxV = reinterpret_cast<const I*>(cv.idxV);
    const E* userK = reinterpret_cast<const E*>(cv.userK);
    const E* userV = reinterpret_cast<const E*>(cv.userV);
    const int duk = cv.full_k ? D : cv.d_user, duv = cv.full_v ? D : cv.d_user;
    const int64_t total = (int64_t)L * G * D;
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(t % D);
        const int64_t ig = t / D;
        const int g = (int)(ig % G);
        const int64_t i = ig / G;
        const int64_t unit = base + (int64_t)g * Lpad + i;
        K_out[t] = c < duk ? userK[unit * duk + c] : poolK[((int64_t)g * n_entries + (int64_t)idxK[unit]) * D + c];
        V_out[t] = c < duv ? userV[unit * duv + c] : poolV[((int64_t)g * n_entries + (int64_t)idxV[unit]) * D + c];
    }
}

// Range check of stored indices that did not go through pack_kernel (imported blobs).
template <typename I>
__global__ void check_indices_kernel(const I* __restrict__ a, const I* __restrict__ b, int64_t n, uint32_t n_entries,
                                     int* __restrict__ bad_flag)
{
    bool bad = false;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        bad |= (a && (uint32_t)a[i] >= n_entries) || (b && (uint32_t)b[i] >= n_entries);
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(bad_flag, 1);
}

inline int grid_for(int64_t total, int block)
{
    int64_t g = (total + block - 1) / block;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (int)g;
}

}  // namespace

cudaError_t launch_pool_layout(int dtype, int G, int m, int d_shared, int D, const void* src,
                               void* dst, cudaStream_t s)
{
    const int64_t rows = (int64_t)G * m;
    const int grid = grid_for(rows * D, 256);
    if (dtype == CKV_BF16)
        pool_layout_kernel<uint16_t><<<grid, 256, 0, s>>>((const uint16_t*)src, (uint16_t*)dst, rows,
                                                          d_shared, D);
    else
        pool_layout_kernel<uint32_t><<<grid, 256, 0, s>>>((const uint32_t*)src, (uint32_t*)dst, rows,
                                                          d_shared, D);
    return cudaGetLastError();
}

cudaError_t launch_pack(int dtype, int G, int n_entries, int idx_bytes, int n_users,
                        const int64_t* hist_off_dev, const int64_t* unit_off_dev,
                        int64_t total_units, int64_t arena_base, const int32_t* idxK,
                        const int32_t* idxV, const void* userK, const void* userV, const CacheView& cv, int D,
                        int* bad_flag, cudaStream_t s)
{
    if (total_units == 0) return cudaSuccess;
    const int grid = grid_for(total_units, 256);
    const SideDst dK{cv.full_k ? nullptr : const_cast<void*>(cv.idxK), const_cast<void*>(cv.userK), cv.full_k ? D : cv.d_user};
    const SideDst dV{cv.full_v ? nullptr : const_cast<void*>(cv.idxV), const_cast<void*>(cv.userV), cv.full_v ? D : cv.d_user};
#define CKV_PACK(E, I)                                                                          \
    pack_kernel<E, I><<<grid, 256, 0, s>>>(G, n_entries, n_users, hist_off_dev, unit_off_dev,   \
                                           total_units, arena_base, idxK, idxV, (const E*)userK, \
                                           (const E*)userV, dK, dV, bad_flag)
    if (dtype == CKV_BF16) {
        if (idx_bytes == 2) CKV_PACK(uint16_t, uint16_t); else CKV_PACK(uint16_t, int32_t);
    } else {
        if (idx_bytes == 2) CKV_PACK(uint32_t, uint16_t); else CKV_PACK(uint32_t, int32_t);
    }
#undef CKV_PACK
    return cudaGetLastError();
}

cudaError_t launch_append(int dtype, int G, int n_entries, int idx_bytes, int64_t old_base, int L_old,
                          int Lpad_old, int64_t dst_base, int L_new, int Lpad_tot, const int32_t* idxK,
                          const int32_t* idxV, const void* userK, const void* userV, const CacheView& cv, int D,
                          int* bad_flag, cudaStream_t s)
{
    const int64_t total = (int64_t)G * Lpad_tot;
    if (total == 0) return cudaSuccess;
    const int grid = grid_for(total, 256);
    const SideDst dK{cv.full_k ? nullptr : const_cast<void*>(cv.idxK), const_cast<void*>(cv.userK), cv.full_k ? D : cv.d_user};
    const SideDst dV{cv.full_v ? nullptr : const_cast<void*>(cv.idxV), const_cast<void*>(cv.userV), cv.full_v ? D : cv.d_user};
#define CKV_APPEND(E, I)                                                                                       \
    append_kernel<E, I><<<grid, 256, 0, s>>>(G, n_entries, old_base, L_old, Lpad_old, dst_base, L_new,        \
                                             Lpad_tot, idxK, idxV, (const E*)userK, (const E*)userV, dK, dV,  \
                                             bad_flag)
    if (dtype == CKV_BF16) {
        if (idx_bytes == 2) CKV_APPEND(uint16_t, uint16_t); else CKV_APPEND(uint16_t, int32_t);
    } else {
        if (idx_bytes == 2) CKV_APPEND(uint32_t, uint16_t); else CKV_APPEND(uint32_t, int32_t);
    }
#undef CKV_APPEND
    return cudaGetLastError();
}

cudaError_t launch_materialize(int dtype, int D, const CacheView& cv, int64_t base, int L, int Lpad,
                               void* K_out, void* V_out, cudaStream_t s)
{
    if (L == 0) return cudaSuccess;
    const int grid = grid_for((int64_t)L * cv.n_groups * D, 256);
#define CKV_MAT(E, I)                                                                            \
    materialize_kernel<E, I><<<grid, 256, 0, s>>>(cv.n_groups, cv.n_entries, D, cv, base, L, Lpad, \
                                                  (E*)K_out, (E*)V_out)
    if (dtype == CKV_BF16) {
        if (cv.idx_bytes == 2) CKV_MAT(uint16_t, uint16_t); else CKV_MAT(uint16_t, int32_t);
    } else {
        if (cv.idx_bytes == 2) CKV_MAT(uint32_t, uint16_t); else CKV_MAT(uint32_t, int32_t);
    }
#undef CKV_MAT
    return cudaGetLastError();
}

cudaError_t launch_check_indices(int idx_bytes, int n_entries, const void* idxK, const void* idxV, int64_t n_units,
                                 int* bad_flag, cudaStream_t s)
{
    if (n_units == 0) return cudaSuccess;
    const int grid = grid_for(n_units, 256);
    if (idx_bytes == 2)
        check_indices_kernel<uint16_t><<<grid, 256, 0, s>>>((const uint16_t*)idxK, (const uint16_t*)idxV, n_units,
                                                            (uint32_t)n_entries, bad_flag);
    else
        check_indices_kernel<int32_t><<<grid, 256, 0, s>>>((const int32_t*)idxK, (const int32_t*)idxV, n_units,
                                                           (uint32_t)n_entries, bad_flag);
    return cudaGetLastError();
}

}  // namespace ckv
