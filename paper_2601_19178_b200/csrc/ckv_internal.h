// Internal declarations shared by the host side of the library and its kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ckv.h"

namespace ckv {

// One request row of an attend plan: where the user's compressed history lives in the
// arena and which query rows belong to it.
struct Req {
    int64_t base;      // first arena unit of the user; unit(g, i) = base + g * Lpad + i
    int32_t L;         // history length
    int32_t Lpad;      // L rounded up to a multiple of 32
    int32_t q0;        // first query row
    int32_t M;         // number of query rows
    int32_t part0;     // first partial-result row block (split requests), else -1
    int32_t n_chunks;  // history chunks this request was cut into (>= 1)
};

// One unit of kernel work: a contiguous chunk of one request's history, for every group.
struct Item {
    int32_t req;
    int32_t begin;     // first position of the chunk
    int32_t len;       // positions in the chunk (0 only for an empty history)
    int32_t part_row;  // first row of this chunk's partial results, or -1: write `out`
};

// An Item merged with its request row, for kernels that read their work list once per unit
// with plain 16-byte loads (48 bytes, 16-byte aligned).
struct Work {
    int64_t base;      // Req::base
    int32_t L, Lpad;   // Req::L, Req::Lpad
    int32_t q0, M;     // Req::q0, Req::M
    int32_t begin, len, part_row;  // Item::begin, Item::len, Item::part_row
    int32_t pad[3];    // [0]: with visible lengths, where the request's query blocks start in AttendArgs::vmax
};

// Everything a kernel needs to find the compressed cache and the pool.
struct CacheView {
    const void* poolK;   // [G][m][D] rows, first d_user slots zero
    const void* poolV;
    const void* idxK;    // arena, idx_bytes per unit
    const void* idxV;
    const void* userK;   // arena, d_user elements per unit
    const void* userV;
    int32_t n_groups;
    int32_t n_entries;
    int32_t d_user;      // user-specific elements per unit of a shared side
    int32_t idx_bytes;   // 2 or 4
    // Sharing only keys or only values: a side that is not shared has no pool and no indices (poolX, idxX
    // null); its userX array holds the full head_dim-wide row of every unit.
    int32_t full_k;
    int32_t full_v;
};

struct AttendArgs {
    CacheView cv;
    const Req* reqs;
    const Item* items;
    const Work* works;     // one per item, same order (tcgen05 family only, else null)
    int32_t n_items;
    const void* queries;   // [Q][G][D]
    const int32_t* vis;    // null, or per query row the number of leading history positions it attends [Q]
    const int32_t* vmax;   // tcgen05 family with visible lengths: largest limit per (request, block of 128 queries)
    void* out;             // [Q][G][D]
    float* partials;       // [part rows][G][D + 2]  (m, l, acc[D])
    int32_t out_dtype;     // ckv_dtype
    int32_t mode;          // ckv_mode
    float scale;
    // What the range-checked build (-DCKV_BOUNDS) compares against; unused otherwise.
    int64_t arena_units;   // units the arena arrays hold
    int64_t q_rows;        // rows of `queries` and `out`
    int64_t part_rows;     // rows of `partials`
    int* err;              // device error word (the context's)
};

// ---- kernels_pack.cu
cudaError_t launch_pool_layout(int dtype, int G, int m, int d_shared, int D, const void* src,
                               void* dst, cudaStream_t s);
// Packs n users' [P][G] indices and [P][G][d_user] user parts into arena units and
// validates index range; *bad_flag (device int) is OR-ed with 1 on a bad index.
// The arena arrays and the sides' widths come from `cv` (head_dim D).
cudaError_t launch_pack(int dtype, int G, int n_entries, int idx_bytes, int n_users,
                        const int64_t* hist_off_dev, const int64_t* unit_off_dev,
                        int64_t total_units, int64_t arena_base, const int32_t* idxK,
                        const int32_t* idxV, const void* userK, const void* userV, const CacheView& cv, int D,
                        int* bad_flag, cudaStream_t s);
// Writes a user's units for L_old + L_new positions at arena unit dst_base: the first L_old positions copied from
// the units at old_base (same arena), the rest packed from the new [L_new][G] indices and [L_new][G][d_user] parts.
cudaError_t launch_append(int dtype, int G, int n_entries, int idx_bytes, int64_t old_base, int L_old,
                          int Lpad_old, int64_t dst_base, int L_new, int Lpad_tot, const int32_t* idxK,
                          const int32_t* idxV, const void* userK, const void* userV, const CacheView& cv, int D,
                          int* bad_flag, cudaStream_t s);
cudaError_t launch_materialize(int dtype, int D, const CacheView& cv, int64_t base, int L, int Lpad,
                               void* K_out, void* V_out, cudaStream_t s);

// ORs 1 into *bad_flag (device int) if any of the n_units stored K or V indices is >= n_entries (idxK or idxV may be
// null: that side is not checked).
cudaError_t launch_check_indices(int idx_bytes, int n_entries, const void* idxK, const void* idxV, int64_t n_units,
                                 int* bad_flag, cudaStream_t s);

// ---- kernels_simt.cu : CUDA-core family (any number of queries, best for few)
cudaError_t launch_attend_simt(int dtype, int D, int max_M, const AttendArgs& a, cudaStream_t s);
// Merges the partial results of split requests into `out`.
cudaError_t launch_combine(int D, const AttendArgs& a, const int32_t* split_reqs, int n_split,
                           cudaStream_t s);

// ---- kernels_mma.cu : warp-level tensor-core family (bf16, head_dim 32 or 64, d_user <= 8)
bool mma_supported(int dtype, int head_dim, int d_user);  // d_user of the shared side(s)
int mma_queries_per_warp(int head_dim, int max_M);
// tensor_maps: null = fill the staging ring with cp.async copies; else the two maps of make_pool_tensor_maps =
// fill it with TMA gathers (err_flag: device int, OR-ed with a code if a bounded wait for a tile ran out).
cudaError_t launch_attend_mma(int head_dim, int max_M, const AttendArgs& a, const void* tensor_maps, int* err_flag,
                              cudaStream_t s);
bool make_pool_tensor_maps(int head_dim, int64_t rows, const void* poolK, const void* poolV, void* maps_out);

// ---- kernels_fact.cu : pool-side factorisation for one query per user (bf16, head_dim 32 or 64, d_user <= 8)
// Largest history the family can take for this shape (its tables and scores share one CTA's shared memory),
// or -1 if the shape is not supported.
int fact_max_history(int dtype, int head_dim, int d_user, int n_entries);
int fact_aux_floats();
int fact_row_floats(int n_entries);
// a.items: one unsplit item per request with a query.  tw: [n_req][G][fact_row_floats(n_entries)] floats,
// aux: [n_req][G][fact_aux_floats()].
cudaError_t launch_attend_fact(int head_dim, const AttendArgs& a, int n_req, int max_L, int n_sms, float* tw,
                               float* aux, cudaStream_t s);

// ---- kernels_route.cu : prefill router, fused scores + row arg-max (bf16, d_in 32 / 64 / 128)
bool route_supported(int d_in);
// out[i][g] = lowest entry j maximising x_i . W[g][j] + bias[g][j]; x [n][d_in], W [G][n_entries][d_in] bf16 (device),
// bias [G][n_entries] fp32 or null, out [n][G] int32.
cudaError_t launch_route(int d_in, const void* x, const void* W, const float* bias, int n, int n_entries, int G,
                         int32_t* out, cudaStream_t s);

// ---- kernels_route_umma.cu : the same router on tcgen05 (TMEM accumulators, warp-specialised)
// err_flag: device int, OR-ed with a non-zero code if a bounded wait inside the kernel ran out (nothing is written then).
cudaError_t launch_route_umma(int d_in, const void* x, const void* W, const float* bias, int n, int n_entries, int G,
                              int32_t* out, int* err_flag, cudaStream_t s);

// out[i][g][c] = x_i . W[g][c] + bias[g][c] (bf16 in and out, fp32 sums); W [G][d_out][d_in], bias [G][d_out] or null.
bool project_supported(int d_in, int d_out, int n_groups);
cudaError_t launch_project(int d_in, int d_out, int G, const void* x, const void* W, const float* bias, int64_t n,
                           void* out, cudaStream_t s);

// ---- kernels_umma.cu : tcgen05 family (bf16, head_dim 32, d_user in {0, 1, 2, 4, 8}, 16-bit stored indices)
bool umma_supported(int dtype, int head_dim, int d_user, int idx_bytes);
// err_flag: device int, OR-ed with a non-zero code if a bounded wait inside the kernel ran out.
// Persistent: one CTA per SM (n_sms of them at most).
cudaError_t launch_attend_umma(int max_M, const AttendArgs& a, int n_sms, int* err_flag, cudaStream_t s);
// Fills vmax (one int per request and block of 128 queries, at Work::pad[0] + block) from a.vis; a.works as for the attend.
cudaError_t launch_vis_block_max(const AttendArgs& a, int32_t* vmax, cudaStream_t s);

}  // namespace ckv
