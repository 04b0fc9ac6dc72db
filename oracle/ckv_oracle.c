/*
 * CPU oracle for the CollectiveKV decode path.  TEST INFRASTRUCTURE ONLY:
 * it exists to check the CUDA library and to be timed as the CPU baseline.
 * It shares no code with the CUDA path and must never serve a product call.
 *
 * What it computes (paper Sec. 4.2, decode stage):
 *   Eq. (Kc):  K_c[i] = P_k[I_k[i]],   V_c[i] = P_v[I_v[i]]       (inference branch:
 *              no sigmoid factor, Sec. 4.3)
 *   Eq. (K) :  K[i] = concat(K_u[i], K_c[i]),  V[i] = concat(V_u[i], V_c[i]),
 *              d_a = d_u + d_g; the user-specific part is the FIRST d_u dims
 *              (discussion of the sharing mechanism, appendix).
 *   then the user's queries attend over K, V (Sec. 4.2, last sentence; Sec. 2.1
 *   target attention: every query is an independent 1 x d row):
 *     softmax mode : s_i = scale * <q, K[i]>,  p = softmax_i(s),  o = sum_i p_i V[i]
 *     pointwise    : o = (1/L_u) * sum_i silu(s_i) V[i],  silu(x) = x / (1 + exp(-x))
 *   A user with L_u = 0 yields a zero output row (the paper does not define the case).
 *
 * Inputs are taken at their stored precision (float32, or bfloat16 bit patterns
 * widened exactly); all arithmetic is double.  No blocking, no online softmax,
 * no reordering: scores are stored, the max is taken, then the weighted sum.
 *
 * ckv_oracle_attend_variants (further down) adds what the ablation on sharing only
 * keys or only values (Sec. 5.5) and self-attention over the cached sequence (Sec. 2.1)
 * need: a shared width per side and a visible length per query.
 *
 * Every function here is pinned by the CPU tests (closed forms, hand-worked
 * fixtures, a library attention routine, brute force); nothing is parity-unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_SOFTMAX = 0, ORACLE_SILU_OVER_L = 1 };

static double widen(const void* base, int64_t i, int dtype)
{
    if (dtype == ORACLE_F32) return (double)((const float*)base)[i];
    uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static size_t elem_size(int dtype) { return dtype == ORACLE_F32 ? 4 : 2; }

/* Eq. (Kc) + Eq. (K) for one (position, group): writes d_u + d_g doubles. */
static void rebuild_row(double* row, int dtype, int G, int m, int d_g, int d_u,
                        const void* pool, const int32_t* idx, const void* user,
                        int64_t pos, int g)
{
    int64_t j = idx[pos * G + g];
    for (int c = 0; c < d_u; ++c)
        row[c] = widen(user, (pos * G + g) * (int64_t)d_u + c, dtype);
    for (int c = 0; c < d_g; ++c)
        row[d_u + c] = widen(pool, ((int64_t)g * m + j) * d_g + c, dtype);
}

/*
 * Full-width K and V of one user, in the INPUT dtype (a pure copy, so the
 * result is a unique bit pattern):  K_out, V_out : [L][G][d_u + d_g].
 * `pos0` is the user's first row in idx_* / user_*.  Returns 0, or 1 when an
 * index is outside [0, m).
 */
int ckv_oracle_materialize(int dtype, int G, int m, int d_g, int d_u,
                           const void* pool_K, const void* pool_V,
                           const int32_t* idx_K, const int32_t* idx_V,
                           const void* user_K, const void* user_V,
                           int64_t pos0, int64_t L, void* K_out, void* V_out)
{
    const size_t e = elem_size(dtype);
    const int d = d_u + d_g;
    for (int64_t i = 0; i < L; ++i)
        for (int g = 0; g < G; ++g) {
            int64_t p = pos0 + i;
            int64_t jk = idx_K[p * G + g], jv = idx_V[p * G + g];
            if (jk < 0 || jk >= m || jv < 0 || jv >= m) return 1;
            char* ko = (char*)K_out + ((i * G + g) * (int64_t)d) * e;
            char* vo = (char*)V_out + ((i * G + g) * (int64_t)d) * e;
            memcpy(ko, (const char*)user_K + ((p * G + g) * (int64_t)d_u) * e, d_u * e);
            memcpy(vo, (const char*)user_V + ((p * G + g) * (int64_t)d_u) * e, d_u * e);
            memcpy(ko + d_u * e, (const char*)pool_K + (((int64_t)g * m + jk) * d_g) * e, d_g * e);
            memcpy(vo + d_u * e, (const char*)pool_V + (((int64_t)g * m + jv) * d_g) * e, d_g * e);
        }
    return 0;
}

/*
 * Attention of the selected users' queries over their rebuilt histories.
 *
 *   hist_off [U+1], q_off [U+1] : ragged offsets of all U users of the arrays
 *   sel [n_sel]                 : which users to compute (NULL => all U, in order)
 *   out                         : double [sum of selected users' M][G][d], packed
 *                                 in the order of `sel`
 * Returns 0, 1 on an out-of-range index, 2 on allocation failure.
 */
int ckv_oracle_attend(int dtype, int mode, double scale,
                      int G, int m, int d_g, int d_u,
                      const void* pool_K, const void* pool_V,
                      int64_t U, const int64_t* hist_off,
                      const int32_t* idx_K, const int32_t* idx_V,
                      const void* user_K, const void* user_V,
                      const int64_t* q_off, const void* queries,
                      int64_t n_sel, const int64_t* sel,
                      double* out, int n_threads)
{
    const int d = d_u + d_g;
    if (sel == NULL) n_sel = U;
    /* packed output offset of every selected user */
    int64_t* out_row = (int64_t*)malloc((size_t)(n_sel + 1) * sizeof(int64_t));
    if (!out_row) return 2;
    out_row[0] = 0;
    for (int64_t s = 0; s < n_sel; ++s) {
        int64_t u = sel ? sel[s] : s;
        out_row[s + 1] = out_row[s] + (q_off[u + 1] - q_off[u]);
    }
    int status = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t s = 0; s < n_sel; ++s) {
        const int64_t u = sel ? sel[s] : s;
        const int64_t p0 = hist_off[u], L = hist_off[u + 1] - hist_off[u];
        const int64_t q0 = q_off[u], M = q_off[u + 1] - q_off[u];
        double* K = (double*)malloc((size_t)(L > 0 ? L : 1) * d * sizeof(double));
        double* V = (double*)malloc((size_t)(L > 0 ? L : 1) * d * sizeof(double));
        double* sc = (double*)malloc((size_t)(L > 0 ? L : 1) * sizeof(double));
        if (!K || !V || !sc) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            status = 2;
            free(K); free(V); free(sc);
            continue;
        }
        for (int g = 0; g < G; ++g) {
            int bad = 0;
            for (int64_t i = 0; i < L; ++i) {
                int64_t jk = idx_K[(p0 + i) * G + g], jv = idx_V[(p0 + i) * G + g];
                if (jk < 0 || jk >= m || jv < 0 || jv >= m) { bad = 1; break; }
                rebuild_row(K + i * d, dtype, G, m, d_g, d_u, pool_K, idx_K, user_K, p0 + i, g);
                rebuild_row(V + i * d, dtype, G, m, d_g, d_u, pool_V, idx_V, user_V, p0 + i, g);
            }
            if (bad) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
                status = 1;
                break;
            }
            for (int64_t r = 0; r < M; ++r) {
                double* o = out + ((out_row[s] + r) * G + g) * (int64_t)d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                if (L == 0) continue;
                double smax = -INFINITY;
                for (int64_t i = 0; i < L; ++i) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c)
                        acc += widen(queries, ((q0 + r) * G + g) * (int64_t)d + c, dtype) * K[i * d + c];
                    sc[i] = scale * acc;
                    if (sc[i] > smax) smax = sc[i];
                }
                if (mode == ORACLE_SOFTMAX) {
                    double denom = 0.0;
                    for (int64_t i = 0; i < L; ++i) {
                        sc[i] = exp(sc[i] - smax);
                        denom += sc[i];
                    }
                    for (int64_t i = 0; i < L; ++i) {
                        double p = sc[i] / denom;
                        for (int c = 0; c < d; ++c) o[c] += p * V[i * d + c];
                    }
                } else {
                    for (int64_t i = 0; i < L; ++i) {
                        double w = sc[i] / (1.0 + exp(-sc[i])) / (double)L;
                        for (int c = 0; c < d; ++c) o[c] += w * V[i * d + c];
                    }
                }
            }
        }
        free(K); free(V); free(sc);
    }
    free(out_row);
    return status;
}

/*
 * Variants of the decode path (same plain definition, more general inputs):
 *
 *  - Sharing only the keys or only the values (ablation study, Sec. 5.5, the table on sharing
 *    keys or values: "CollectiveK" shares the keys and keeps classical values, "CollectiveV"
 *    the reverse).  Each side has its own shared width: d_gk for K, d_gv for V.  A side with
 *    shared width 0 has no pool and no indices: its cached part is the full d_a-wide row, as
 *    in a classical KV cache.  Otherwise Eq. (Kc) / Eq. (K) apply to that side with
 *    d_u = d_a - d_g, user part first.
 *  - Self-attention over the cached sequence (Sec. 2.1: in self-attention models the s queries
 *    come from the sequence itself).  The paper does not restate the mask; the reading taken
 *    here is a per-query visible length: query row r attends positions 0 .. vis[r]-1 of its
 *    user's history (causal self-attention is vis[i] = i + 1; vis NULL means every query sees
 *    all L_u positions).  vis[r] = 0 gives a zero row.  In pointwise mode the divisor stays the
 *    user's history length L_u (HSTU normalises by the sequence length, not by the number of
 *    visible positions).
 *
 *   pool_K [G][m][d_gk] (ignored when d_gk = 0), pool_V [G][m][d_gv] (ignored when d_gv = 0)
 *   idx_K, idx_V [P][G]  (ignored for a side without a pool)
 *   user_K [P][G][d_a - d_gk], user_V [P][G][d_a - d_gv]
 *   vis    int32 [Q] indexed like the query rows, or NULL
 * Other arguments and the return value as ckv_oracle_attend; 3 = some vis[r] outside [0, L_u].
 */
static void rebuild_side(double* row, int dtype, int G, int m, int d_a, int d_g,
                         const void* pool, const int32_t* idx, const void* cached,
                         int64_t pos, int g)
{
    const int d_u = d_a - d_g;
    for (int c = 0; c < d_u; ++c)
        row[c] = widen(cached, (pos * G + g) * (int64_t)d_u + c, dtype);
    if (d_g > 0) {
        const int64_t j = idx[pos * G + g];
        for (int c = 0; c < d_g; ++c)
            row[d_u + c] = widen(pool, ((int64_t)g * m + j) * d_g + c, dtype);
    }
}

int ckv_oracle_attend_variants(int dtype, int mode, double scale,
                               int G, int m, int d_a, int d_gk, int d_gv,
                               const void* pool_K, const void* pool_V,
                               int64_t U, const int64_t* hist_off,
                               const int32_t* idx_K, const int32_t* idx_V,
                               const void* user_K, const void* user_V,
                               const int64_t* q_off, const void* queries, const int32_t* vis,
                               int64_t n_sel, const int64_t* sel,
                               double* out, int n_threads)
{
    const int d = d_a;
    if (sel == NULL) n_sel = U;
    int64_t* out_row = (int64_t*)malloc((size_t)(n_sel + 1) * sizeof(int64_t));
    if (!out_row) return 2;
    out_row[0] = 0;
    for (int64_t s = 0; s < n_sel; ++s) {
        int64_t u = sel ? sel[s] : s;
        out_row[s + 1] = out_row[s] + (q_off[u + 1] - q_off[u]);
    }
    int status = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t s = 0; s < n_sel; ++s) {
        const int64_t u = sel ? sel[s] : s;
        const int64_t p0 = hist_off[u], L = hist_off[u + 1] - hist_off[u];
        const int64_t q0 = q_off[u], M = q_off[u + 1] - q_off[u];
        double* K = (double*)malloc((size_t)(L > 0 ? L : 1) * d * sizeof(double));
        double* V = (double*)malloc((size_t)(L > 0 ? L : 1) * d * sizeof(double));
        double* sc = (double*)malloc((size_t)(L > 0 ? L : 1) * sizeof(double));
        if (!K || !V || !sc) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            status = 2;
            free(K); free(V); free(sc);
            continue;
        }
        for (int g = 0; g < G; ++g) {
            int bad = 0;
            for (int64_t i = 0; i < L; ++i) {
                if (d_gk > 0) {
                    int64_t jk = idx_K[(p0 + i) * G + g];
                    if (jk < 0 || jk >= m) { bad = 1; break; }
                }
                if (d_gv > 0) {
                    int64_t jv = idx_V[(p0 + i) * G + g];
                    if (jv < 0 || jv >= m) { bad = 1; break; }
                }
                rebuild_side(K + i * d, dtype, G, m, d_a, d_gk, pool_K, idx_K, user_K, p0 + i, g);
                rebuild_side(V + i * d, dtype, G, m, d_a, d_gv, pool_V, idx_V, user_V, p0 + i, g);
            }
            for (int64_t r = 0; r < M && !bad; ++r)
                if (vis && (vis[q0 + r] < 0 || vis[q0 + r] > L)) bad = 3;
            if (bad) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
                status = bad;
                break;
            }
            for (int64_t r = 0; r < M; ++r) {
                double* o = out + ((out_row[s] + r) * G + g) * (int64_t)d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                const int64_t n_vis = vis ? vis[q0 + r] : L;   /* the query sees positions [0, n_vis) */
                if (n_vis == 0) continue;
                double smax = -INFINITY;
                for (int64_t i = 0; i < n_vis; ++i) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c)
                        acc += widen(queries, ((q0 + r) * G + g) * (int64_t)d + c, dtype) * K[i * d + c];
                    sc[i] = scale * acc;
                    if (sc[i] > smax) smax = sc[i];
                }
                if (mode == ORACLE_SOFTMAX) {
                    double denom = 0.0;
                    for (int64_t i = 0; i < n_vis; ++i) {
                        sc[i] = exp(sc[i] - smax);
                        denom += sc[i];
                    }
                    for (int64_t i = 0; i < n_vis; ++i) {
                        double p = sc[i] / denom;
                        for (int c = 0; c < d; ++c) o[c] += p * V[i * d + c];
                    }
                } else {
                    for (int64_t i = 0; i < n_vis; ++i) {
                        double w = sc[i] / (1.0 + exp(-sc[i])) / (double)L;
                        for (int c = 0; c < d; ++c) o[c] += w * V[i * d + c];
                    }
                }
            }
        }
        free(K); free(V); free(sc);
    }
    free(out_row);
    return status;
}

/*
 * Full-width rows of ONE side (K or V) of one user, in the input dtype, for a side with
 * shared width d_g (0: the cached part already is the full row): out [L][G][d_a].
 * Returns 0, or 1 when an index is outside [0, m).
 */
int ckv_oracle_materialize_side(int dtype, int G, int m, int d_a, int d_g,
                                const void* pool, const int32_t* idx, const void* cached,
                                int64_t pos0, int64_t L, void* out)
{
    const size_t e = elem_size(dtype);
    const int d_u = d_a - d_g;
    for (int64_t i = 0; i < L; ++i)
        for (int g = 0; g < G; ++g) {
            const int64_t p = pos0 + i;
            char* o = (char*)out + ((i * G + g) * (int64_t)d_a) * e;
            memcpy(o, (const char*)cached + ((p * G + g) * (int64_t)d_u) * e, d_u * e);
            if (d_g > 0) {
                const int64_t j = idx[p * G + g];
                if (j < 0 || j >= m) return 1;
                memcpy(o + d_u * e, (const char*)pool + (((int64_t)g * m + j) * d_g) * e, d_g * e);
            }
        }
    return 0;
}

/*
 * Storage accounting of the latency analysis (Sec. 4.4): a classical cache
 * holds s*d_a elements per K (or V) sequence, the compressed one s*d_u + s
 * (user-specific part plus one index element per position).  The compression
 * rate of Sec. 5.1 is their ratio.
 */
double ckv_oracle_compression_rate(int d_a, int d_u)
{
    return ((double)d_u + 1.0) / (double)d_a;
}

int ckv_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
