// Host side of the library: context, pool and compressed-cache management, attend
// planning (history chunking for the split-along-history reduction) and kernel dispatch.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "ckv_internal.h"

using namespace ckv;

namespace {

struct UserEntry {
    int64_t base;
    int32_t L;
    int32_t Lpad;
};

// User id -> cache entry: open addressing with linear probing and backward-shift deletion.  A decode
// call looks up every user of its request list, so a lookup has to cost one cache line, not a node chase.
class UserTable {
    struct Slot {
        int64_t key;
        UserEntry e;
        uint32_t used;
    };
    std::vector<Slot> slots_;
    size_t n_ = 0, mask_ = 0;
    static size_t hash(int64_t k)
    {
        uint64_t x = (uint64_t)k + 0x9e3779b97f4a7c15ull;
        x = (x ^ (x >> 30)) * 0xbf58476d1ce4e5b9ull;
        x = (x ^ (x >> 27)) * 0x94d049bb133111ebull;
        return (size_t)(x ^ (x >> 31));
    }
    void rehash(size_t cap)
    {
        std::vector<Slot> old;
        old.swap(slots_);
        slots_.assign(cap, Slot{0, {0, 0, 0}, 0});
        mask_ = cap - 1;
        n_ = 0;
        for (const Slot& sl : old)
            if (sl.used) *insert(sl.key) = sl.e;
    }

public:
    size_t size() const { return n_; }
    bool empty() const { return n_ == 0; }
    void clear()
    {
        slots_.clear();
        n_ = mask_ = 0;
    }
    const UserEntry* find(int64_t key) const
    {
        if (n_ == 0) return nullptr;
        for (size_t i = hash(key) & mask_;; i = (i + 1) & mask_) {
            const Slot& sl = slots_[i];
            if (!sl.used) return nullptr;
            if (sl.key == key) return &sl.e;
        }
    }
    UserEntry* find(int64_t key) { return const_cast<UserEntry*>(static_cast<const UserTable*>(this)->find(key)); }
    // a hint that `key` is about to be looked up (a request list names tens of thousands of users whose slots
    // are scattered over a table larger than the host's caches)
    void prefetch(int64_t key) const
    {
        if (n_) __builtin_prefetch(&slots_[hash(key) & mask_]);
    }
    // the entry of `key`, created (zeroed) if absent; may throw std::bad_alloc
    UserEntry* insert(int64_t key)
    {
        if (slots_.empty() || (n_ + 1) * 2 > slots_.size()) rehash(slots_.empty() ? 64 : slots_.size() * 2);
        for (size_t i = hash(key) & mask_;; i = (i + 1) & mask_) {
            Slot& sl = slots_[i];
            if (!sl.used) {
                sl.used = 1;
                sl.key = key;
                sl.e = UserEntry{0, 0, 0};
                ++n_;
                return &sl.e;
            }
            if (sl.key == key) return &sl.e;
        }
    }
    bool erase(int64_t key)
    {
        if (n_ == 0) return false;
        size_t i = hash(key) & mask_;
        for (;; i = (i + 1) & mask_) {
            if (!slots_[i].used) return false;
            if (slots_[i].key == key) break;
        }
        // close the gap: move back every follower whose home slot is not inside (i, j]
        for (size_t j = (i + 1) & mask_; slots_[j].used; j = (j + 1) & mask_) {
            const size_t h = hash(slots_[j].key) & mask_;
            const bool stays = i <= j ? (h > i && h <= j) : (h > i || h <= j);
            if (!stays) {
                slots_[i] = slots_[j];
                i = j;
            }
        }
        slots_[i].used = 0;
        --n_;
        return true;
    }
    // room for `extra` more users, so that `insert` cannot fail half-way through a batch
    void reserve_more(size_t extra)
    {
        size_t cap = slots_.empty() ? 64 : slots_.size();
        while ((n_ + extra) * 2 > cap) cap *= 2;
        if (cap != slots_.size()) rehash(cap);
    }
};

constexpr int kMaxRanges = 8;

struct DevBuf {  // grow-only device buffer
    void* p = nullptr;
    size_t cap = 0;
};

// A cached attend plan.  Its tables live in one pinned host block and one device block that the slot keeps
// (grow-only) when another request list takes it over, so a new request list costs no allocation once the
// blocks have reached their size.
struct Plan {
    bool live = false;
    std::vector<int64_t> users;
    std::vector<int32_t> q_off;
    uint64_t generation = 0;
    int64_t opt_split = 0, opt_kernel = 0;
    bool with_vis = false;   // planned for a call with visible lengths (other kernel choice)
    // The request list cut into n_ranges runs of consecutive users (host-buffer calls are pipelined range by
    // range): items and the split list are grouped by range, r_item / r_split give each range's slice.
    int32_t n_ranges = 1;
    int32_t r_user[kMaxRanges + 1] = {}, r_item[kMaxRanges + 1] = {}, r_split[kMaxRanges + 1] = {};
    DevBuf dev;              // reqs | items | split list | works
    void* host = nullptr;    // pinned mirror the tables are built in
    size_t host_cap = 0;
    cudaEvent_t uploaded = nullptr;  // recorded behind the last upload from `host`
    Req* d_reqs = nullptr;
    Item* d_items = nullptr;
    int32_t* d_split = nullptr;
    Work* d_works = nullptr;
    int32_t n_items = 0, n_split = 0, split_items = 0, max_M = 0, max_L = 0, n_req = 0, family = 1, n_vblocks = 0;
    int64_t part_rows = 0;
    uint64_t last_use = 0;
};

constexpr int kMaxPlans = 4;

struct DeviceGuard {
    int prev = -1;
    bool ok;
    explicit DeviceGuard(int dev)
    {
        ok = cudaGetDevice(&prev) == cudaSuccess;
        if (ok && prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace

struct ckv_ctx {
    ckv_config cfg{};
    float scale = 1.f;
    int elem = 2;  // bytes per element of cfg.dtype
    int n_sms = 148;
    // pool
    int n_entries = 0, d_shared = 0, d_user = 0, idx_bytes = 0;
    bool full_k = false, full_v = false;  // the side is not shared: cached full width, no pool, no indices
    void* pool = nullptr;  // K rows then V rows, each [G][m][D] (a side that is not shared has none)
    bool has_mma = false;         // the warp-level tensor-core family can run
    bool has_tma = false;         // ... and its TMA-gather loader too (tensor maps of the pool encoded)
    alignas(64) unsigned char tmaps[256] = {};  // two CUtensorMap: K pool, V pool
    bool has_umma = false;
    int* d_err = nullptr;  // OR of error codes from kernels whose bounded waits ran out
    size_t pool_half = 0;  // bytes of one side's rows
    int n_pool_sides = 2;  // sides that have a pool
    // arena of compressed caches (units = (position, group) slots).  Units [0, used_units) are handed out;
    // runs inside that range given back by evicted, replaced or appended-to users wait in free_runs
    // (first unit -> length, neighbours merged) and are reused first-fit.
    void *a_idxK = nullptr, *a_idxV = nullptr, *a_userK = nullptr, *a_userV = nullptr;
    int64_t cap_units = 0, used_units = 0, live_positions = 0;
    std::map<int64_t, int64_t> free_runs;
    UserTable users;
    uint64_t generation = 1;
    // scratch
    DevBuf stage_q, stage_out, stage_vis, vmax, partials;
    int* d_flag = nullptr;
    Plan plans[kMaxPlans];
    uint64_t tick = 0;
    // options
    int64_t opt_split = 0, opt_kernel = 0, opt_l2 = 1, opt_time = 0, opt_loader = 0;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};  // around the main kernel and the combine
    bool ev_valid = false;
    // host-buffer calls: one internal stream per range of users, so that the upload of one range, the kernels of
    // another and the download of a third overlap; events tie them to the caller's stream at both ends
    cudaStream_t pipe_stream[kMaxRanges] = {};
    cudaEvent_t pipe_start = nullptr, pipe_plan = nullptr, pipe_h2d[kMaxRanges] = {}, pipe_done[kMaxRanges] = {};
    bool pipe_ready = false;
    // L2 residency of the pool: an access-policy window over the pool allocation is put on the caller's
    // stream around the kernels of a decode call and taken off again before the call returns
    bool l2_ready = false;       // the persisting-L2 carve-out of this device was raised for this context
    size_t l2_window = 0;        // bytes of the window (0: not available)
    float l2_ratio = 1.f;
    // statistics of the last attend
    int64_t st_launches = 0, st_items = 0, st_split = 0, st_kernel = 0, st_ws = 0, st_hit = 0, st_loader = 0,
            st_allocs = 0, st_l2 = 0, st_ranges = 1;
    std::string cuda_err;

    ckv_status fail(cudaError_t e)
    {
        cuda_err = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e);
        cudaGetLastError();  // clear the sticky-free error state
        return e == cudaErrorMemoryAllocation ? CKV_ERR_OOM : CKV_ERR_CUDA;
    }
};

#define CK(call)                                        \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) return ctx->fail(e_);    \
    } while (0)

namespace {

bool is_device_ptr(const void* p)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

// A temporary device copy of host input, freed by the destructor.
struct Staged {
    const void* dev = nullptr;
    void* owned = nullptr;
    ~Staged()
    {
        if (owned) cudaFree(owned);
    }
    cudaError_t init(const void* src, size_t bytes, cudaStream_t s)
    {
        if (bytes == 0 || src == nullptr || is_device_ptr(src)) {
            dev = src;
            return cudaSuccess;
        }
        cudaError_t e = cudaMalloc(&owned, bytes);
        if (e != cudaSuccess) return e;
        dev = owned;
        return cudaMemcpyAsync(owned, src, bytes, cudaMemcpyHostToDevice, s);
    }
};

cudaError_t grow(DevBuf& b, size_t bytes, int64_t* allocs = nullptr)
{
    if (bytes <= b.cap) return cudaSuccess;
    if (allocs) ++*allocs;
    if (b.p) {
        cudaError_t e = cudaFree(b.p);  // waits for work that may still use it
        b.p = nullptr;
        b.cap = 0;
        if (e != cudaSuccess) return e;
    }
    size_t want = bytes + bytes / 4;
    cudaError_t e = cudaMalloc(&b.p, want);
    if (e != cudaSuccess) {
        cudaGetLastError();
        want = bytes;
        e = cudaMalloc(&b.p, want);
        if (e != cudaSuccess) return e;
    }
    b.cap = want;
    return cudaSuccess;
}

void free_plan(Plan& p)
{
    if (p.dev.p) cudaFree(p.dev.p);
    if (p.host) cudaFreeHost(p.host);
    if (p.uploaded) cudaEventDestroy(p.uploaded);
    p = Plan();
}

void drop_plans(ckv_ctx* ctx)
{
    for (auto& p : ctx->plans) free_plan(p);
}

CacheView view_of(const ckv_ctx* ctx)
{
    CacheView v;
    v.poolK = ctx->full_k ? nullptr : ctx->pool;
    v.poolV = ctx->full_v ? nullptr : (const char*)ctx->pool + (ctx->full_k ? 0 : ctx->pool_half);
    v.idxK = ctx->a_idxK;
    v.idxV = ctx->a_idxV;
    v.userK = ctx->a_userK;
    v.userV = ctx->a_userV;
    v.n_groups = ctx->cfg.n_groups;
    v.n_entries = ctx->n_entries;
    v.d_user = ctx->d_user;
    v.idx_bytes = ctx->idx_bytes;
    v.full_k = ctx->full_k;
    v.full_v = ctx->full_v;
    return v;
}

// Bytes one unit takes in the four arena arrays: K indices, V indices, K user part, V user part.  A side that
// is not shared keeps no index and the whole head_dim-wide row.
void unit_bytes(const ckv_ctx* ctx, int64_t (&eb)[4])
{
    const int64_t D = ctx->cfg.head_dim;
    eb[0] = ctx->full_k ? 0 : ctx->idx_bytes;
    eb[1] = ctx->full_v ? 0 : ctx->idx_bytes;
    eb[2] = (ctx->full_k ? D : ctx->d_user) * ctx->elem;
    eb[3] = (ctx->full_v ? D : ctx->d_user) * ctx->elem;
}

// Capacity for units [0, need_end), keeping what is stored.
ckv_status ensure_arena(ckv_ctx* ctx, int64_t need_end, cudaStream_t s)
{
    if (need_end <= ctx->cap_units) return CKV_OK;
    int64_t cap = std::max<int64_t>(ctx->cap_units * 2, need_end);
    cap = (cap + 1023) / 1024 * 1024;
    int64_t eb[4];
    unit_bytes(ctx, eb);
    void* n[4] = {nullptr, nullptr, nullptr, nullptr};
    void* old[4] = {ctx->a_idxK, ctx->a_idxV, ctx->a_userK, ctx->a_userV};
    for (int i = 0; i < 4; ++i) {
        if (eb[i] == 0) continue;  // nothing is stored there (no user part, or no indices on a side that is not shared)
        cudaError_t e = cudaMalloc(&n[i], (size_t)cap * eb[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j)
                if (n[j]) cudaFree(n[j]);
            return ctx->fail(e);
        }
    }
    for (int i = 0; i < 4; ++i)
        if (eb[i] && ctx->used_units) {
            cudaError_t e = cudaMemcpyAsync(n[i], old[i], (size_t)ctx->used_units * eb[i], cudaMemcpyDeviceToDevice, s);
            if (e != cudaSuccess) {
                for (int j = 0; j < 4; ++j)
                    if (n[j]) cudaFree(n[j]);
                return ctx->fail(e);
            }
        }
    CK(cudaStreamSynchronize(s));
    for (int i = 0; i < 4; ++i)
        if (old[i]) cudaFree(old[i]);
    ctx->a_idxK = n[0];
    ctx->a_idxV = n[1];
    ctx->a_userK = n[2];
    ctx->a_userV = n[3];
    ctx->cap_units = cap;
    return CKV_OK;
}

// A run of `units` contiguous arena units: the first free run that is large enough, else fresh units behind
// everything handed out so far (growing the arena if need be).
ckv_status arena_take(ckv_ctx* ctx, int64_t units, cudaStream_t s, int64_t* base)
{
    for (auto it = ctx->free_runs.begin(); it != ctx->free_runs.end(); ++it) {
        if (it->second < units) continue;
        *base = it->first;
        const int64_t rest = it->second - units;
        ctx->free_runs.erase(it);
        if (rest > 0) ctx->free_runs.emplace(*base + units, rest);
        return CKV_OK;
    }
    ckv_status st = ensure_arena(ctx, ctx->used_units + units, s);
    if (st != CKV_OK) return st;
    *base = ctx->used_units;
    ctx->used_units += units;
    return CKV_OK;
}

// Gives a run back.  Work already enqueued on the context's stream may still read it; whatever reuses it is
// enqueued behind that work on the same stream.
void arena_give(ckv_ctx* ctx, int64_t base, int64_t units)
{
    if (units <= 0) return;
    try {
        auto it = ctx->free_runs.emplace(base, units).first;
        auto nx = std::next(it);
        if (nx != ctx->free_runs.end() && it->first + it->second == nx->first) {
            it->second += nx->second;
            ctx->free_runs.erase(nx);
        }
        if (it != ctx->free_runs.begin()) {
            auto pv = std::prev(it);
            if (pv->first + pv->second == it->first) {
                pv->second += it->second;
                ctx->free_runs.erase(it);
                it = pv;
            }
        }
        if (it->first + it->second == ctx->used_units) {  // the run touches the end: shrink instead of keeping it
            ctx->used_units = it->first;
            ctx->free_runs.erase(it);
        }
    } catch (const std::bad_alloc&) {
        // the run is lost until the arena is cleared; nothing else depends on it
    }
}

int64_t units_of_len(const ckv_ctx* ctx, int64_t L) { return (int64_t)ctx->cfg.n_groups * ((L + 31) / 32 * 32); }

int64_t auto_split_len(const ckv_ctx* ctx, int64_t total_positions, int family, int max_M)
{
    // Enough (chunk, group) blocks to fill the SMs several times over, but chunks long
    // enough that the merge of partial results stays a small fraction of the work.
    int64_t c;
    if (family == 3) {  // persistent CTAs share (chunk, group, 128 queries) units round-robin: a few units per SM
        c = total_positions * ctx->cfg.n_groups * ((max_M + 127) / 128) / (ctx->n_sms * 4);
        c = (c + 127) / 128 * 128;
        return std::min<int64_t>(std::max<int64_t>(c, 1024), 16384);
    }
    if (family == 2) {
        const int qpw = mma_queries_per_warp(ctx->cfg.head_dim, max_M);
        c = total_positions * ctx->cfg.n_groups * ((max_M + qpw - 1) / qpw) / (ctx->n_sms * 32);
        c = (c + 63) / 64 * 64;
        return std::min<int64_t>(std::max<int64_t>(c, 256), 4096);
    }
    c = total_positions * ctx->cfg.n_groups / (ctx->n_sms * 16);
    c = (c + 63) / 64 * 64;
    return std::min<int64_t>(std::max<int64_t>(c, 256), 2048);
}

// Orders the item indices [begin, end) by descending chunk length, equal lengths in their original order (two
// 16-bit counting passes over the complemented length: linear in the number of items).
void order_longest_first(const std::vector<Item>& items, size_t begin, size_t end, std::vector<uint32_t>& order,
                         std::vector<uint32_t>& tmp, std::vector<uint32_t>& count)
{
    const size_t n = end - begin;
    bool same = true;
    for (size_t i = begin; i < end; ++i) {
        order[i] = (uint32_t)i;
        same = same && items[i].len == items[begin].len;
    }
    if (same || n < 2) return;
    tmp.resize(items.size());
    count.resize(65536 + 1);
    for (int pass = 0; pass < 2; ++pass) {
        const int shift = 16 * pass;
        std::fill(count.begin(), count.end(), 0u);
        for (size_t i = begin; i < end; ++i) ++count[((~(uint32_t)items[order[i]].len >> shift) & 0xffffu) + 1];
        for (size_t d = 0; d < 65536; ++d) count[d + 1] += count[d];
        for (size_t i = begin; i < end; ++i)
            tmp[begin + count[(~(uint32_t)items[order[i]].len >> shift) & 0xffffu]++] = order[i];
        std::copy(tmp.begin() + begin, tmp.begin() + end, order.begin() + begin);
    }
}

ckv_status build_plan(ckv_ctx* ctx, Plan& pl, int32_t n, const int64_t* users, const int32_t* q_off, bool with_vis,
                      int n_ranges, const int32_t* r_user, cudaStream_t s)
{
    std::vector<Req> reqs((size_t)n);
    int64_t total_pos = 0, n_active = 0;
    int32_t max_M = 0, max_L = 0;
    bool all_single = true;
    for (int32_t k = 0; k < n; ++k) {
        if (k + 12 < n) ctx->users.prefetch(users[k + 12]);
        const UserEntry* f = ctx->users.find(users[k]);
        if (!f) return CKV_ERR_UNKNOWN_USER;
        Req& r = reqs[k];
        r.base = f->base;
        r.L = f->L;
        r.Lpad = f->Lpad;
        r.q0 = q_off[k];
        r.M = q_off[k + 1] - q_off[k];
        r.part0 = -1;
        r.n_chunks = 1;
        if (r.M > 0) {
            total_pos += r.L;
            max_L = std::max(max_L, r.L);
            n_active++;
            all_single = all_single && r.M == 1;
        }
        max_M = std::max(max_M, r.M);
    }
    pl.max_M = max_M;
    pl.max_L = max_L;
    pl.n_req = n;
    const bool can_mma = ctx->has_mma;
    // visible lengths and sides that are not shared are served by every gathering kernel, not by the pool-side
    // factorisation
    const bool plain = !with_vis && !ctx->full_k && !ctx->full_v;
    const bool can_umma = ctx->has_umma;
    // tcgen05 from three 16-query blocks on, else the warp-level tensor-core kernel (faster than the CUDA-core
    // kernel from a single query on); the CUDA-core kernel serves what neither supports
    // One query per user: the pool-side factorisation trades the row gathers for two tables per (user, group) in
    // HBM (n_entries floats per request and group: not beyond 2 GiB of workspace).
    const bool can_fact = plain && all_single && n_active > 0 &&
                          fact_max_history(ctx->cfg.dtype, ctx->cfg.head_dim, ctx->d_user, ctx->n_entries) >= max_L &&
                          (int64_t)n * ctx->cfg.n_groups * (fact_row_floats(ctx->n_entries) + fact_aux_floats()) *
                                  (int64_t)sizeof(float) <= ((int64_t)2 << 30);
    // It pays when histories are long against the pool and there are enough (user, group) pairs to fill the SMs
    // (one CTA holds a whole pair; the gathering kernel splits long histories over CTAs).  Cost lines fitted to
    // B200 measurements, in microseconds of one SM: a pair costs a + b n_entries + c L on the factorised path,
    // a position d on the gathering path.
    bool fact_pays = false;
    if (can_fact) {
        const bool wide = ctx->cfg.head_dim == 64;
        const double a = wide ? 4.8 : 4.7, b = wide ? 0.00032 : 0.00024, c = wide ? 0.0010 : 0.0008,
                     d = wide ? 0.0047 : 0.0025;
        const double pairs = (double)n_active * ctx->cfg.n_groups, mean_L = (double)total_pos / (double)n_active;
        const double waves = std::ceil(pairs / ctx->n_sms);
        const double t_fact = waves * (a + b * ctx->n_entries + c * mean_L);
        const double t_gather = d * (double)total_pos * ctx->cfg.n_groups / ctx->n_sms;
        fact_pays = t_fact < t_gather;
    }
    if (ctx->opt_kernel == 0)
        pl.family = can_umma && max_M >= 48 ? 3 : fact_pays ? 4 : can_mma ? 2 : 1;
    else if (ctx->opt_kernel == 4 && can_fact) pl.family = 4;
    else if (ctx->opt_kernel == 1) pl.family = 1;
    else if (ctx->opt_kernel == 2 && can_mma) pl.family = 2;
    else if (ctx->opt_kernel == 3 && can_umma) pl.family = 3;
    else return CKV_ERR_UNSUPPORTED;
    const int64_t C = pl.family == 4         ? (int64_t)INT32_MAX  // one CTA holds a whole history
                      : ctx->opt_split > 0 ? ctx->opt_split
                                           : auto_split_len(ctx, total_pos, pl.family, max_M);
    std::vector<Item> items;
    std::vector<int32_t> split;
    items.reserve((size_t)n);
    int64_t part_rows = 0;
    if (pl.family == 4) n_ranges = 1;  // its three launches work on all requests at once
    pl.n_ranges = n_ranges;
    for (int32_t k = 0, rg = 0; k <= n; ++k) {
        while (rg <= n_ranges && (n_ranges == 1 ? (rg == 0 ? 0 : n) : r_user[rg]) == k) {
            pl.r_user[rg] = k;
            pl.r_item[rg] = (int32_t)items.size();
            pl.r_split[rg] = (int32_t)split.size();
            ++rg;
        }
        if (k == n) break;
        Req& r = reqs[k];
        if (r.M <= 0) continue;
        const int64_t nc = r.L == 0 ? 1 : (r.L + C - 1) / C;
        r.n_chunks = (int32_t)nc;
        if (nc == 1) {
            items.push_back(Item{k, 0, r.L, -1});
            continue;
        }
        if (part_rows + nc * r.M > INT32_MAX) return CKV_ERR_UNSUPPORTED;
        r.part0 = (int32_t)part_rows;
        split.push_back(k);
        for (int64_t c = 0; c < nc; ++c) {
            const int32_t b = (int32_t)(c * C);
            items.push_back(Item{k, b, (int32_t)std::min<int64_t>(C, r.L - b), (int32_t)(part_rows + c * r.M)});
        }
        part_rows += nc * r.M;
    }
    // longest chunks first (inside every range): the tail of a grid is made of short ones
    std::vector<uint32_t> order(items.size()), tmp, count;
    for (int rg = 0; rg < n_ranges; ++rg)
        order_longest_first(items, (size_t)pl.r_item[rg], (size_t)pl.r_item[rg + 1], order, tmp, count);
    pl.n_items = (int32_t)items.size();
    pl.n_split = (int32_t)split.size();
    pl.split_items = 0;
    for (const Item& it : items) pl.split_items += it.part_row >= 0;
    pl.part_rows = part_rows;

    // the tables are laid out in the slot's pinned block and go to the device in one copy
    const size_t n_works = pl.family == 3 ? items.size() : 0;
    const size_t b_req = sizeof(Req) * reqs.size(), b_item = sizeof(Item) * items.size(),
                 b_split = sizeof(int32_t) * split.size(), b_work = sizeof(Work) * n_works;
    const size_t o_item = (b_req + 255) / 256 * 256, o_split = o_item + (b_item + 255) / 256 * 256,
                 o_work = o_split + (b_split + 255) / 256 * 256, total = o_work + b_work + 256;
    if (pl.uploaded) CK(cudaEventSynchronize(pl.uploaded));  // the block's previous upload has left the host
    else CK(cudaEventCreateWithFlags(&pl.uploaded, cudaEventDisableTiming));
    if (total > pl.host_cap) {
        ctx->st_allocs++;
        if (pl.host) cudaFreeHost(pl.host);
        pl.host = nullptr;
        pl.host_cap = 0;
        CK(cudaMallocHost(&pl.host, total + total / 4));
        pl.host_cap = total + total / 4;
    }
    CK(grow(pl.dev, total, &ctx->st_allocs));
    char* h = (char*)pl.host;
    std::memcpy(h, reqs.data(), b_req);
    Item* h_items = (Item*)(h + o_item);
    for (size_t i = 0; i < items.size(); ++i) h_items[i] = items[order[i]];
    if (b_split) std::memcpy(h + o_split, split.data(), b_split);
    Work* h_works = (Work*)(h + o_work);
    // where each request's blocks of 128 queries start in the table of largest visible lengths
    std::vector<int32_t> vb_off(n_works ? reqs.size() : 0);
    pl.n_vblocks = 0;
    for (size_t k = 0; k < vb_off.size(); ++k) {
        vb_off[k] = pl.n_vblocks;
        pl.n_vblocks += (reqs[k].M + 127) / 128;
    }
    for (size_t i = 0; i < n_works; ++i) {
        const Item& it = h_items[i];
        const Req& r = reqs[it.req];
        h_works[i] = Work{r.base, r.L, r.Lpad, r.q0, r.M, it.begin, it.len, it.part_row, {vb_off[it.req], 0, 0}};
    }
    pl.d_reqs = (Req*)pl.dev.p;
    pl.d_items = (Item*)((char*)pl.dev.p + o_item);
    pl.d_split = (int32_t*)((char*)pl.dev.p + o_split);
    pl.d_works = (Work*)((char*)pl.dev.p + o_work);
    CK(cudaMemcpyAsync(pl.dev.p, h, o_work + b_work, cudaMemcpyHostToDevice, s));
    CK(cudaEventRecord(pl.uploaded, s));
    pl.users.assign(users, users + n);
    pl.q_off.assign(q_off, q_off + n + 1);
    pl.generation = ctx->generation;
    pl.opt_split = ctx->opt_split;
    pl.opt_kernel = ctx->opt_kernel;
    pl.with_vis = with_vis;
    pl.live = true;
    return CKV_OK;
}

ckv_status get_plan(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off, bool with_vis,
                    int n_ranges, const int32_t* r_user, cudaStream_t s, Plan** out)
{
    ctx->tick++;
    Plan* victim = nullptr;
    for (auto& p : ctx->plans) {
        if (p.live && p.generation != ctx->generation) p.live = false;  // stale: the cache has changed since
        if (p.live && p.opt_split == ctx->opt_split && p.opt_kernel == ctx->opt_kernel && p.with_vis == with_vis &&
            (p.n_ranges == n_ranges || (p.family == 4 && p.n_ranges == 1)) && (int32_t)p.users.size() == n &&
            std::memcmp(p.users.data(), users, sizeof(int64_t) * (size_t)n) == 0 &&
            std::memcmp(p.q_off.data(), q_off, sizeof(int32_t) * ((size_t)n + 1)) == 0) {
            p.last_use = ctx->tick;
            ctx->st_hit = 1;
            *out = &p;
            return CKV_OK;
        }
        // the slot a new plan takes: a dead one, else the least recently used
        if (!victim || (!p.live && victim->live) || (p.live == victim->live && p.last_use < victim->last_use))
            victim = &p;
    }
    ctx->st_hit = 0;
    victim->live = false;
    ckv_status st;
    try {
        st = build_plan(ctx, *victim, n, users, q_off, with_vis, n_ranges, r_user, s);
    } catch (const std::bad_alloc&) {
        st = CKV_ERR_OOM;
    }
    if (st != CKV_OK) return st;
    victim->last_use = ctx->tick;
    *out = victim;
    return CKV_OK;
}

// ---- L2 residency of the pool ------------------------------------------------------------------------
// The pool is read by every work item of every decode call while the compressed caches stream through L2
// once.  The device's persisting-L2 carve-out is raised to the pool's size (a per-process setting that ends
// with the process; the previous value comes back when the last context on the device goes away), and each
// decode call puts an access-policy window over the pool on the caller's stream while it enqueues its
// kernels: pool lines are then kept in the carve-out and the streaming data cannot evict them.
std::mutex g_l2_mu;
int g_l2_users[64];
size_t g_l2_prev[64];

void l2_prepare(ckv_ctx* ctx)
{
    ctx->l2_window = 0;
    const int dev = ctx->cfg.device;
    if (dev >= 64) return;
    int max_persist = 0, max_window = 0;
    if (cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, dev) != cudaSuccess ||
        max_persist <= 0 || max_window <= 0) {
        cudaGetLastError();
        return;
    }
    const size_t pool_bytes = (size_t)ctx->n_pool_sides * ctx->pool_half;
    if (pool_bytes == 0) return;
    const size_t want = std::min(pool_bytes, (size_t)max_persist);
    std::lock_guard<std::mutex> lock(g_l2_mu);
    size_t cur = 0;
    if (cudaDeviceGetLimit(&cur, cudaLimitPersistingL2CacheSize) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    if (!ctx->l2_ready) {
        if (g_l2_users[dev]++ == 0) g_l2_prev[dev] = cur;
        ctx->l2_ready = true;
    }
    if (cur < want && cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    if (cur < want) cur = want;
    ctx->l2_window = std::min(pool_bytes, (size_t)max_window);
    ctx->l2_ratio = ctx->l2_window <= cur ? 1.0f : (float)((double)cur / (double)ctx->l2_window);
}

void l2_release(ckv_ctx* ctx)
{
    if (!ctx->l2_ready) return;
    const int dev = ctx->cfg.device;
    std::lock_guard<std::mutex> lock(g_l2_mu);
    if (--g_l2_users[dev] == 0) {
        cudaCtxResetPersistingL2Cache();
        cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, g_l2_prev[dev]);
        cudaGetLastError();
    }
    ctx->l2_ready = false;
}

// Puts the pool's window on a stream for the lifetime of the object and restores what the stream had.
struct L2Window {
    cudaStream_t s;
    cudaStreamAttrValue prev;
    bool on = false;
    L2Window(ckv_ctx* ctx, cudaStream_t stream) : s(stream)
    {
        ctx->st_l2 = 0;
        if (!ctx->opt_l2 || ctx->l2_window == 0) return;
        if (cudaStreamGetAttribute(s, cudaStreamAttributeAccessPolicyWindow, &prev) != cudaSuccess) {
            cudaGetLastError();
            return;
        }
        cudaStreamAttrValue v;
        std::memset(&v, 0, sizeof v);
        v.accessPolicyWindow.base_ptr = ctx->pool;
        v.accessPolicyWindow.num_bytes = ctx->l2_window;
        v.accessPolicyWindow.hitRatio = ctx->l2_ratio;
        v.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        v.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        if (cudaStreamSetAttribute(s, cudaStreamAttributeAccessPolicyWindow, &v) != cudaSuccess) {
            cudaGetLastError();
            return;
        }
        on = true;
        ctx->st_l2 = 1;
    }
    ~L2Window()
    {
        if (on && cudaStreamSetAttribute(s, cudaStreamAttributeAccessPolicyWindow, &prev) != cudaSuccess)
            cudaGetLastError();
    }
};

bool offsets_ok32(const int32_t* off, int32_t n)
{
    if (off[0] != 0) return false;
    for (int32_t k = 0; k < n; ++k)
        if (off[k + 1] < off[k]) return false;
    return true;
}

}  // namespace

extern "C" {

ckv_status ckv_create(const ckv_config* cfg, ckv_ctx** out)
{
    if (!cfg || !out) return CKV_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_groups < 1 || cfg->n_groups > 65535) return CKV_ERR_INVALID_ARG;
    if ((cfg->dtype != CKV_F32 && cfg->dtype != CKV_BF16) ||
        (cfg->out_dtype != CKV_F32 && cfg->out_dtype != CKV_BF16) ||
        (cfg->mode != CKV_SOFTMAX && cfg->mode != CKV_SILU_OVER_L) || cfg->device < 0)
        return CKV_ERR_INVALID_ARG;
    if (cfg->head_dim != 16 && cfg->head_dim != 32 && cfg->head_dim != 64 && cfg->head_dim != 128)
        return CKV_ERR_UNSUPPORTED;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device >= ndev) {
        cudaGetLastError();
        return CKV_ERR_CUDA;
    }
    ckv_ctx* ctx = new (std::nothrow) ckv_ctx();
    if (!ctx) return CKV_ERR_OOM;
    ctx->cfg = *cfg;
    ctx->elem = cfg->dtype == CKV_BF16 ? 2 : 4;
    ctx->scale = cfg->scale > 0.f ? cfg->scale
                                  : (cfg->mode == CKV_SOFTMAX ? 1.0f / std::sqrt((float)cfg->head_dim) : 1.0f);
    DeviceGuard dg(cfg->device);
    if (!dg.ok || cudaMalloc((void**)&ctx->d_flag, 2 * sizeof(int)) != cudaSuccess ||
        cudaMemset(ctx->d_flag, 0, 2 * sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return CKV_ERR_CUDA;
    }
    ctx->d_err = ctx->d_flag + 1;
    if (cudaDeviceGetAttribute(&ctx->n_sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || ctx->n_sms < 1) {
        cudaGetLastError();
        ctx->n_sms = 148;
    }
    *out = ctx;
    return CKV_OK;
}

ckv_status ckv_destroy(ckv_ctx* ctx)
{
    if (!ctx) return CKV_OK;
    DeviceGuard dg(ctx->cfg.device);
    drop_plans(ctx);
    void* bufs[] = {ctx->pool,    ctx->a_idxK,     ctx->a_idxV,      ctx->a_userK,   ctx->a_userV,
                    ctx->d_flag,  ctx->stage_q.p,  ctx->stage_out.p, ctx->partials.p, ctx->stage_vis.p, ctx->vmax.p};
    for (void* b : bufs)
        if (b) cudaFree(b);
    for (auto& e : ctx->ev)
        if (e) cudaEventDestroy(e);
    for (int r = 0; r < kMaxRanges; ++r) {
        if (ctx->pipe_stream[r]) cudaStreamDestroy(ctx->pipe_stream[r]);
        if (ctx->pipe_h2d[r]) cudaEventDestroy(ctx->pipe_h2d[r]);
        if (ctx->pipe_done[r]) cudaEventDestroy(ctx->pipe_done[r]);
    }
    if (ctx->pipe_start) cudaEventDestroy(ctx->pipe_start);
    if (ctx->pipe_plan) cudaEventDestroy(ctx->pipe_plan);
    l2_release(ctx);
    cudaGetLastError();
    delete ctx;
    return CKV_OK;
}

ckv_status ckv_pool_load_sides(ckv_ctx* ctx, const void* pool_K, const void* pool_V, int32_t n_entries,
                               int32_t d_shared_k, int32_t d_shared_v, void* stream)
{
    if (!ctx || n_entries < 1) return CKV_ERR_INVALID_ARG;
    const int D = ctx->cfg.head_dim, G = ctx->cfg.n_groups;
    if (d_shared_k < 0 || d_shared_k > D || d_shared_v < 0 || d_shared_v > D) return CKV_ERR_SHAPE;
    if (d_shared_k > 0 && d_shared_v > 0 && d_shared_k != d_shared_v) return CKV_ERR_SHAPE;
    const bool full_k = d_shared_k == 0, full_v = d_shared_v == 0;
    if ((!full_k && !pool_K) || (!full_v && !pool_V)) return CKV_ERR_INVALID_ARG;
    const int d_shared = std::max(d_shared_k, d_shared_v);  // of the shared side(s); 0: no side is shared
    if (!ctx->users.empty() && (n_entries != ctx->n_entries || d_shared != ctx->d_shared || full_k != ctx->full_k ||
                                full_v != ctx->full_v))
        return CKV_ERR_SHAPE;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t half = (size_t)G * n_entries * D * ctx->elem;
    const size_t src_bytes = (size_t)G * n_entries * d_shared * ctx->elem;
    const int n_sides = (full_k ? 0 : 1) + (full_v ? 0 : 1);
    Staged sk, sv;
    if (!full_k) CK(sk.init(pool_K, src_bytes, s));
    if (!full_v) CK(sv.init(pool_V, src_bytes, s));
    const bool layout_changes = ctx->n_entries != n_entries || ctx->d_shared != d_shared || ctx->full_k != full_k ||
                                ctx->full_v != full_v || !ctx->pool;
    if (layout_changes || half != ctx->pool_half) {
        void* np = nullptr;
        CK(cudaMalloc(&np, std::max<size_t>((size_t)n_sides * half, 256)));
        if (ctx->pool) cudaFree(ctx->pool);
        ctx->pool = np;
        ctx->pool_half = half;
    }
    void* dst_k = ctx->pool;
    void* dst_v = (char*)ctx->pool + (full_k ? 0 : half);
    const int du = D - d_shared;  // user-specific width of the shared side(s)
    ctx->has_mma = mma_supported(ctx->cfg.dtype, D, n_sides ? du : 0);
    ctx->has_tma = ctx->has_mma && n_sides == 2 &&
                   make_pool_tensor_maps(D, (int64_t)G * n_entries, dst_k, dst_v, ctx->tmaps);
    ctx->has_umma = umma_supported(ctx->cfg.dtype, D, n_sides ? du : 0, n_entries <= 65536 ? 2 : 4);
    if (!full_k) CK(launch_pool_layout(ctx->cfg.dtype, G, n_entries, d_shared, D, sk.dev, dst_k, s));
    if (!full_v) CK(launch_pool_layout(ctx->cfg.dtype, G, n_entries, d_shared, D, sv.dev, dst_v, s));
    if (sk.owned || sv.owned) CK(cudaStreamSynchronize(s));
    if (ctx->users.empty() && layout_changes) {
        // index width or the sides' widths may change: restart the (empty) arena
        void* old[4] = {ctx->a_idxK, ctx->a_idxV, ctx->a_userK, ctx->a_userV};
        for (void* b : old)
            if (b) cudaFree(b);
        ctx->a_idxK = ctx->a_idxV = ctx->a_userK = ctx->a_userV = nullptr;
        ctx->cap_units = ctx->used_units = 0;
        ctx->free_runs.clear();
    }
    ctx->n_entries = n_entries;
    ctx->d_shared = d_shared;
    ctx->d_user = D - d_shared;
    ctx->full_k = full_k;
    ctx->full_v = full_v;
    ctx->idx_bytes = n_entries <= 65536 ? 2 : 4;
    ctx->n_pool_sides = n_sides;
    l2_prepare(ctx);
    return CKV_OK;
}

ckv_status ckv_pool_load(ckv_ctx* ctx, const void* pool_K, const void* pool_V, int32_t n_entries,
                         int32_t d_shared, void* stream)
{
    if (!ctx || !pool_K || !pool_V || n_entries < 1) return CKV_ERR_INVALID_ARG;
    if (d_shared < 1 || d_shared > ctx->cfg.head_dim) return CKV_ERR_SHAPE;
    return ckv_pool_load_sides(ctx, pool_K, pool_V, n_entries, d_shared, d_shared, stream);
}

ckv_status ckv_cache_put_batch(ckv_ctx* ctx, int32_t n, const int64_t* users, const int64_t* hist_off,
                               const int32_t* idx_K, const int32_t* idx_V, const void* user_K,
                               const void* user_V, int32_t d_user, void* stream)
{
    if (!ctx || n < 0 || (n > 0 && (!users || !hist_off))) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    if (d_user != ctx->d_user) return CKV_ERR_SHAPE;
    if (n == 0) return CKV_OK;
    if (hist_off[0] != 0) return CKV_ERR_INVALID_ARG;
    const int G = ctx->cfg.n_groups;
    std::vector<int64_t> unit_off((size_t)n + 1);
    unit_off[0] = 0;
    for (int32_t k = 0; k < n; ++k) {
        const int64_t L = hist_off[k + 1] - hist_off[k];
        if (L < 0 || L > INT32_MAX - 32) return CKV_ERR_INVALID_ARG;
        unit_off[k + 1] = unit_off[k] + (int64_t)G * ((L + 31) / 32 * 32);
    }
    const int64_t P = hist_off[n], total_units = unit_off[n];
    int64_t eb[4];
    unit_bytes(ctx, eb);
    if (P > 0 && ((eb[0] && !idx_K) || (eb[1] && !idx_V) || (eb[2] && !user_K) || (eb[3] && !user_V)))
        return CKV_ERR_INVALID_ARG;

    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    try {
        ctx->users.reserve_more((size_t)n);
    } catch (const std::bad_alloc&) {
        return CKV_ERR_OOM;
    }
    int64_t base = 0;
    if (total_units > 0) {
        Staged sik, siv, suk, suv, sho, suo;
        const size_t ib = (size_t)P * G * sizeof(int32_t);
        if (eb[0]) CK(sik.init(idx_K, ib, s));
        if (eb[1]) {
            if (idx_V == idx_K && eb[0]) siv.dev = sik.dev; else CK(siv.init(idx_V, ib, s));
        }
        CK(suk.init(user_K, (size_t)P * G * eb[2], s));
        CK(suv.init(user_V, (size_t)P * G * eb[3], s));
        CK(sho.init(hist_off, sizeof(int64_t) * ((size_t)n + 1), s));
        CK(suo.init(unit_off.data(), sizeof(int64_t) * ((size_t)n + 1), s));
        ckv_status st = arena_take(ctx, total_units, s, &base);
        if (st != CKV_OK) return st;
        cudaError_t e = cudaMemsetAsync(ctx->d_flag, 0, sizeof(int), s);
        if (e == cudaSuccess)
            e = launch_pack(ctx->cfg.dtype, G, ctx->n_entries, ctx->idx_bytes, n, (const int64_t*)sho.dev,
                            (const int64_t*)suo.dev, total_units, base, (const int32_t*)sik.dev,
                            (const int32_t*)siv.dev, suk.dev, suv.dev, view_of(ctx), ctx->cfg.head_dim, ctx->d_flag, s);
        int bad = 0;
        if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess || bad) {  // nothing was stored: the units go back
            arena_give(ctx, base, total_units);
            return e != cudaSuccess ? ctx->fail(e) : CKV_ERR_INDEX_RANGE;
        }
    }
    for (int32_t k = 0; k < n; ++k) {
        const int64_t L = hist_off[k + 1] - hist_off[k];
        UserEntry* f = ctx->users.insert(users[k]);
        if (f->Lpad > 0) arena_give(ctx, f->base, (int64_t)G * f->Lpad);  // the entry this one replaces
        ctx->live_positions += L - f->L;
        *f = UserEntry{base + unit_off[k], (int32_t)L, (int32_t)((L + 31) / 32 * 32)};
    }
    ctx->generation++;
    return CKV_OK;
}

ckv_status ckv_cache_put(ckv_ctx* ctx, int64_t user, int32_t L, const int32_t* idx_K, const int32_t* idx_V,
                         const void* user_K, const void* user_V, int32_t d_user, void* stream)
{
    if (L < 0) return CKV_ERR_INVALID_ARG;
    const int64_t off[2] = {0, L};
    return ckv_cache_put_batch(ctx, 1, &user, off, idx_K, idx_V, user_K, user_V, d_user, stream);
}

ckv_status ckv_cache_append(ckv_ctx* ctx, int64_t user, int32_t L_new, const int32_t* idx_K, const int32_t* idx_V,
                            const void* user_K, const void* user_V, int32_t d_user, void* stream)
{
    if (!ctx || L_new < 0) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    if (d_user != ctx->d_user) return CKV_ERR_SHAPE;
    UserEntry* f = ctx->users.find(user);
    if (!f) return CKV_ERR_UNKNOWN_USER;
    if (L_new == 0) return CKV_OK;
    int64_t eb[4];
    unit_bytes(ctx, eb);
    if ((eb[0] && !idx_K) || (eb[1] && !idx_V) || (eb[2] && !user_K) || (eb[3] && !user_V)) return CKV_ERR_INVALID_ARG;
    const UserEntry old = *f;
    if ((int64_t)old.L + L_new > INT32_MAX - 32) return CKV_ERR_INVALID_ARG;
    const int G = ctx->cfg.n_groups;
    const int32_t L_tot = old.L + L_new, Lpad_tot = (L_tot + 31) / 32 * 32;
    const int64_t units = (int64_t)G * Lpad_tot;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    Staged sik, siv, suk, suv;
    const size_t ib = (size_t)L_new * G * sizeof(int32_t);
    if (eb[0]) CK(sik.init(idx_K, ib, s));
    if (eb[1]) {
        if (idx_V == idx_K && eb[0]) siv.dev = sik.dev; else CK(siv.init(idx_V, ib, s));
    }
    CK(suk.init(user_K, (size_t)L_new * G * eb[2], s));
    CK(suv.init(user_V, (size_t)L_new * G * eb[3], s));
    // the longer history is written to a run of its own (the old units are read while it is written) and the
    // old run is given back afterwards
    int64_t base = 0;
    ckv_status st = arena_take(ctx, units, s, &base);
    if (st != CKV_OK) return st;
    cudaError_t e = cudaMemsetAsync(ctx->d_flag, 0, sizeof(int), s);
    if (e == cudaSuccess)
        e = launch_append(ctx->cfg.dtype, G, ctx->n_entries, ctx->idx_bytes, old.base, old.L, old.Lpad, base,
                          L_new, Lpad_tot, (const int32_t*)sik.dev, (const int32_t*)siv.dev, suk.dev, suv.dev,
                          view_of(ctx), ctx->cfg.head_dim, ctx->d_flag, s);
    int bad = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess || bad) {  // the user keeps the old history
        arena_give(ctx, base, units);
        return e != cudaSuccess ? ctx->fail(e) : CKV_ERR_INDEX_RANGE;
    }
    arena_give(ctx, old.base, (int64_t)G * old.Lpad);
    *f = UserEntry{base, L_tot, Lpad_tot};
    ctx->live_positions += L_new;
    ctx->generation++;
    return CKV_OK;
}

namespace {

// Section offsets of a blob holding `total_units` units: K indices, V indices, user K, user V, end.
void blob_sections(const ckv_ctx* ctx, int64_t total_units, int64_t (&off)[5])
{
    int64_t eb[4];
    unit_bytes(ctx, eb);
    off[0] = 0;
    for (int i = 0; i < 4; ++i) off[i + 1] = (off[i] + total_units * eb[i] + 255) / 256 * 256;
}

int64_t units_of(const ckv_ctx* ctx, int64_t L) { return (int64_t)ctx->cfg.n_groups * ((L + 31) / 32 * 32); }

}  // namespace

ckv_status ckv_cache_blob_bytes(ckv_ctx* ctx, int32_t n, const int32_t* L, int64_t* bytes)
{
    if (!ctx || n < 0 || (n > 0 && !L) || !bytes) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    int64_t total = 0;
    for (int32_t k = 0; k < n; ++k) {
        if (L[k] < 0 || L[k] > INT32_MAX - 32) return CKV_ERR_INVALID_ARG;
        total += units_of(ctx, L[k]);
    }
    int64_t off[5];
    blob_sections(ctx, total, off);
    *bytes = off[4];
    return CKV_OK;
}

ckv_status ckv_cache_export(ckv_ctx* ctx, int32_t n, const int64_t* users, void* blob, int64_t bytes, void* stream)
{
    if (!ctx || n < 0 || (n > 0 && (!users || !blob))) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    int64_t total = 0;
    for (int32_t k = 0; k < n; ++k) {
        const UserEntry* f = ctx->users.find(users[k]);
        if (!f) return CKV_ERR_UNKNOWN_USER;
        total += units_of(ctx, f->L);
    }
    int64_t off[5];
    blob_sections(ctx, total, off);
    if (bytes != off[4]) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    int64_t eb[4];  // a section is empty where nothing is stored (no user part; no indices of a side that is not shared)
    unit_bytes(ctx, eb);
    const char* src[4] = {(const char*)ctx->a_idxK, (const char*)ctx->a_idxV, (const char*)ctx->a_userK,
                          (const char*)ctx->a_userV};
    int64_t done = 0;
    for (int32_t k = 0; k < n; ++k) {
        const UserEntry& e = *ctx->users.find(users[k]);
        const int64_t u = units_of(ctx, e.L);
        for (int i = 0; i < 4 && u > 0; ++i)
            if (eb[i] > 0)
                CK(cudaMemcpyAsync((char*)blob + off[i] + done * eb[i], src[i] + e.base * eb[i], (size_t)(u * eb[i]),
                               cudaMemcpyDefault, s));
        done += u;
    }
    return CKV_OK;
}

ckv_status ckv_cache_import(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* L, const void* blob,
                            int64_t bytes, void* stream)
{
    if (!ctx || n < 0 || (n > 0 && (!users || !L))) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    if (n == 0) return CKV_OK;
    std::vector<int64_t> unit_off((size_t)n + 1);
    unit_off[0] = 0;
    for (int32_t k = 0; k < n; ++k) {
        if (L[k] < 0 || L[k] > INT32_MAX - 32) return CKV_ERR_INVALID_ARG;
        unit_off[k + 1] = unit_off[k] + units_of(ctx, L[k]);
    }
    const int64_t total = unit_off[n];
    int64_t off[5];
    blob_sections(ctx, total, off);
    if (bytes != off[4] || (total > 0 && !blob)) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    try {
        ctx->users.reserve_more((size_t)n);
    } catch (const std::bad_alloc&) {
        return CKV_ERR_OOM;
    }
    int64_t base = 0;
    if (total > 0) {
        ckv_status st = arena_take(ctx, total, s, &base);
        if (st != CKV_OK) return st;
        int64_t eb[4];
        unit_bytes(ctx, eb);
        char* dst[4] = {(char*)ctx->a_idxK, (char*)ctx->a_idxV, (char*)ctx->a_userK, (char*)ctx->a_userV};
        // the batch takes one run of contiguous units: one copy per section
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < 4 && e == cudaSuccess; ++i)
            if (eb[i] > 0)
                e = cudaMemcpyAsync(dst[i] + base * eb[i], (const char*)blob + off[i], (size_t)(total * eb[i]),
                                    cudaMemcpyDefault, s);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_flag, 0, sizeof(int), s);
        if (e == cudaSuccess)
            e = launch_check_indices(ctx->idx_bytes, ctx->n_entries, eb[0] ? dst[0] + base * eb[0] : nullptr,
                                     eb[1] ? dst[1] + base * eb[1] : nullptr, total, ctx->d_flag, s);
        int bad = 0;
        if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess || bad) {  // nothing was stored: the units go back
            arena_give(ctx, base, total);
            return e != cudaSuccess ? ctx->fail(e) : CKV_ERR_INDEX_RANGE;
        }
    }
    const int G = ctx->cfg.n_groups;
    for (int32_t k = 0; k < n; ++k) {
        UserEntry* f = ctx->users.insert(users[k]);
        if (f->Lpad > 0) arena_give(ctx, f->base, (int64_t)G * f->Lpad);  // the entry this one replaces
        ctx->live_positions += L[k] - f->L;
        *f = UserEntry{base + unit_off[k], L[k], (L[k] + 31) / 32 * 32};
    }
    ctx->generation++;
    return CKV_OK;
}

ckv_status ckv_cache_evict(ckv_ctx* ctx, int64_t user)
{
    if (!ctx) return CKV_ERR_INVALID_ARG;
    const UserEntry* f = ctx->users.find(user);
    if (!f) return CKV_ERR_UNKNOWN_USER;
    ctx->live_positions -= f->L;
    arena_give(ctx, f->base, (int64_t)ctx->cfg.n_groups * f->Lpad);
    ctx->users.erase(user);
    ctx->generation++;
    return CKV_OK;
}

ckv_status ckv_cache_clear(ckv_ctx* ctx)
{
    if (!ctx) return CKV_ERR_INVALID_ARG;
    ctx->users.clear();
    ctx->free_runs.clear();
    ctx->live_positions = 0;
    ctx->used_units = 0;
    ctx->generation++;
    return CKV_OK;
}

namespace {

// The warp-level tensor-core kernel with the loader the options ask for.  The cp.async loader is the default:
// on B200 a warp spends about 100 clocks per TMA gather instruction it issues, so with the compute warps doing
// their own gathers the TMA loader measured slower (cfg4: 607 against 522 us; cfg5, Zipf indices that profit
// from L1, which TMA bypasses: 5.07 against 2.37 ms).  Both loaders give the same bits.
ckv_status run_mma(ckv_ctx* ctx, int D, int max_M, const AttendArgs& a, cudaStream_t s)
{
    const int loader = ctx->opt_loader == 2 ? 2 : 1;
    // the TMA loader serves the plain form only (both sides shared, no visible lengths)
    if (loader == 2 && (!ctx->has_tma || a.cv.full_k || a.cv.full_v || a.vis)) return CKV_ERR_UNSUPPORTED;
    ctx->st_loader = loader;
    CK(launch_attend_mma(D, max_M, a, loader == 2 ? ctx->tmaps : nullptr, ctx->d_err, s));
    return CKV_OK;
}

}  // namespace

}  // extern "C"

namespace {

constexpr size_t kPipeMinBytes = size_t(4) << 20;  // host query buffers below this are not worth pipelining
constexpr size_t kPipeManyBytes = size_t(96) << 20;  // from here on: eight ranges instead of four

cudaError_t pipe_prepare(ckv_ctx* ctx)
{
    if (ctx->pipe_ready) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    for (int r = 0; r < kMaxRanges && e == cudaSuccess; ++r) {
        if (!ctx->pipe_stream[r]) e = cudaStreamCreateWithFlags(&ctx->pipe_stream[r], cudaStreamNonBlocking);
        if (e == cudaSuccess && !ctx->pipe_h2d[r]) e = cudaEventCreateWithFlags(&ctx->pipe_h2d[r], cudaEventDisableTiming);
        if (e == cudaSuccess && !ctx->pipe_done[r]) e = cudaEventCreateWithFlags(&ctx->pipe_done[r], cudaEventDisableTiming);
    }
    if (e == cudaSuccess && !ctx->pipe_start) e = cudaEventCreateWithFlags(&ctx->pipe_start, cudaEventDisableTiming);
    if (e == cudaSuccess && !ctx->pipe_plan) e = cudaEventCreateWithFlags(&ctx->pipe_plan, cudaEventDisableTiming);
    ctx->pipe_ready = e == cudaSuccess;
    return e;
}

// The kernels of one slice of a plan (items [i0, i1), split requests [s0, s1)) on stream s.
ckv_status launch_slice(ckv_ctx* ctx, const Plan* pl, AttendArgs a, int i0, int i1, int s0, int s1, bool time_it,
                        cudaStream_t s)
{
    const int D = ctx->cfg.head_dim, G = ctx->cfg.n_groups;
    a.items = pl->d_items + i0;
    a.works = pl->d_works ? pl->d_works + i0 : nullptr;
    a.n_items = i1 - i0;
    L2Window l2(ctx, s);
    if (time_it) CK(cudaEventRecord(ctx->ev[0], s));
    if (a.n_items > 0) {
        if (pl->family == 4) {
            float* tw = (float*)ctx->partials.p;
            CK(launch_attend_fact(D, a, pl->n_req, pl->max_L, ctx->n_sms, tw,
                                  tw + (size_t)pl->n_req * G * fact_row_floats(ctx->n_entries), s));
            ctx->st_launches += 2;
        } else if (pl->family == 3)
            CK(launch_attend_umma(pl->max_M, a, ctx->n_sms, ctx->d_err, s));
        else if (pl->family == 2) {
            ckv_status st2 = run_mma(ctx, D, pl->max_M, a, s);
            if (st2 != CKV_OK) return st2;
        } else
            CK(launch_attend_simt(ctx->cfg.dtype, D, pl->max_M, a, s));
        ctx->st_launches++;
    }
    if (time_it) CK(cudaEventRecord(ctx->ev[1], s));
    if (s1 > s0) {
        CK(launch_combine(D, a, pl->d_split + s0, s1 - s0, s));
        ctx->st_launches++;
    }
    if (time_it) CK(cudaEventRecord(ctx->ev[2], s));
    return CKV_OK;
}

// ckv_attend (vis null) and ckv_attend_visible
ckv_status attend_impl(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off, const int32_t* vis,
                       const void* queries, void* out, void* stream)
{
    if (!ctx || n < 0 || (n > 0 && (!users || !q_off))) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    if (n == 0) return CKV_OK;
    if (!offsets_ok32(q_off, n)) return CKV_ERR_INVALID_ARG;
    const int64_t Q = q_off[n];
    if (Q > 0 && (!queries || !out)) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    ctx->st_launches = 0;
    ctx->st_allocs = 0;
    ctx->st_ranges = 1;
    const int D = ctx->cfg.head_dim, G = ctx->cfg.n_groups;
    const size_t q_row = (size_t)G * D * ctx->elem, o_row = (size_t)G * D * (ctx->cfg.out_dtype == CKV_BF16 ? 2 : 4);
    const size_t q_bytes = (size_t)Q * q_row, o_bytes = (size_t)Q * o_row;
    const bool q_host = Q > 0 && !is_device_ptr(queries), o_host = Q > 0 && !is_device_ptr(out);

    // Host buffers on both sides and enough of them: the request list is cut into ranges of consecutive users
    // with about equal numbers of query rows, and every range gets a stream of its own for its upload, its
    // kernels and its download.  The uploads are enqueued before the plan is looked up or built, so that host
    // work overlaps them too.
    int n_ranges = 1;
    int32_t r_user[kMaxRanges + 1];
    r_user[0] = 0;
    for (int r = 1; r <= kMaxRanges; ++r) r_user[r] = n;
    if (q_host && o_host && q_bytes >= kPipeMinBytes && n >= 8 && pipe_prepare(ctx) == cudaSuccess) {
        // four ranges; eight once a range is still tens of MB (the first upload and the last download, which
        // nothing overlaps, are then an eighth of the traffic instead of a quarter)
        n_ranges = (q_bytes >= kPipeManyBytes && n >= 2 * kMaxRanges) ? kMaxRanges : 4;
        int32_t k = 0;
        for (int r = 1; r < n_ranges; ++r) {
            const int64_t want = Q * r / n_ranges;
            while (k < n && q_off[k] < want) ++k;
            r_user[r] = k;
        }
        r_user[n_ranges] = n;
    }
    const void* d_q = queries;
    void* d_out = out;
    if (q_host) {
        CK(grow(ctx->stage_q, q_bytes, &ctx->st_allocs));
        d_q = ctx->stage_q.p;
    }
    if (o_host) {
        CK(grow(ctx->stage_out, o_bytes, &ctx->st_allocs));
        d_out = ctx->stage_out.p;
    }
    const int32_t* d_vis = vis;
    if (vis && Q > 0 && !is_device_ptr(vis)) {
        CK(grow(ctx->stage_vis, (size_t)Q * sizeof(int32_t), &ctx->st_allocs));
        CK(cudaMemcpyAsync(ctx->stage_vis.p, vis, (size_t)Q * sizeof(int32_t), cudaMemcpyHostToDevice, s));
        d_vis = (const int32_t*)ctx->stage_vis.p;
    }
    // The first range's upload (the first two for long request lists) goes out before the plan is looked up or built, so that
    // the host work overlaps it; the other ranges follow the plan's own (small) upload, which would otherwise
    // queue behind all of them on the copy engine and hold back the first kernels.
    auto upload_range = [&](int r) -> cudaError_t {
        cudaStream_t ps = ctx->pipe_stream[r];
        cudaError_t e = cudaStreamWaitEvent(ps, ctx->pipe_start, 0);
        const size_t r0 = (size_t)q_off[r_user[r]], r1 = (size_t)q_off[r_user[r + 1]];
        if (e == cudaSuccess && r1 > r0)
            e = cudaMemcpyAsync((char*)ctx->stage_q.p + r0 * q_row, (const char*)queries + r0 * q_row, (r1 - r0) * q_row,
                                cudaMemcpyHostToDevice, ps);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->pipe_h2d[r], ps);
        return e;
    };
    const int n_early = (n_ranges > 4 && n >= 8192) ? 2 : 1;  // planning thousands of users takes about as long as two uploads
    if (n_ranges > 1) {
        CK(cudaEventRecord(ctx->pipe_start, s));
        for (int r = 0; r < n_early; ++r) CK(upload_range(r));
    } else if (q_host) {
        CK(cudaMemcpyAsync(ctx->stage_q.p, queries, q_bytes, cudaMemcpyHostToDevice, s));
    }

    Plan* pl = nullptr;
    ckv_status st = get_plan(ctx, n, users, q_off, vis != nullptr, n_ranges, r_user, s, &pl);
    if (st != CKV_OK) {
        if (n_ranges > 1)  // the uploads already enqueued stay inside the call
            for (int r = 0; r < n_early; ++r) cudaStreamWaitEvent(s, ctx->pipe_h2d[r], 0);
        return st;
    }
    if (n_ranges > 1) {
        CK(cudaEventRecord(ctx->pipe_plan, s));
        for (int r = n_early; r < n_ranges; ++r) CK(upload_range(r));
    }
    ctx->st_items = pl->n_items;
    ctx->st_split = pl->split_items;
    ctx->st_kernel = pl->family;
    if (Q == 0) return CKV_OK;

    // split-reduction partials, or the factorisation's tables (per request and group: n_entries + a few floats)
    const size_t ws = pl->family == 4
                          ? (size_t)pl->n_req * G * ((size_t)fact_row_floats(ctx->n_entries) + fact_aux_floats()) * sizeof(float)
                          : (size_t)pl->part_rows * G * (D + 2) * sizeof(float);
    if (ws) CK(grow(ctx->partials, ws, &ctx->st_allocs));
    ctx->st_ws = (int64_t)ws;

    AttendArgs a;
    a.cv = view_of(ctx);
    a.reqs = pl->d_reqs;
    a.items = pl->d_items;
    a.works = pl->d_works;
    a.n_items = pl->n_items;
    a.queries = d_q;
    a.vis = d_vis;
    a.vmax = nullptr;
    a.out = d_out;
    a.partials = (float*)ctx->partials.p;
    a.out_dtype = ctx->cfg.out_dtype;
    a.mode = ctx->cfg.mode;
    a.scale = ctx->scale;
    a.arena_units = ctx->cap_units;
    a.q_rows = Q;
    a.part_rows = pl->family == 4 ? 0 : pl->part_rows;
    a.err = ctx->d_err;
    ctx->ev_valid = false;
    if (d_vis && pl->family == 3 && pl->n_items > 0) {
        // the tcgen05 kernel's roles skip what lies behind every row's limit: the largest limit per block of queries
        CK(grow(ctx->vmax, (size_t)std::max(pl->n_vblocks, 1) * sizeof(int32_t), &ctx->st_allocs));
        cudaStream_t vs = n_ranges > 1 ? ctx->pipe_stream[0] : s;
        if (n_ranges > 1) CK(cudaStreamWaitEvent(vs, ctx->pipe_plan, 0));
        CK(launch_vis_block_max(a, (int32_t*)ctx->vmax.p, vs));
        a.vmax = (const int32_t*)ctx->vmax.p;
        if (n_ranges > 1) {  // every range's kernels need the whole table
            CK(cudaEventRecord(ctx->pipe_plan, vs));
        }
    }

    if (n_ranges == 1) {
        const bool time_it = ctx->opt_time != 0;
        if (time_it)
            for (auto& e : ctx->ev)
                if (!e) CK(cudaEventCreate(&e));
        st = launch_slice(ctx, pl, a, 0, pl->n_items, 0, pl->n_split, time_it, s);
        if (st != CKV_OK) return st;
        ctx->ev_valid = time_it;
        if (o_host) CK(cudaMemcpyAsync(out, d_out, o_bytes, cudaMemcpyDeviceToHost, s));
        return CKV_OK;
    }

    // pipelined: the plan's tables (uploaded on the caller's stream if the plan is new) come first on every stream
    ctx->st_ranges = n_ranges;
    ckv_status result = CKV_OK;
    if (pl->n_ranges == 1) {
        // a plan that is not cut into ranges (pool-side factorisation): one pass on the first stream behind all uploads
        cudaStream_t ps = ctx->pipe_stream[0];
        CK(cudaStreamWaitEvent(ps, ctx->pipe_plan, 0));
        for (int r = 1; r < n_ranges; ++r) CK(cudaStreamWaitEvent(ps, ctx->pipe_h2d[r], 0));
        result = launch_slice(ctx, pl, a, 0, pl->n_items, 0, pl->n_split, false, ps);
        if (result == CKV_OK) {
            cudaError_t e = cudaMemcpyAsync(out, d_out, o_bytes, cudaMemcpyDeviceToHost, ps);
            if (e != cudaSuccess) result = ctx->fail(e);
        }
    } else {
        for (int r = 0; r < n_ranges && result == CKV_OK; ++r) {
            cudaStream_t ps = ctx->pipe_stream[r];
            CK(cudaStreamWaitEvent(ps, ctx->pipe_plan, 0));
            result = launch_slice(ctx, pl, a, pl->r_item[r], pl->r_item[r + 1], pl->r_split[r], pl->r_split[r + 1], false, ps);
            const size_t r0 = (size_t)q_off[r_user[r]], r1 = (size_t)q_off[r_user[r + 1]];
            if (result == CKV_OK && r1 > r0) {
                cudaError_t e = cudaMemcpyAsync((char*)out + r0 * o_row, (const char*)d_out + r0 * o_row, (r1 - r0) * o_row,
                                                cudaMemcpyDeviceToHost, ps);
                if (e != cudaSuccess) result = ctx->fail(e);
            }
        }
    }
    // whatever happened, the caller's stream continues behind everything that was enqueued on the internal ones
    for (int r = 0; r < n_ranges; ++r) {
        cudaEventRecord(ctx->pipe_done[r], ctx->pipe_stream[r]);
        cudaStreamWaitEvent(s, ctx->pipe_done[r], 0);
    }
    return result;
}

}  // namespace

extern "C" {

ckv_status ckv_attend(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off,
                      const void* queries, void* out, void* stream)
{
    return attend_impl(ctx, n, users, q_off, nullptr, queries, out, stream);
}

ckv_status ckv_attend_visible(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off, const int32_t* vis,
                              const void* queries, void* out, void* stream)
{
    if (n > 0 && q_off && q_off[n] > 0 && !vis) return CKV_ERR_INVALID_ARG;
    return attend_impl(ctx, n, users, q_off, vis, queries, out, stream);
}

ckv_status ckv_materialize(ckv_ctx* ctx, int64_t user, void* K_out, void* V_out, void* stream)
{
    if (!ctx || !K_out || !V_out) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    const UserEntry* f = ctx->users.find(user);
    if (!f) return CKV_ERR_UNKNOWN_USER;
    const UserEntry& e = *f;
    if (e.L == 0) return CKV_OK;
    DeviceGuard dg(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    const int D = ctx->cfg.head_dim;
    const size_t bytes = (size_t)e.L * ctx->cfg.n_groups * D * ctx->elem;
    const bool kh = !is_device_ptr(K_out), vh = !is_device_ptr(V_out);
    void *dk = K_out, *dv = V_out, *tk = nullptr, *tv = nullptr;
    if (kh) {
        CK(cudaMalloc(&tk, bytes));
        dk = tk;
    }
    if (vh) {
        cudaError_t er = cudaMalloc(&tv, bytes);
        if (er != cudaSuccess) {
            if (tk) cudaFree(tk);
            return ctx->fail(er);
        }
        dv = tv;
    }
    cudaError_t er = launch_materialize(ctx->cfg.dtype, D, view_of(ctx), e.base, e.L, e.Lpad, dk, dv, s);
    if (er == cudaSuccess && kh) er = cudaMemcpyAsync(K_out, dk, bytes, cudaMemcpyDeviceToHost, s);
    if (er == cudaSuccess && vh) er = cudaMemcpyAsync(V_out, dv, bytes, cudaMemcpyDeviceToHost, s);
    if (er == cudaSuccess && (kh || vh)) er = cudaStreamSynchronize(s);
    if (tk) cudaFree(tk);
    if (tv) cudaFree(tv);
    if (er != cudaSuccess) return ctx->fail(er);
    return CKV_OK;
}

ckv_status ckv_user_length(ckv_ctx* ctx, int64_t user, int64_t* L)
{
    if (!ctx || !L) return CKV_ERR_INVALID_ARG;
    const UserEntry* f = ctx->users.find(user);
    if (!f) return CKV_ERR_UNKNOWN_USER;
    *L = f->L;
    return CKV_OK;
}

ckv_status ckv_cache_bytes(ckv_ctx* ctx, int64_t* compressed, int64_t* full_width)
{
    if (!ctx || !compressed || !full_width) return CKV_ERR_INVALID_ARG;
    const int64_t pg = ctx->live_positions * ctx->cfg.n_groups;
    int64_t eb[4] = {0, 0, 0, 0};
    if (ctx->pool) unit_bytes(ctx, eb);
    *compressed = pg * (eb[0] + eb[1] + eb[2] + eb[3]);
    *full_width = pg * 2 * (int64_t)ctx->cfg.head_dim * ctx->elem;
    return CKV_OK;
}

namespace {

// one error word per device for the context-free tcgen05 router (allocated on first use, never freed)
int* route_err_word(int device)
{
    static std::mutex mu;
    static int* words[64] = {};
    std::lock_guard<std::mutex> lock(mu);
    if (device >= 64) return nullptr;
    if (!words[device]) {
        int* p = nullptr;
        if (cudaMalloc(&p, sizeof(int)) != cudaSuccess || cudaMemset(p, 0, sizeof(int)) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        words[device] = p;
    }
    return words[device];
}

}  // namespace

ckv_status ckv_route(int32_t device, int32_t n, int32_t n_groups, int32_t d_in, int32_t n_entries, const void* x,
                     const void* W, const float* bias, int32_t* idx_out, int32_t variant, void* stream)
{
    if (n < 0 || n_groups < 1 || n_entries < 1 || device < 0 || variant < 0 || variant > 2) return CKV_ERR_INVALID_ARG;
    if (!route_supported(d_in)) return CKV_ERR_UNSUPPORTED;
    if (n == 0) return CKV_OK;
    if (!x || !W || !idx_out) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(device);
    if (!dg.ok) return CKV_ERR_CUDA;
    if (!is_device_ptr(x) || !is_device_ptr(W) || !is_device_ptr(idx_out) || (bias && !is_device_ptr(bias)))
        return CKV_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (variant == 1) {
        e = launch_route(d_in, x, W, bias, n, n_entries, n_groups, idx_out, s);
    } else {
        int* word = route_err_word(device);
        if (!word) return CKV_ERR_OOM;
        e = launch_route_umma(d_in, x, W, bias, n, n_entries, n_groups, idx_out, word, s);
        int bad = 0;
        if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, word, sizeof(int), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e == cudaSuccess && bad) {  // a bounded wait inside the kernel ran out: the output is not valid
            cudaMemsetAsync(word, 0, sizeof(int), s);
            return CKV_ERR_CUDA;
        }
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CKV_ERR_CUDA;
    }
    return CKV_OK;
}

ckv_status ckv_project(int32_t device, int32_t n, int32_t n_groups, int32_t d_in, int32_t d_out, const void* x,
                       const void* W, const float* bias, void* out, void* stream)
{
    if (n < 0 || n_groups < 1 || device < 0) return CKV_ERR_INVALID_ARG;
    if (!project_supported(d_in, d_out, n_groups)) return CKV_ERR_UNSUPPORTED;
    if (n == 0) return CKV_OK;
    if (!x || !W || !out) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(device);
    if (!dg.ok) return CKV_ERR_CUDA;
    if (!is_device_ptr(x) || !is_device_ptr(W) || !is_device_ptr(out) || (bias && !is_device_ptr(bias)))
        return CKV_ERR_INVALID_ARG;
    const cudaError_t e = launch_project(d_in, d_out, n_groups, x, W, bias, n, out, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CKV_ERR_CUDA;
    }
    return CKV_OK;
}

ckv_status ckv_set_option(ckv_ctx* ctx, const char* name, int64_t value)
{
    if (!ctx || !name) return CKV_ERR_INVALID_ARG;
    if (!std::strcmp(name, "split_len")) {
        if (value < 0) return CKV_ERR_INVALID_ARG;
        ctx->opt_split = value == 0 ? 0 : (value + 63) / 64 * 64;
    } else if (!std::strcmp(name, "kernel")) {
        if (value < 0 || value > 4) return CKV_ERR_INVALID_ARG;
        ctx->opt_kernel = value;
    } else if (!std::strcmp(name, "mma_loader")) {
        if (value < 0 || value > 2) return CKV_ERR_INVALID_ARG;
        ctx->opt_loader = value;
    } else if (!std::strcmp(name, "l2_persist")) {
        ctx->opt_l2 = value != 0;
    } else if (!std::strcmp(name, "time_kernels")) {
        ctx->opt_time = value != 0;
    } else {
        return CKV_ERR_INVALID_ARG;
    }
    return CKV_OK;
}

ckv_status ckv_get_option(ckv_ctx* ctx, const char* name, int64_t* value)
{
    if (!ctx || !name || !value) return CKV_ERR_INVALID_ARG;
    if (!std::strcmp(name, "split_len")) *value = ctx->opt_split;
    else if (!std::strcmp(name, "kernel")) *value = ctx->opt_kernel;
    else if (!std::strcmp(name, "mma_loader")) *value = ctx->opt_loader;
    else if (!std::strcmp(name, "l2_persist")) *value = ctx->opt_l2;
    else if (!std::strcmp(name, "time_kernels")) *value = ctx->opt_time;
    else return CKV_ERR_INVALID_ARG;
    return CKV_OK;
}

ckv_status ckv_last_stat(ckv_ctx* ctx, const char* name, int64_t* value)
{
    if (!ctx || !name || !value) return CKV_ERR_INVALID_ARG;
    if (!std::strcmp(name, "launches")) *value = ctx->st_launches;
    else if (!std::strcmp(name, "work_items")) *value = ctx->st_items;
    else if (!std::strcmp(name, "split_items")) *value = ctx->st_split;
    else if (!std::strcmp(name, "kernel")) *value = ctx->st_kernel;
    else if (!std::strcmp(name, "mma_loader")) *value = ctx->st_loader;
    else if (!std::strcmp(name, "workspace_bytes")) *value = ctx->st_ws;
    else if (!std::strcmp(name, "plan_cache_hit")) *value = ctx->st_hit;
    else if (!std::strcmp(name, "alloc_calls")) *value = ctx->st_allocs;
    else if (!std::strcmp(name, "l2_window")) *value = ctx->st_l2;
    else if (!std::strcmp(name, "pipeline_ranges")) *value = ctx->st_ranges;
    else if (!std::strcmp(name, "arena_capacity_units")) *value = ctx->cap_units;
    else if (!std::strcmp(name, "arena_used_units")) *value = ctx->used_units;
    else if (!std::strcmp(name, "arena_free_runs")) *value = (int64_t)ctx->free_runs.size();
    else if (!std::strcmp(name, "device_errors")) {
        DeviceGuard dg(ctx->cfg.device);
        int v = 0;
        CK(cudaMemcpy(&v, ctx->d_err, sizeof(int), cudaMemcpyDeviceToHost));
        *value = v;
    }
    else if (!std::strcmp(name, "main_kernel_ns") || !std::strcmp(name, "combine_kernel_ns")) {
        if (!ctx->ev_valid) return CKV_ERR_STATE;
        DeviceGuard dg(ctx->cfg.device);
        const bool main = name[0] == 'm';
        float ms = 0.f;
        CK(cudaEventSynchronize(ctx->ev[2]));
        CK(cudaEventElapsedTime(&ms, ctx->ev[main ? 0 : 1], ctx->ev[main ? 1 : 2]));
        *value = (int64_t)(ms * 1e6);
    }
    else return CKV_ERR_INVALID_ARG;
    return CKV_OK;
}

const char* ckv_strerror(ckv_status s)
{
    switch (s) {
        case CKV_OK: return "ok";
        case CKV_ERR_INVALID_ARG: return "invalid argument";
        case CKV_ERR_SHAPE: return "shape mismatch";
        case CKV_ERR_STATE: return "no pool loaded";
        case CKV_ERR_INDEX_RANGE: return "pool index out of range";
        case CKV_ERR_UNKNOWN_USER: return "unknown user";
        case CKV_ERR_OOM: return "out of memory";
        case CKV_ERR_CUDA: return "CUDA error";
        case CKV_ERR_UNSUPPORTED: return "unsupported configuration";
        case CKV_ERR_TOO_LARGE: return "request exceeds the fixed capacity of this entry point";
    }
    return "unknown status";
}

const char* ckv_last_cuda_error(ckv_ctx* ctx) { return ctx ? ctx->cuda_err.c_str() : ""; }

int32_t ckv_version(void) { return 100; }

}  // extern "C"

// ------------------------------------------------------------------------------------------
// ckv_attend_static: the decode call for callers that must not allocate.
//
// Everything ckv_attend would put into freshly allocated or grown device memory -- the
// request/work-item tables and the partial results of the split-along-history reduction --
// lives in one fixed array in the library's device image instead.  The array exists once per
// GPU that loads the library and is shared by every call on that GPU.  The tables reach it as
// kernel arguments of a small kernel that writes them out, so no host buffer has to outlive the
// call and no copy from pageable memory is enqueued.
// ------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticBytes = size_t(8) << 20;  // CKV_STATIC_SCRATCH_BYTES
constexpr int kStaticMaxReqs = 256;                // CKV_STATIC_MAX_USERS
constexpr int kStaticMaxItems = 4096;
constexpr int kStaticMaxDevices = 64;
constexpr size_t kOffItems = sizeof(Req) * kStaticMaxReqs;
constexpr size_t kOffSplit = kOffItems + sizeof(Item) * kStaticMaxItems;
constexpr size_t kOffPartials = (kOffSplit + sizeof(int32_t) * kStaticMaxReqs + 255) / 256 * 256;

static __device__ __align__(256) unsigned char ckv_static_scratch[kStaticBytes];

// In host code `ckv_static_scratch` is only a handle for the runtime, not a device address.
// The address a kernel can use is looked up once per device, with that device current.
void* g_static_addr[kStaticMaxDevices];
std::mutex g_static_mu;

cudaError_t static_scratch_address(int device, void** out)
{
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, ckv_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_addr[device] = p;
    }
    *out = g_static_addr[device];
    return cudaSuccess;
}

// One launch carries the plan rows of up to kStaticChunk requests as its argument (under the 4 KB that
// kernel arguments may take) and thread t writes request t's row, its history chunks and its entry of
// the split list into the array.
constexpr int kStaticChunk = 80;
struct StaticRow {
    Req req;
    int32_t item0;       // first work item of the request (-1: no queries, no items)
    int32_t split_slot;  // position in the list of split requests, or -1
    int32_t chunk_len;   // positions per history chunk
};
struct StaticRows {
    int32_t first, count;
    StaticRow row[kStaticChunk];
};
static_assert(sizeof(StaticRows) <= 4000, "kernel arguments");

__global__ void static_plan_kernel(const StaticRows rows)
{
    const int t = threadIdx.x;
    if (t >= rows.count) return;
    const StaticRow& r = rows.row[t];
    const int k = rows.first + t;
    reinterpret_cast<Req*>(ckv_static_scratch)[k] = r.req;
    if (r.item0 < 0) return;
    Item* items = reinterpret_cast<Item*>(ckv_static_scratch + kOffItems) + r.item0;
    if (r.split_slot < 0) {
        items[0] = Item{k, 0, r.req.L, -1};
        return;
    }
    reinterpret_cast<int32_t*>(ckv_static_scratch + kOffSplit)[r.split_slot] = k;
    for (int c = 0; c < r.req.n_chunks; ++c) {
        const int b = c * r.chunk_len;
        items[c] = Item{k, b, min(r.chunk_len, r.req.L - b), r.req.part0 + c * r.req.M};
    }
}

}  // namespace

extern "C" ckv_status ckv_attend_static(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off,
                                        const void* queries, void* out, void* stream)
{
    if (!ctx || n < 0 || (n > 0 && (!users || !q_off))) return CKV_ERR_INVALID_ARG;
    if (!ctx->pool) return CKV_ERR_STATE;
    if (n == 0) return CKV_OK;
    if (n > kStaticMaxReqs) return CKV_ERR_TOO_LARGE;
    if (!offsets_ok32(q_off, n)) return CKV_ERR_INVALID_ARG;
    if (ctx->cfg.device >= kStaticMaxDevices) return CKV_ERR_UNSUPPORTED;
    const int64_t Q = q_off[n];
    if (Q == 0) return CKV_OK;
    if (!queries || !out) return CKV_ERR_INVALID_ARG;
    DeviceGuard dg(ctx->cfg.device);
    if (!is_device_ptr(queries) || !is_device_ptr(out)) return CKV_ERR_INVALID_ARG;  // staging would allocate
    cudaStream_t s = (cudaStream_t)stream;
    void* scratch = nullptr;
    CK(static_scratch_address(ctx->cfg.device, &scratch));

    // the plan, in fixed-size host arrays; nothing is enqueued before the request is known to fit
    StaticRow rows[kStaticMaxReqs];
    const int D = ctx->cfg.head_dim, G = ctx->cfg.n_groups;
    int64_t total_pos = 0;
    int32_t max_M = 0;
    for (int32_t k = 0; k < n; ++k) {
        const UserEntry* f = ctx->users.find(users[k]);
        if (!f) return CKV_ERR_UNKNOWN_USER;
        Req& r = rows[k].req;
        r.base = f->base;
        r.L = f->L;
        r.Lpad = f->Lpad;
        r.q0 = q_off[k];
        r.M = q_off[k + 1] - q_off[k];
        r.part0 = -1;
        r.n_chunks = 1;
        if (r.M > 0) total_pos += r.L;
        max_M = std::max(max_M, r.M);
    }
    int family;
    if (ctx->opt_kernel == 0) family = ctx->has_mma ? 2 : 1;
    else if (ctx->opt_kernel == 1) family = 1;
    else if (ctx->opt_kernel == 2 && ctx->has_mma) family = 2;
    else return CKV_ERR_UNSUPPORTED;
    const int64_t C = ctx->opt_split > 0 ? ctx->opt_split : auto_split_len(ctx, total_pos, family, max_M);
    const int64_t row_floats = (int64_t)G * (D + 2);
    const int64_t cap_rows = (int64_t)((kStaticBytes - kOffPartials) / sizeof(float)) / row_floats;
    int32_t n_items = 0, n_split = 0;
    int64_t part_rows = 0;
    for (int32_t k = 0; k < n; ++k) {
        StaticRow& row = rows[k];
        Req& r = row.req;
        row.item0 = row.split_slot = -1;
        row.chunk_len = (int32_t)std::min<int64_t>(C, INT32_MAX);
        if (r.M <= 0) continue;
        const int64_t nc = r.L == 0 ? 1 : (r.L + C - 1) / C;
        if (n_items + nc > kStaticMaxItems) return CKV_ERR_TOO_LARGE;
        r.n_chunks = (int32_t)nc;
        row.item0 = n_items;
        n_items += (int32_t)nc;
        if (nc == 1) continue;
        if (part_rows + nc * r.M > cap_rows) return CKV_ERR_TOO_LARGE;
        r.part0 = (int32_t)part_rows;
        row.split_slot = n_split++;
        part_rows += nc * r.M;
    }

    for (int32_t k0 = 0; k0 < n; k0 += kStaticChunk) {
        StaticRows arg;
        arg.first = k0;
        arg.count = std::min<int32_t>(kStaticChunk, n - k0);
        std::memcpy(arg.row, rows + k0, sizeof(StaticRow) * (size_t)arg.count);
        static_plan_kernel<<<1, kStaticChunk, 0, s>>>(arg);
        CK(cudaGetLastError());
    }

    char* base = (char*)scratch;
    AttendArgs a;
    a.cv = view_of(ctx);
    a.reqs = (const Req*)base;
    a.items = (const Item*)(base + kOffItems);
    a.works = nullptr;
    a.n_items = n_items;
    a.queries = queries;
    a.vis = nullptr;
    a.vmax = nullptr;
    a.out = out;
    a.partials = (float*)(base + kOffPartials);  // every entry that is read was written by this call
    a.out_dtype = ctx->cfg.out_dtype;
    a.mode = ctx->cfg.mode;
    a.scale = ctx->scale;
    a.arena_units = ctx->cap_units;
    a.q_rows = Q;
    a.part_rows = part_rows;
    a.err = ctx->d_err;
    if (n_items > 0) {
        if (family == 2)
            CK(launch_attend_mma(D, max_M, a, nullptr, ctx->d_err, s));
        else
            CK(launch_attend_simt(ctx->cfg.dtype, D, max_M, a, s));
    }
    if (n_split > 0) CK(launch_combine(D, a, (const int32_t*)(base + kOffSplit), n_split, s));
    return CKV_OK;
}
