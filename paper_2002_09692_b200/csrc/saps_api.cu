// C ABI of libsaps: context, argument validation, error codes, the round scheduler
// (Algorithm 1's loop) and the host-buffer entry point.  No device arithmetic lives here.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/saps.h"
#include "internal.h"

using namespace saps;

struct saps_ctx {
    int n;
    uint64_t N;
    uint64_t ld;
    uint64_t seed;
    uint32_t ntiles;
    uint64_t col_offset;    // global index of column 0 when this context holds a column shard
    cudaEvent_t ev_before, ev_after;  // optional: recorded around the round kernel
    int gossip_first;       // update order: 0 Algorithm 2, 1 Eq. 7
    int staging;            // SAPS_STAGING_*
    int staging_give_up;    // test hook of the staged form's bounded wait
    uint32_t spin_limit;    // poll budget of the look-back
    uint32_t skip_tile;     // test hook, 0xFFFFFFFF = off
    double* partials;       // device, for the consensus distance: one double per block of columns
    uint64_t cap_override;  // 0 = capacity from the binomial bound
    // device scratch, allocated on first use on the then-current device
    void* scratch;
    int scratch_device;
    // pipeline of the host-buffer entry point, created on first use: kMaxLanes streams that
    // copy a column chunk in and run the round on it, one stream that copies results out
    static constexpr int kMaxLanes = 6;
    cudaStream_t lane_stream[kMaxLanes];
    cudaEvent_t lane_event[kMaxLanes];
    cudaStream_t out_stream;
    cudaEvent_t scan_event;
    bool lanes_ready;
    int host_lanes;             // lanes in use
    uint32_t host_chunk_tiles;  // column tiles per chunk
    // Mask counts of the emitting round (saps_round_pack): kept columns per tile, and per group
    // of 2^group_shift tiles, for the current round and, counted ahead by the fused kernel
    // itself, for the next one.  The group sums rotate over three buffers: read this round,
    // accumulated for the next round, cleared for the round after.
    uint32_t* emit_mem;        // device: cnt[2][ntiles], group_cnt[3][ngroups]
    uint32_t group_shift, ngroups;
    int emit_cur;              // which cnt buffer the next call looks at
    int group_cur;             // which group_cnt buffer the next call looks at
    bool ahead_valid;          // cnt[emit_cur] holds the counts of round ahead_t ...
    uint64_t ahead_t, ahead_thr;
    uint32_t ahead_col_offset; // ... for this threshold and column offset
    int run_ahead;             // 1 = let the fused kernel count the next round's mask (default)
    SelectState select;
};

namespace {

bool valid_frac(double p) { return p >= 0.0 && p <= 1.0; }  // false for NaN

uint64_t threshold64(double keep_frac)
{
    double s = std::floor(keep_frac * 4294967296.0);
    if (!(s > 0.0)) return 0;
    if (s >= 4294967296.0) return 1ull << 32;
    return (uint64_t)s;
}

RoundKey make_key(uint64_t seed, uint64_t t, double keep_frac)
{
    RoundKey key;
    uint32_t k0 = 0, k1 = 0;
    saps_round_key(seed, t, &k0, &k1);
    key.k0f = fold16(k0);
    key.k1f = fold16(k1);
    const uint64_t thr = threshold64(keep_frac);
    key.all = thr >= (1ull << 32) ? 1u : 0u;
    key.thr32 = key.all ? 0xFFFFFFFFu : (uint32_t)thr;
    return key;
}

int check_pairs(int n, const int32_t* pairs)
{
    if (pairs == nullptr) return SAPS_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        const int32_t j = pairs[i];
        if (j < 0 || j >= n || pairs[j] != i) return SAPS_ERR_PAIRS;
    }
    return SAPS_OK;
}

// Row groups of a round.  A worker without a peer needs a pass only when there is an SGD
// step to apply or a wire buffer to emit.
RowGroups make_groups(int n, const int32_t* pairs, bool singles)
{
    RowGroups rg;
    rg.count = 0;
    for (int i = 0; i < n; ++i) {
        const int j = pairs[i];
        if (j > i) {
            rg.a[rg.count] = (uint8_t)i;
            rg.b[rg.count] = (uint8_t)j;
            ++rg.count;
        } else if (j == i && singles) {
            rg.a[rg.count] = (uint8_t)i;
            rg.b[rg.count] = kNoPeer;
            ++rg.count;
        }
    }
    return rg;
}

// The scratch is cleared on the stream of the call that creates it, so that the clear is
// ordered before that call's kernels whatever kind of stream it is.
int ensure_scratch(saps_ctx* ctx, cudaStream_t stream)
{
    if (ctx->scratch != nullptr) return SAPS_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    void* p = nullptr;
    const size_t bytes = scratch_bytes(ctx->ntiles);
    if (cudaMalloc(&p, bytes) != cudaSuccess) {
        cudaGetLastError();
        return SAPS_ERR_NOMEM;
    }
    if (cudaMemsetAsync(p, 0, bytes, stream) != cudaSuccess) {
        cudaFree(p);
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    ctx->scratch = p;
    ctx->scratch_device = dev;
    return SAPS_OK;
}

int check_round_args(const saps_ctx* ctx, const float* x, const float* g, float lr, uint64_t t,
                     double keep_frac)
{
    if (ctx == nullptr || x == nullptr || t == 0 || !valid_frac(keep_frac)) return SAPS_ERR_INVALID;
    if (g == nullptr && lr != 0.0f) return SAPS_ERR_INVALID;
    if (lr != lr) return SAPS_ERR_INVALID;
    return SAPS_OK;
}

RoundArgs round_args(const saps_ctx* ctx, float* x, const float* g, float lr, const RowGroups& rg,
                     const RoundKey& key, uint64_t ld = 0)
{
    RoundArgs a;
    a.x = x;
    a.g = g;
    a.ld = (size_t)(ld ? ld : ctx->ld);
    a.N = (uint32_t)ctx->N;
    a.lr = lr;
    a.groups = rg;
    a.key = key;
    a.col_offset = (uint32_t)ctx->col_offset;
    a.tile_begin = 0;
    a.tile_count = ctx->ntiles;
    a.gossip_first = ctx->gossip_first;
    a.staging = ctx->staging;
    a.staging_give_up = ctx->staging_give_up;
    // a round without gradient rewrites only the vectors that hold a kept column, unless the mask
    // is so dense (more than one column in 25) that a full coalesced write stream is cheaper
    a.store_all = key.all || key.thr32 > 0x0A3D70A3u;
    a.store_sectors = reinterpret_cast<uintptr_t>(x) % 32 == 0 && (a.ld * sizeof(float)) % 32 == 0;
    a.out_vals = nullptr;
    a.out_rows = nullptr;
    a.cap = 0;
    a.tile_cnt = nullptr;
    a.group_cnt = nullptr;
    a.group_shift = ctx->group_shift;
    a.ngroups = ctx->ngroups;
    a.out_idx = nullptr;
    a.out_count = nullptr;
    a.status = static_cast<int*>(ctx->scratch);   // NULL until a call of this context created the scratch
    a.next_cnt = nullptr;
    a.next_group_cnt = nullptr;
    a.clear_group_cnt = nullptr;
    a.next_key = key;
    return a;
}

// Launch of the round kernel, bracketed by the caller's timing events when they are set.
int timed_round(const saps_ctx* ctx, const RoundArgs& a, bool emit, cudaStream_t stream)
{
    if (ctx->ev_before != nullptr && cudaEventRecord(ctx->ev_before, stream) != cudaSuccess) return SAPS_ERR_CUDA;
    if (launch_round(a, emit, stream) != cudaSuccess) return SAPS_ERR_CUDA;
    if (ctx->ev_after != nullptr && cudaEventRecord(ctx->ev_after, stream) != cudaSuccess) return SAPS_ERR_CUDA;
    return SAPS_OK;
}

uint64_t capacity_for(uint64_t N, double keep_frac)
{
    const double p = (double)threshold64(keep_frac) / 4294967296.0;
    const double mean = (double)N * p;
    const double sd = std::sqrt((double)N * p * (1.0 - p));
    uint64_t c = (uint64_t)std::ceil(mean + 8.0 * sd) + 64;
    c = (c + 31) / 32 * 32;
    return c < N ? c : N;
}

}  // namespace

extern "C" {

int saps_create_ld(int n, uint64_t N, uint64_t ld, uint64_t seed, saps_ctx** out)
{
    if (out == nullptr) return SAPS_ERR_INVALID;
    *out = nullptr;
    if (n < 1 || n > (int)kMaxWorkers || N < 1 || N > 0xFFFFFFFFull || ld < N) return SAPS_ERR_INVALID;
    saps_ctx* ctx = new (std::nothrow) saps_ctx();
    if (ctx == nullptr) return SAPS_ERR_NOMEM;
    ctx->n = n;
    ctx->N = N;
    ctx->ld = ld;
    ctx->seed = seed;
    ctx->ntiles = (uint32_t)((N + kTileCols - 1) / kTileCols);
    ctx->cap_override = 0;
    ctx->gossip_first = 0;
    ctx->staging = SAPS_STAGING_AUTO;
    ctx->staging_give_up = 0;
    ctx->spin_limit = kSpinLimit;
    ctx->skip_tile = 0xFFFFFFFFu;
    ctx->partials = nullptr;
    ctx->ev_before = nullptr;
    ctx->ev_after = nullptr;
    ctx->col_offset = 0;
    ctx->scratch = nullptr;
    ctx->scratch_device = -1;
    ctx->lanes_ready = false;
    ctx->host_lanes = 3;
    ctx->host_chunk_tiles = 512;
    ctx->emit_mem = nullptr;
    ctx->emit_cur = 0;
    ctx->group_cur = 0;
    // groups of about sqrt(ntiles) tiles: a block then adds up at most about 2 sqrt(ntiles) numbers
    ctx->group_shift = 0;
    while ((1ull << (2 * ctx->group_shift)) < ctx->ntiles) ++ctx->group_shift;
    ctx->ngroups = (ctx->ntiles + (1u << ctx->group_shift) - 1) >> ctx->group_shift;
    ctx->ahead_valid = false;
    ctx->ahead_t = ctx->ahead_thr = 0;
    ctx->ahead_col_offset = 0;
    ctx->run_ahead = 1;
    ctx->select.n = n;
    ctx->select.seed = seed;
    try {
        ctx->select.R.assign((size_t)n * n, kNever);
    } catch (...) {
        delete ctx;
        return SAPS_ERR_NOMEM;
    }
    *out = ctx;
    return SAPS_OK;
}

int saps_create(int n, uint64_t N, uint64_t seed, saps_ctx** out)
{
    return saps_create_ld(n, N, N, seed, out);
}

int saps_destroy(saps_ctx* ctx)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    if (ctx->lanes_ready) {
        for (int l = 0; l < saps_ctx::kMaxLanes; ++l) {
            cudaStreamDestroy(ctx->lane_stream[l]);
            cudaEventDestroy(ctx->lane_event[l]);
        }
        cudaStreamDestroy(ctx->out_stream);
        cudaEventDestroy(ctx->scan_event);
    }
    if (ctx->scratch != nullptr) cudaFree(ctx->scratch);
    if (ctx->partials != nullptr) cudaFree(ctx->partials);
    if (ctx->emit_mem != nullptr) cudaFree(ctx->emit_mem);
    delete ctx;
    return SAPS_OK;
}

void saps_round_key(uint64_t seed, uint64_t t, uint32_t* k0, uint32_t* k1)
{
    uint32_t a = mix32((uint32_t)(seed & 0xFFFFFFFFull) ^ kSeedPad);
    a = mix32(a ^ (uint32_t)(seed >> 32));
    a = mix32(a ^ (uint32_t)(t & 0xFFFFFFFFull));
    a = mix32(a ^ (uint32_t)(t >> 32));
    if (k0) *k0 = a;
    if (k1) *k1 = mix32(a ^ kKeyPad);
}

uint64_t saps_threshold(double keep_frac) { return threshold64(keep_frac); }

int saps_mask(saps_ctx* ctx, uint64_t t, double keep_frac, uint32_t* out_bits, void* stream)
{
    if (ctx == nullptr || out_bits == nullptr || t == 0 || !valid_frac(keep_frac)) return SAPS_ERR_INVALID;
    const RoundKey key = make_key(ctx->seed, t, keep_frac);
    return launch_mask((uint32_t)ctx->N, (uint32_t)ctx->col_offset, key, out_bits, (cudaStream_t)stream) == cudaSuccess ? SAPS_OK
                                                                                              : SAPS_ERR_CUDA;
}

int saps_round(saps_ctx* ctx, float* x, const float* g, float lr, const int32_t* pairs, uint64_t t,
               double keep_frac, void* stream)
{
    int rc = check_round_args(ctx, x, g, lr, t, keep_frac);
    if (rc != SAPS_OK) return rc;
    rc = check_pairs(ctx->n, pairs);
    if (rc != SAPS_OK) return rc;
    const RowGroups rg = make_groups(ctx->n, pairs, g != nullptr);
    const RoundArgs a = round_args(ctx, x, g, lr, rg, make_key(ctx->seed, t, keep_frac));
    return timed_round(ctx, a, false, (cudaStream_t)stream);
}

uint64_t saps_pack_capacity(const saps_ctx* ctx, double keep_frac)
{
    if (ctx == nullptr || !valid_frac(keep_frac)) return 0;
    if (ctx->cap_override != 0) return ctx->cap_override < ctx->N ? ctx->cap_override : ctx->N;
    return capacity_for(ctx->N, keep_frac);
}

int saps_set_column_offset(saps_ctx* ctx, uint64_t col_offset)
{
    if (ctx == nullptr || col_offset + ctx->N > (1ull << 32)) return SAPS_ERR_INVALID;
    ctx->col_offset = col_offset;
    return SAPS_OK;
}

int saps_set_staging(saps_ctx* ctx, int staging)
{
    if (ctx == nullptr || staging < SAPS_STAGING_AUTO || staging > SAPS_STAGING_BULK) return SAPS_ERR_INVALID;
    ctx->staging = staging;
    return SAPS_OK;
}

int saps_set_update_order(saps_ctx* ctx, int order)
{
    if (ctx == nullptr || (order != SAPS_ORDER_SGD_FIRST && order != SAPS_ORDER_GOSSIP_FIRST)) return SAPS_ERR_INVALID;
    ctx->gossip_first = order == SAPS_ORDER_GOSSIP_FIRST;
    return SAPS_OK;
}

namespace {

int unpack_avg_impl(saps_ctx* ctx, float* x, const float* recv_vals, const uint32_t* idx, const uint32_t* count,
                    double keep_frac, const uint8_t* src, cudaStream_t stream)
{
    UnpackArgs a;
    std::memcpy(a.src, src, kMaxWorkers);
    a.x = x;
    a.ld = (size_t)ctx->ld;
    a.n = ctx->n;
    a.recv = recv_vals;
    a.cap = (uint32_t)saps_pack_capacity(ctx, keep_frac);
    a.idx = idx;
    a.count = count;
    a.col_offset = (uint32_t)ctx->col_offset;
    a.N = (uint32_t)ctx->N;
    return launch_unpack_avg(a, stream) == cudaSuccess ? SAPS_OK : SAPS_ERR_CUDA;
}

}  // namespace

int saps_unpack_avg(saps_ctx* ctx, float* x, const float* recv_vals, const uint32_t* idx, const uint32_t* count,
                    double keep_frac, const int32_t* pairs, void* stream)
{
    if (ctx == nullptr || x == nullptr || recv_vals == nullptr || idx == nullptr || count == nullptr ||
        !valid_frac(keep_frac))
        return SAPS_ERR_INVALID;
    if (pairs != nullptr) {
        const int rc = check_pairs(ctx->n, pairs);
        if (rc != SAPS_OK) return rc;
    }
    uint8_t src[kMaxWorkers] = {};
    for (int i = 0; i < ctx->n; ++i)
        src[i] = pairs == nullptr ? (uint8_t)i : (pairs[i] == i ? kNoPeer : (uint8_t)pairs[i]);
    return unpack_avg_impl(ctx, x, recv_vals, idx, count, keep_frac, src, (cudaStream_t)stream);
}

int saps_unpack_avg_rows(saps_ctx* ctx, float* x, const float* recv_vals, const uint32_t* idx,
                         const uint32_t* count, double keep_frac, const int32_t* src_rows, void* stream)
{
    if (ctx == nullptr || x == nullptr || recv_vals == nullptr || idx == nullptr || count == nullptr ||
        src_rows == nullptr || !valid_frac(keep_frac))
        return SAPS_ERR_INVALID;
    uint8_t src[kMaxWorkers] = {};
    for (int i = 0; i < ctx->n; ++i) {
        if (src_rows[i] < -1 || src_rows[i] >= ctx->n) return SAPS_ERR_INVALID;
        src[i] = src_rows[i] < 0 ? kNoPeer : (uint8_t)src_rows[i];
    }
    return unpack_avg_impl(ctx, x, recv_vals, idx, count, keep_frac, src, (cudaStream_t)stream);
}

int saps_consensus_distance(saps_ctx* ctx, const float* x, double* out, void* stream)
{
    if (ctx == nullptr || x == nullptr || out == nullptr) return SAPS_ERR_INVALID;
    if (ctx->partials == nullptr) {
        void* p = nullptr;
        if (cudaMalloc(&p, (size_t)consensus_blocks((uint32_t)ctx->N) * sizeof(double)) != cudaSuccess) {
            cudaGetLastError();
            return SAPS_ERR_NOMEM;
        }
        ctx->partials = static_cast<double*>(p);
    }
    return launch_consensus(x, (size_t)ctx->ld, (uint32_t)ctx->N, ctx->n, ctx->partials, out,
                            (cudaStream_t)stream) == cudaSuccess
               ? SAPS_OK
               : SAPS_ERR_CUDA;
}

int saps_comm_stats(const saps_ctx* ctx, const double* bandwidth, const int32_t* pairs, uint64_t count,
                    double bits_per_s_per_unit, double* out5)
{
    if (ctx == nullptr || bandwidth == nullptr || out5 == nullptr || !(bits_per_s_per_unit > 0.0)) return SAPS_ERR_INVALID;
    const int n = ctx->n;
    const int rc = check_pairs(n, pairs);
    if (rc != SAPS_OK) return rc;
    double lo = 0.0, sum = 0.0;
    int links = 0;
    for (int i = 0; i < n; ++i) {
        const int j = pairs[i];
        if (j <= i) continue;
        const double a = bandwidth[(size_t)i * n + j], b = bandwidth[(size_t)j * n + i];
        const double bw = a < b ? a : b;
        if (links == 0 || bw < lo) lo = bw;
        sum += bw;
        ++links;
    }
    out5[0] = 2.0 * (double)count;                       // values sent + received per matched worker
    out5[1] = 8.0 * (double)count;                       // the same in bytes (fp32)
    out5[2] = links ? lo : 0.0;                          // bottleneck bandwidth of the round
    out5[3] = links ? sum / links : 0.0;                 // mean bandwidth of the chosen links
    out5[4] = (links && lo > 0.0) ? 32.0 * (double)count / (lo * bits_per_s_per_unit) : 0.0;  // seconds
    return SAPS_OK;
}

int saps_debug_inject(saps_ctx* ctx, uint32_t skip_tile, uint32_t spin_limit)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    ctx->skip_tile = skip_tile;
    ctx->spin_limit = spin_limit == 0 ? kSpinLimit : spin_limit;
    return SAPS_OK;
}

int saps_debug_staging_wait(saps_ctx* ctx, int give_up)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    ctx->staging_give_up = give_up != 0;
    return SAPS_OK;
}

int saps_set_timing_events(saps_ctx* ctx, void* before, void* after)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    ctx->ev_before = (cudaEvent_t)before;
    ctx->ev_after = (cudaEvent_t)after;
    return SAPS_OK;
}

int saps_set_pack_capacity(saps_ctx* ctx, uint64_t cap)
{
    if (ctx == nullptr || cap > 0xFFFFFFFFull) return SAPS_ERR_INVALID;
    ctx->cap_override = cap;
    return SAPS_OK;
}

int saps_pack(saps_ctx* ctx, const float* x, uint64_t t, double keep_frac, float* out_vals,
              uint32_t* out_idx, uint32_t* out_count, void* stream)
{
    if (ctx == nullptr || x == nullptr || out_vals == nullptr || out_count == nullptr || t == 0 ||
        !valid_frac(keep_frac))
        return SAPS_ERR_INVALID;
    int rc = ensure_scratch(ctx, (cudaStream_t)stream);
    if (rc != SAPS_OK) return rc;
    PackArgs a;
    a.x = x;
    a.ld = (size_t)ctx->ld;
    a.N = (uint32_t)ctx->N;
    a.n = ctx->n;
    a.key = make_key(ctx->seed, t, keep_frac);
    a.col_offset = (uint32_t)ctx->col_offset;
    a.cap = (uint32_t)saps_pack_capacity(ctx, keep_frac);
    a.out_vals = out_vals;
    a.out_idx = out_idx;
    a.out_count = out_count;
    a.scratch = scratch_view(ctx->scratch, ctx->ntiles);
    a.spin_limit = ctx->spin_limit;
    a.skip_tile = ctx->skip_tile;
    return launch_pack(a, (cudaStream_t)stream) == cudaSuccess ? SAPS_OK : SAPS_ERR_CUDA;
}

int saps_pack_noalloc(saps_ctx* ctx, const float* x, uint64_t t, double keep_frac, float* out_vals,
                      uint32_t* out_idx, uint32_t* out_count, int* out_status, void* stream)
{
    if (ctx == nullptr || x == nullptr || out_vals == nullptr || out_count == nullptr || t == 0 ||
        !valid_frac(keep_frac))
        return SAPS_ERR_INVALID;
    if (ctx->N > SAPS_NOALLOC_MAX_N) return SAPS_ERR_TOO_LARGE;
    PackArgs a;
    a.x = x;
    a.ld = (size_t)ctx->ld;
    a.N = (uint32_t)ctx->N;
    a.n = ctx->n;
    a.key = make_key(ctx->seed, t, keep_frac);
    a.col_offset = (uint32_t)ctx->col_offset;
    a.cap = (uint32_t)saps_pack_capacity(ctx, keep_frac);
    a.out_vals = out_vals;
    a.out_idx = out_idx;
    a.out_count = out_count;
    a.spin_limit = ctx->spin_limit;
    a.skip_tile = ctx->skip_tile;
    if (launch_pack_static(a, ctx->ntiles, out_status, (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    return SAPS_OK;
}

namespace {

int ensure_emit_memory(saps_ctx* ctx)
{
    if (ctx->emit_mem != nullptr) return SAPS_OK;
    void* p = nullptr;
    if (cudaMalloc(&p, ((size_t)2 * ctx->ntiles + (size_t)3 * ctx->ngroups) * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        return SAPS_ERR_NOMEM;
    }
    ctx->emit_mem = static_cast<uint32_t*>(p);
    return SAPS_OK;
}

// Everything the fused kernel needs to emit round t's wire buffer: the per-tile and per-group
// counts of round t (taken from the previous call's run-ahead when they are there, counted now
// on `stream` otherwise).  Fills the emission fields of `a` and arranges for the kernel to count
// round t+1 ahead.
int prepare_emission(saps_ctx* ctx, uint64_t t, double keep_frac, uint32_t cap, uint32_t* out_idx,
                     uint32_t* out_count, float* out_vals, cudaStream_t stream, RoundArgs* a)
{
    int rc = ensure_scratch(ctx, stream);
    if (rc != SAPS_OK) return rc;
    rc = ensure_emit_memory(ctx);
    if (rc != SAPS_OK) return rc;
    const uint32_t nt = ctx->ntiles, ng = ctx->ngroups;
    const uint64_t thr = threshold64(keep_frac);
    uint32_t* cnt_now = ctx->emit_mem + (size_t)ctx->emit_cur * nt;
    uint32_t* cnt_next = ctx->emit_mem + (size_t)(ctx->emit_cur ^ 1) * nt;
    uint32_t* groups = ctx->emit_mem + (size_t)2 * nt;
    uint32_t* grp_now = groups + (size_t)ctx->group_cur * ng;
    uint32_t* grp_next = groups + (size_t)((ctx->group_cur + 1) % 3) * ng;
    uint32_t* grp_clear = groups + (size_t)((ctx->group_cur + 2) % 3) * ng;
    const bool have = ctx->ahead_valid && ctx->ahead_t == t && ctx->ahead_thr == thr &&
                      ctx->ahead_col_offset == (uint32_t)ctx->col_offset;
    ctx->ahead_valid = false;
    if (!have) {
        // nothing usable from the previous call: clear all group sums, count this round's mask
        if (cudaMemsetAsync(groups, 0, (size_t)3 * ng * sizeof(uint32_t), stream) != cudaSuccess ||
            launch_mask_count((uint32_t)ctx->N, (uint32_t)ctx->col_offset, make_key(ctx->seed, t, keep_frac), nt,
                              cnt_now, grp_now, ctx->group_shift, stream) != cudaSuccess) {
            cudaGetLastError();
            return SAPS_ERR_CUDA;
        }
    }
    a->out_vals = out_vals;
    a->cap = cap;
    a->tile_cnt = cnt_now;
    a->group_cnt = grp_now;
    a->out_idx = out_idx;
    a->out_count = out_count;
    a->status = static_cast<int*>(ctx->scratch);
    a->next_cnt = nullptr;
    a->next_group_cnt = nullptr;
    a->clear_group_cnt = nullptr;
    if (ctx->run_ahead && t + 1 != 0) {
        a->next_cnt = cnt_next;
        a->next_group_cnt = grp_next;
        a->clear_group_cnt = grp_clear;
        a->next_key = make_key(ctx->seed, t + 1, keep_frac);
        ctx->ahead_valid = true;   // true once the kernel the caller enqueues next has run
        ctx->ahead_t = t + 1;
        ctx->ahead_thr = thr;
        ctx->ahead_col_offset = (uint32_t)ctx->col_offset;
        ctx->emit_cur ^= 1;
        ctx->group_cur = (ctx->group_cur + 1) % 3;
    }
    return SAPS_OK;
}

}  // namespace

int saps_round_pack(saps_ctx* ctx, float* x, const float* g, float lr, const int32_t* pairs,
                    uint64_t t, double keep_frac, float* out_vals, uint32_t* out_idx,
                    uint32_t* out_count, void* stream)
{
    int rc = check_round_args(ctx, x, g, lr, t, keep_frac);
    if (rc != SAPS_OK) return rc;
    if (out_vals == nullptr || out_count == nullptr) return SAPS_ERR_INVALID;
    rc = check_pairs(ctx->n, pairs);
    if (rc != SAPS_OK) return rc;
    const RoundKey key = make_key(ctx->seed, t, keep_frac);
    const uint32_t cap = (uint32_t)saps_pack_capacity(ctx, keep_frac);
    // the kept columns per tile come from the previous call's kernel, or are counted now
    const RowGroups rg = make_groups(ctx->n, pairs, true);
    RoundArgs a = round_args(ctx, x, g, lr, rg, key);
    rc = prepare_emission(ctx, t, keep_frac, cap, out_idx, out_count, out_vals, (cudaStream_t)stream, &a);
    if (rc != SAPS_OK) return rc;
    // the fused round writes the kept columns and each worker's kept values at their ranks
    rc = timed_round(ctx, a, true, (cudaStream_t)stream);
    if (rc != SAPS_OK) ctx->ahead_valid = false;
    return rc;
}

int saps_round_pack_rows(saps_ctx* ctx, float* x, const float* g, float lr, const int32_t* pairs, uint64_t t,
                         double keep_frac, float* const* out_rows, uint32_t* out_idx, uint32_t* out_count,
                         void* stream)
{
    int rc = check_round_args(ctx, x, g, lr, t, keep_frac);
    if (rc != SAPS_OK) return rc;
    if (out_rows == nullptr || out_count == nullptr) return SAPS_ERR_INVALID;
    rc = check_pairs(ctx->n, pairs);
    if (rc != SAPS_OK) return rc;
    const RoundKey key = make_key(ctx->seed, t, keep_frac);
    const uint32_t cap = (uint32_t)saps_pack_capacity(ctx, keep_frac);
    const RowGroups rg = make_groups(ctx->n, pairs, true);
    RoundArgs a = round_args(ctx, x, g, lr, rg, key);
    rc = prepare_emission(ctx, t, keep_frac, cap, out_idx, out_count, nullptr, (cudaStream_t)stream, &a);
    if (rc != SAPS_OK) return rc;
    a.out_rows = out_rows;
    rc = timed_round(ctx, a, true, (cudaStream_t)stream);
    if (rc != SAPS_OK) ctx->ahead_valid = false;
    return rc;
}

int saps_set_run_ahead(saps_ctx* ctx, int enabled)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    ctx->run_ahead = enabled != 0;
    ctx->ahead_valid = false;
    return SAPS_OK;
}

int saps_set_select_params(saps_ctx* ctx, double b_thres, int t_thres)
{
    if (ctx == nullptr || t_thres < 0) return SAPS_ERR_INVALID;
    ctx->select.b_thres_default = b_thres != b_thres;
    ctx->select.b_thres = ctx->select.b_thres_default ? 0.0 : b_thres;
    ctx->select.t_thres = t_thres;
    return SAPS_OK;
}

int saps_select_peers(saps_ctx* ctx, const double* bandwidth, uint64_t t, int32_t* out_pairs)
{
    if (ctx == nullptr || bandwidth == nullptr || out_pairs == nullptr || t == 0 || t > SAPS_SELECT_MAX_T)
        return SAPS_ERR_INVALID;
    return select_peers(ctx->select, bandwidth, t, out_pairs);
}

int saps_select_reset(saps_ctx* ctx)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    ctx->select.R.assign(ctx->select.R.size(), kNever);
    ctx->select.last_t = 0;
    return SAPS_OK;
}

int saps_get_select_state(const saps_ctx* ctx, int64_t* out_R, uint64_t* out_last_t)
{
    if (ctx == nullptr) return SAPS_ERR_INVALID;
    if (out_R) std::memcpy(out_R, ctx->select.R.data(), ctx->select.R.size() * sizeof(int64_t));
    if (out_last_t) *out_last_t = ctx->select.last_t;
    return SAPS_OK;
}

int saps_set_select_state(saps_ctx* ctx, const int64_t* R, uint64_t last_t)
{
    if (ctx == nullptr || last_t > SAPS_SELECT_MAX_T) return SAPS_ERR_INVALID;
    if (R) {
        for (size_t e = 0; e < ctx->select.R.size(); ++e)
            if (R[e] != kNever && (R[e] < 0 || (uint64_t)R[e] > SAPS_SELECT_MAX_T)) return SAPS_ERR_INVALID;
        std::memcpy(ctx->select.R.data(), R, ctx->select.R.size() * sizeof(int64_t));
    }
    ctx->select.last_t = last_t;
    return SAPS_OK;
}

namespace {

// The coordinator's loop (Algorithm 1): for every round, the matching, then the fused round
// (with the wire buffer when out_vals is given), enqueued back to back without any
// host-device synchronisation.
int run_rounds_impl(saps_ctx* ctx, float* x, const float* g, float lr, uint64_t t_first, uint64_t T,
                    double keep_frac, const float* lr_list, const int32_t* pairs_list, const double* bandwidth,
                    int32_t* out_pairs_log, float* out_vals, uint32_t* out_idx, uint32_t* out_counts,
                    cudaStream_t stream)
{
    int rc = check_round_args(ctx, x, g, lr, t_first, keep_frac);
    if (rc != SAPS_OK) return rc;
    if (pairs_list == nullptr && bandwidth == nullptr) return SAPS_ERR_INVALID;
    if (t_first + T < t_first) return SAPS_ERR_INVALID;
    if (pairs_list == nullptr && T > 0 && t_first + T - 1 > SAPS_SELECT_MAX_T) return SAPS_ERR_INVALID;
    if (lr_list != nullptr) {
        if (g == nullptr) return SAPS_ERR_INVALID;
        for (uint64_t r = 0; r < T; ++r)
            if (lr_list[r] != lr_list[r]) return SAPS_ERR_INVALID;
    }
    const bool emit = out_vals != nullptr;
    if (emit && out_counts == nullptr) return SAPS_ERR_INVALID;
    const int n = ctx->n;
    const uint32_t cap = emit ? (uint32_t)saps_pack_capacity(ctx, keep_frac) : 0;
    int32_t chosen[kMaxWorkers];
    for (uint64_t r = 0; r < T; ++r) {
        const uint64_t t = t_first + r;
        const int32_t* pairs;
        if (pairs_list != nullptr) {
            pairs = pairs_list + r * (uint64_t)n;
        } else {
            rc = select_peers(ctx->select, bandwidth, t, chosen);
            if (rc != SAPS_OK) return rc;
            pairs = chosen;
        }
        rc = check_pairs(n, pairs);
        if (rc != SAPS_OK) return rc;
        if (out_pairs_log != nullptr) std::memcpy(out_pairs_log + r * (uint64_t)n, pairs, sizeof(int32_t) * n);
        const float lr_t = lr_list != nullptr ? lr_list[r] : lr;
        const RowGroups rg = make_groups(n, pairs, g != nullptr || emit);
        RoundArgs a = round_args(ctx, x, g, lr_t, rg, make_key(ctx->seed, t, keep_frac));
        if (emit) {
            rc = prepare_emission(ctx, t, keep_frac, cap, out_idx, out_counts + r, out_vals, stream, &a);
            if (rc != SAPS_OK) return rc;
        }
        if (launch_round(a, emit, stream) != cudaSuccess) {
            ctx->ahead_valid = false;
            return SAPS_ERR_CUDA;
        }
    }
    return SAPS_OK;
}

}  // namespace

int saps_run_rounds(saps_ctx* ctx, float* x, const float* g, float lr, uint64_t t_first, uint64_t T,
                    double keep_frac, const float* lr_list, const int32_t* pairs_list,
                    const double* bandwidth, int32_t* out_pairs_log, void* stream)
{
    return run_rounds_impl(ctx, x, g, lr, t_first, T, keep_frac, lr_list, pairs_list, bandwidth, out_pairs_log,
                           nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

int saps_run_rounds_pack(saps_ctx* ctx, float* x, const float* g, float lr, uint64_t t_first, uint64_t T,
                         double keep_frac, const float* lr_list, const int32_t* pairs_list,
                         const double* bandwidth, int32_t* out_pairs_log, float* out_vals, uint32_t* out_idx,
                         uint32_t* out_counts, void* stream)
{
    if (out_vals == nullptr) return SAPS_ERR_INVALID;
    return run_rounds_impl(ctx, x, g, lr, t_first, T, keep_frac, lr_list, pairs_list, bandwidth, out_pairs_log,
                           out_vals, out_idx, out_counts, (cudaStream_t)stream);
}

namespace {

// Optional wire-buffer outputs of the host-buffer entry point.
struct HostPack {
    float* vals_host;      // [n, cap]
    uint32_t* idx_host;    // [cap] or NULL
    uint32_t* count_host;  // one word
    float* d_vals;         // device staging
    uint32_t* d_idx;
    uint32_t* d_count;
};

int ensure_lanes(saps_ctx* ctx)
{
    if (ctx->lanes_ready) return SAPS_OK;
    constexpr int kStreams = saps_ctx::kMaxLanes + 1, kEvents = saps_ctx::kMaxLanes + 1;
    cudaStream_t streams[kStreams];
    cudaEvent_t events[kEvents];
    int ns = 0, ne = 0;
    while (ns < kStreams && cudaStreamCreateWithFlags(&streams[ns], cudaStreamNonBlocking) == cudaSuccess) ++ns;
    while (ns == kStreams && ne < kEvents &&
           cudaEventCreateWithFlags(&events[ne], cudaEventDisableTiming) == cudaSuccess)
        ++ne;
    if (ne != kEvents) {
        for (int m = 0; m < ne; ++m) cudaEventDestroy(events[m]);
        for (int m = 0; m < ns; ++m) cudaStreamDestroy(streams[m]);
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    for (int l = 0; l < saps_ctx::kMaxLanes; ++l) {
        ctx->lane_stream[l] = streams[l];
        ctx->lane_event[l] = events[l];
    }
    ctx->out_stream = streams[saps_ctx::kMaxLanes];
    ctx->scan_event = events[saps_ctx::kMaxLanes];
    ctx->lanes_ready = true;
    return SAPS_OK;
}

// The round acts column by column, so column chunks are independent.  Each chunk is copied in
// and computed on one of a few lane streams (round-robin); its result is copied out on a
// stream of its own, so that a lane can start its next copy-in without waiting for its last
// copy-out: the two copy directions and the kernels overlap, and the copy-in queue never
// runs dry.  With a wire buffer whose per-tile counts are not there yet, the counting kernel
// (which touches no model data) runs first on lane 0 and the other lanes wait for it.
int round_host_impl(saps_ctx* ctx, float* x_host, const float* g_host, float lr, const int32_t* pairs,
                    uint64_t t, double keep_frac, float* d_x, float* d_g, const HostPack* pack)
{
    // x_host == NULL: the model stays resident in d_x; only the gradients travel in
    int rc = check_round_args(ctx, d_x, g_host, lr, t, keep_frac);
    if (rc != SAPS_OK) return rc;
    if (d_x == nullptr || (g_host != nullptr && d_g == nullptr)) return SAPS_ERR_INVALID;
    if (pack != nullptr && (pack->vals_host == nullptr || pack->count_host == nullptr || pack->d_vals == nullptr ||
                            pack->d_count == nullptr || (pack->idx_host != nullptr && pack->d_idx == nullptr)))
        return SAPS_ERR_INVALID;
    rc = check_pairs(ctx->n, pairs);
    if (rc != SAPS_OK) return rc;
    rc = ensure_lanes(ctx);
    if (rc != SAPS_OK) return rc;
    const int n = ctx->n;
    const int lanes = ctx->host_lanes;
    const uint64_t N = ctx->N;
    const uint64_t ld_dev = ctx->ld;   // the staging matrices use the context's row stride
    const bool emit = pack != nullptr;
    const RowGroups rg = make_groups(n, pairs, g_host != nullptr || emit);
    const RoundKey key = make_key(ctx->seed, t, keep_frac);
    const uint32_t cap = emit ? (uint32_t)saps_pack_capacity(ctx, keep_frac) : 0;
    bool failed = false;
    RoundArgs emit_args = round_args(ctx, d_x, g_host != nullptr ? d_g : nullptr, lr, rg, key, ld_dev);
    if (emit) {
        // a counting kernel, if one was needed, runs on lane 0: the other lanes wait for it
        rc = prepare_emission(ctx, t, keep_frac, cap, pack->idx_host != nullptr ? pack->d_idx : nullptr,
                              pack->d_count, pack->d_vals, ctx->lane_stream[0], &emit_args);
        if (rc != SAPS_OK) return rc;
        failed |= cudaEventRecord(ctx->scan_event, ctx->lane_stream[0]) != cudaSuccess;
        for (int l = 1; l < lanes; ++l)
            failed |= cudaStreamWaitEvent(ctx->lane_stream[l], ctx->scan_event, 0) != cudaSuccess;
    }
    // Chunks of host_chunk_tiles column tiles; towards the end they halve (down to kMinChunkTiles),
    // because what follows the last copy-in (its kernel and its copy-out) is not overlapped with
    // anything and should be short.
    constexpr uint32_t kMinChunkTiles = 32;
    const uint32_t tiles_per_chunk = ctx->host_chunk_tiles;
    int lane = 0;
    uint32_t tc = 0;
    for (uint32_t tb = 0; tb < ctx->ntiles && !failed; tb += tc, lane = (lane + 1) % lanes) {
        const uint32_t remaining = ctx->ntiles - tb;
        const uint32_t half = (remaining + 1) / 2;
        const uint32_t tail = half >= kMinChunkTiles ? half : remaining;   // fewer than two small chunks left: one
        tc = tail < tiles_per_chunk ? tail : tiles_per_chunk;
        const uint64_t c0 = (uint64_t)tb * kTileCols;
        const uint64_t c1 = c0 + (uint64_t)tc * kTileCols < N ? c0 + (uint64_t)tc * kTileCols : N;
        const size_t width = (size_t)(c1 - c0) * sizeof(float);
        cudaStream_t s = ctx->lane_stream[lane];
        if (x_host != nullptr)
            failed |= cudaMemcpy2DAsync(d_x + c0, ld_dev * sizeof(float), x_host + c0, N * sizeof(float), width, n,
                                        cudaMemcpyHostToDevice, s) != cudaSuccess;
        if (g_host != nullptr)
            failed |= cudaMemcpy2DAsync(d_g + c0, ld_dev * sizeof(float), g_host + c0, N * sizeof(float), width,
                                        n, cudaMemcpyHostToDevice, s) != cudaSuccess;
        RoundArgs a = emit_args;
        a.tile_begin = tb;
        a.tile_count = tc;
        failed |= launch_round(a, emit, s) != cudaSuccess;
        // everything that leaves the device does so on out_stream, behind this chunk's kernel
        failed |= cudaEventRecord(ctx->lane_event[lane], s) != cudaSuccess;
        failed |= cudaStreamWaitEvent(ctx->out_stream, ctx->lane_event[lane], 0) != cudaSuccess;
        if (x_host != nullptr)
            failed |= cudaMemcpy2DAsync(x_host + c0, N * sizeof(float), d_x + c0, ld_dev * sizeof(float), width, n,
                                        cudaMemcpyDeviceToHost, ctx->out_stream) != cudaSuccess;
    }
    if (emit && !failed) {
        // out_stream has waited for every chunk's kernel, so the wire buffer is complete there
        cudaStream_t so = ctx->out_stream;
        failed |= cudaMemcpyAsync(pack->count_host, pack->d_count, sizeof(uint32_t), cudaMemcpyDeviceToHost, so) !=
                  cudaSuccess;
        failed |= cudaMemcpyAsync(pack->vals_host, pack->d_vals, (size_t)n * cap * sizeof(float),
                                  cudaMemcpyDeviceToHost, so) != cudaSuccess;
        if (pack->idx_host != nullptr)
            failed |= cudaMemcpyAsync(pack->idx_host, pack->d_idx, (size_t)cap * sizeof(uint32_t),
                                      cudaMemcpyDeviceToHost, so) != cudaSuccess;
    }
    for (int l = 0; l < lanes; ++l) failed |= cudaStreamSynchronize(ctx->lane_stream[l]) != cudaSuccess;
    failed |= cudaStreamSynchronize(ctx->out_stream) != cudaSuccess;
    if (failed) {
        ctx->ahead_valid = false;
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    return SAPS_OK;
}

}  // namespace

int saps_set_host_pipeline(saps_ctx* ctx, uint64_t chunk_columns, int lanes)
{
    if (ctx == nullptr || lanes < 0 || lanes > saps_ctx::kMaxLanes) return SAPS_ERR_INVALID;
    if (chunk_columns != 0) {
        const uint64_t tiles = (chunk_columns + kTileCols - 1) / kTileCols;
        ctx->host_chunk_tiles = tiles > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)tiles;
    }
    if (lanes != 0) ctx->host_lanes = lanes;
    return SAPS_OK;
}

int saps_round_host(saps_ctx* ctx, float* x_host, const float* g_host, float lr, const int32_t* pairs,
                    uint64_t t, double keep_frac, float* d_x, float* d_g)
{
    return round_host_impl(ctx, x_host, g_host, lr, pairs, t, keep_frac, d_x, d_g, nullptr);
}

int saps_round_pack_host(saps_ctx* ctx, float* x_host, const float* g_host, float lr, const int32_t* pairs,
                         uint64_t t, double keep_frac, float* d_x, float* d_g, float* out_vals_host,
                         uint32_t* out_idx_host, uint32_t* out_count_host, float* d_vals, uint32_t* d_idx,
                         uint32_t* d_count)
{
    const HostPack pack{out_vals_host, out_idx_host, out_count_host, d_vals, d_idx, d_count};
    return round_host_impl(ctx, x_host, g_host, lr, pairs, t, keep_frac, d_x, d_g, &pack);
}

int saps_status(saps_ctx* ctx, void* stream, int* out_device_status)
{
    if (ctx == nullptr || out_device_status == nullptr) return SAPS_ERR_INVALID;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    *out_device_status = SAPS_OK;
    if (ctx->scratch == nullptr) return SAPS_OK;
    // read and clear on the caller's stream: a non-blocking stream is not ordered with the
    // legacy default stream, and the clear must not land behind a later kernel's report
    cudaStream_t s = (cudaStream_t)stream;
    int st = 0;
    if (cudaMemcpyAsync(&st, ctx->scratch, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess ||
        (st != 0 && (cudaMemsetAsync(ctx->scratch, 0, sizeof(int), s) != cudaSuccess ||
                     cudaStreamSynchronize(s) != cudaSuccess))) {
        cudaGetLastError();
        return SAPS_ERR_CUDA;
    }
    *out_device_status = st;
    return SAPS_OK;
}

const char* saps_strerror(int status)
{
    switch (status) {
        case SAPS_OK: return "ok";
        case SAPS_ERR_INVALID: return "invalid argument";
        case SAPS_ERR_PAIRS: return "pairs is not an involution on 0..n-1";
        case SAPS_ERR_CUDA: return "CUDA runtime call failed";
        case SAPS_ERR_OVERFLOW: return "more kept columns than the pack capacity";
        case SAPS_ERR_TIMEOUT: return "a bounded wait on the device ran out (compaction look-back or staged copies)";
        case SAPS_ERR_NOMEM: return "out of memory";
        case SAPS_ERR_TOO_LARGE: return "N exceeds what the static scratch area of saps_pack_noalloc covers";
        default: return "unknown status";
    }
}

}  // extern "C"
