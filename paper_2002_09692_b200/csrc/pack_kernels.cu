// Compaction of the kept coordinates (x~ = x o m, Eq. 2; the buffer a worker sends,
// Section II-B) and the mask bitmap.
//
// Single pass over column tiles: each warp hashes 32 consecutive columns at a time, a
// ballot gives their mask word and popc the count; a block scan orders the warps; a
// decoupled look-back over tile states orders the tiles.  Tiles take their number from an
// atomic ticket, so every predecessor of a waiting tile is already running or done; the
// wait is bounded all the same and ends with an error status, never a hang.
#include <mutex>

#include "internal.h"

namespace saps {
namespace {

// Scratch of the allocation-free compaction entry point: the same layout as a context's
// scratch (status word, ticket, tile states) for up to kStaticMaxTiles column
// tiles.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[16 + (size_t)kStaticMaxTiles * 8];

constexpr unsigned long long kFlagAggregate = 1ull << 32;
constexpr unsigned long long kFlagInclusive = 2ull << 32;

__device__ __forceinline__ unsigned long long peek_state(const unsigned long long* p)
{
    return *reinterpret_cast<const volatile unsigned long long*>(p);
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// Decoupled look-back, run by one full warp: publishes this tile's count, sums the counts of
// all earlier tiles (32 tile states per step), then publishes the inclusive prefix.
// Returns false when a predecessor did not publish within the poll budget (or another tile
// already reported an error); the status word then holds SAPS_ERR_TIMEOUT.
__device__ __forceinline__ bool lookback_exclusive(const ScratchView& sc, uint32_t tile, uint32_t total,
                                                   uint32_t spin_limit, uint32_t skip_tile, int lane,
                                                   uint32_t* out_excl)
{
    const bool publish = tile != skip_tile;  // the test hook makes one tile stay silent
    if (lane == 0 && publish)
        atomicExch(&sc.tile_state[tile], (tile == 0 ? kFlagInclusive : kFlagAggregate) | total);
    uint32_t excl = 0;
    bool ok = true;
    if (tile > 0) {
        long long look = (long long)tile - 1;  // newest tile of the window
        uint32_t polls = 0;
        while (true) {
            const long long idx = look - lane;
            // tiles before the first count as "inclusive prefix 0"
            const unsigned long long st = idx >= 0 ? peek_state(&sc.tile_state[idx]) : kFlagInclusive;
            const uint32_t flag = (uint32_t)(st >> 32);
            const uint32_t incl = __ballot_sync(0xFFFFFFFFu, flag == 2u);
            const uint32_t empty = __ballot_sync(0xFFFFFFFFu, flag == 0u);
            const int first = incl ? (__ffs(incl) - 1) : 32;  // nearest inclusive prefix
            const uint32_t needed = first >= 31 ? 0xFFFFFFFFu : ((2u << first) - 1u);
            if (empty & needed) {
                // a predecessor has not published yet: back off and poll again
                ++polls;
                bool give_up = polls > spin_limit;
                if ((polls & 63u) == 0u) give_up |= *reinterpret_cast<volatile int*>(sc.status) != 0;
                if (__any_sync(0xFFFFFFFFu, give_up)) {
                    ok = false;
                    break;
                }
                __nanosleep(polls < 64u ? 40u : 400u);
                continue;
            }
            const uint32_t mine = ((needed >> lane) & 1u) ? (uint32_t)st : 0u;
            excl += warp_sum(mine);
            if (first < 32) break;
            look -= 32;
        }
    }
    if (lane == 0) {
        if (ok) {
            if (tile > 0 && publish) atomicExch(&sc.tile_state[tile], kFlagInclusive | (excl + total));
        } else {
            atomicCAS(sc.status, 0, -5 /* SAPS_ERR_TIMEOUT */);
        }
    }
    *out_excl = excl;
    return ok;
}

// One kept value of x.  A sparse gather touches one 32-byte sector per value; the qualifier
// asks the L2 to fetch 64 bytes for it instead of the whole 128-byte line it would fetch by
// default, which halves the DRAM traffic of the gather (there is no smaller request size).
__device__ __forceinline__ float load_gather(const float* p)
{
    float v;
    asm volatile("ld.global.nc.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// THREADS = 256, or 128 for very sparse masks (a tile then has fewer values to gather than a
// large block has threads, and more, smaller blocks hide the look-back's latency better).
template <bool GATHER, int THREADS>
__global__ void __launch_bounds__(THREADS) pack_kernel(const PackArgs a)
{
    constexpr int kWarps = THREADS / 32;
    constexpr int kSteps = kTileCols / THREADS;  // ballots per warp
    __shared__ uint32_t s_tile, s_excl, s_abort;
    __shared__ uint32_t s_warp_cnt[kWarps];
    __shared__ uint16_t s_kept[kTileCols];        // kept columns as offsets inside the tile

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        s_tile = atomicAdd(a.scratch.ticket, 1u);
        s_abort = 0;
    }
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= a.scratch.ntiles) return;  // cannot happen with a cleared ticket; stay in bounds

    // ---- mask words of this warp's 8 x 32 columns ----
    // 32-bit column arithmetic: N < 2^32, so the tile's first column fits, and `rem` is the
    // number of columns from there to the end of the row.  The hash input of a column beyond
    // the row may wrap; it is masked by the bounds test.
    const uint32_t col0 = tile * (uint32_t)kTileCols;
    const uint32_t rem = a.N - col0;
    const uint32_t off0 = (uint32_t)warp * (32 * kSteps) + lane;
    const uint32_t hash0 = a.col_offset + col0 + off0;
    uint32_t word[kSteps];
    uint32_t cnt = 0;
    if (rem >= (uint32_t)kTileCols) {
#pragma unroll
        for (int s = 0; s < kSteps; ++s) {
            word[s] = __ballot_sync(0xFFFFFFFFu, column_kept(hash0 + s * 32, a.key));
            cnt += __popc(word[s]);
        }
    } else {
#pragma unroll
        for (int s = 0; s < kSteps; ++s) {
            word[s] = __ballot_sync(0xFFFFFFFFu, (off0 + s * 32 < rem) && column_kept(hash0 + s * 32, a.key));
            cnt += __popc(word[s]);
        }
    }
    if (lane == 0) s_warp_cnt[warp] = cnt;
    __syncthreads();
    uint32_t warp_off = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const uint32_t c = s_warp_cnt[w];
        warp_off += (w < warp) ? c : 0u;
        total += c;
    }

    // ---- order the tiles ----
    if (warp == 0) {
        uint32_t excl;
        const bool ok = lookback_exclusive(a.scratch, tile, total, a.spin_limit, a.skip_tile, lane, &excl);
        if (lane == 0) {
            if (ok)
                s_excl = excl;
            else
                s_abort = 1;
        }
    }

    // ---- the tile's kept columns, ascending, to shared memory (this needs no prefix) ----
    const uint32_t below = (1u << lane) - 1u;
    uint32_t r = warp_off;
#pragma unroll
    for (int s = 0; s < kSteps; ++s) {
        if ((word[s] >> lane) & 1u) s_kept[r + __popc(word[s] & below)] = (uint16_t)(off0 + s * 32);
        r += __popc(word[s]);
    }
    __syncthreads();
    if (s_abort) return;
    const uint32_t base = s_excl;

    if (tile == a.scratch.ntiles - 1 && tid == 0) {
        if (a.out_count != nullptr) *a.out_count = base + total;
        if (base + total > a.cap) atomicCAS(a.scratch.status, 0, -4 /* SAPS_ERR_OVERFLOW */);
    }
    if (total == 0) return;
    const uint32_t room = base < a.cap ? a.cap - base : 0u;
    const uint32_t take = total < room ? total : room;
    if (a.out_idx != nullptr)
        for (uint32_t q = tid; q < take; q += THREADS) a.out_idx[base + q] = a.col_offset + col0 + s_kept[q];

    // ---- gather: only the kept lanes of x are ever loaded ----
    if constexpr (GATHER) {
        // one flat loop over (worker, kept column): with a sparse mask a tile keeps only a few
        // columns, so looping over workers inside keeps every thread busy and all the
        // (uncoalesced, sector-sized) loads of a tile in flight at once
        const float* xt = a.x + col0;
        const uint32_t items = (uint32_t)a.n * take;
#pragma unroll 4
        for (uint32_t e = tid; e < items; e += THREADS) {
            const uint32_t i = e / take, q = e - i * take;
            a.out_vals[(size_t)i * a.cap + base + q] = load_gather(xt + (size_t)i * a.ld + s_kept[q]);
        }
    }
}

// Kept columns of every tile under one round's mask (no model data): one block per tile, and
// the sums over groups of 2^group_shift tiles (group_cnt must be zero before).
__global__ void __launch_bounds__(kThreads) mask_count_kernel(uint32_t N, uint32_t col_offset, RoundKey key,
                                                             uint32_t* tile_cnt, uint32_t* group_cnt,
                                                             uint32_t group_shift)
{
    constexpr int kSteps = kTileCols / kThreads;
    __shared__ uint32_t s_warp_cnt[kThreads / 32];
    const uint32_t tile = blockIdx.x;
    const uint32_t col0 = tile * (uint32_t)kTileCols;   // N < 2^32: no wrap
    const uint32_t rem = N - col0;
    const uint32_t hash0 = col_offset + col0 + threadIdx.x;
    uint32_t cnt = 0;
    if (rem >= (uint32_t)kTileCols) {
#pragma unroll
        for (int s = 0; s < kSteps; ++s) cnt += column_kept(hash0 + s * kThreads, key) ? 1u : 0u;
    } else {
#pragma unroll
        for (int s = 0; s < kSteps; ++s)
            cnt += (threadIdx.x + s * kThreads < rem && column_kept(hash0 + s * kThreads, key)) ? 1u : 0u;
    }
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if ((threadIdx.x & 31) == 0) s_warp_cnt[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t total = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) total += s_warp_cnt[w];
        tile_cnt[tile] = total;
        atomicAdd(group_cnt + (tile >> group_shift), total);
    }
}

__global__ void __launch_bounds__(kThreads) mask_kernel(uint32_t N, uint32_t col_offset, RoundKey key,
                                                        uint32_t* out_bits)
{
    const uint64_t k = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool kept = (k < N) && column_kept(col_offset + (uint32_t)k, key);
    const uint32_t w = __ballot_sync(0xFFFFFFFFu, kept);
    if ((threadIdx.x & 31) == 0 && k < N) out_bits[k >> 5] = w;
}

// Receiving side of the exchange (Algorithm 2, merge): one thread per (worker, received entry).
// The argument block stays in the constant bank (__grid_constant__): src[] is indexed by the block
// row, and without the qualifier every thread would first copy the whole block to local memory.
__global__ void __launch_bounds__(kThreads) unpack_avg_kernel(const __grid_constant__ UnpackArgs a)
{
    const uint32_t src = a.src[blockIdx.y];
    if (src == kNoPeer) return;
    uint32_t count = *a.count;
    if (count > a.cap) count = a.cap;
    const uint32_t r = blockIdx.x * kThreads + threadIdx.x;
    if (r >= count) return;
    const uint32_t k = __ldg(a.idx + r) - a.col_offset;
    if (k >= a.N) return;  // an index list of another shard: stay in bounds
    float* p = a.x + (size_t)blockIdx.y * a.ld + k;
    // an isolated value of a row: ask the L2 for 64 bytes, not for the whole 128-byte line
    float own;
    asm volatile("ld.global.L2::64B.f32 %0, [%1];" : "=f"(own) : "l"(p) : "memory");
    *p = __fmul_rn(0.5f, __fadd_rn(own, __ldg(a.recv + (size_t)src * a.cap + r)));
}

// Consensus distance, one block per kConsensusCols columns (half a column tile: blocks this
// small keep the last, partly filled wave of the grid short).  Per column the deviations are taken from
// worker 0's value (exact in fp64), sum d^2 - (sum d)^2 / n, so that identical workers give
// exactly zero and nearly identical ones lose no digits.  VEC = 4 streams 128-bit vectors.
// The kernel is a pure read stream: every thread first issues the loads of a batch of kRowBatch
// workers (independent 16-byte loads, all in flight together), then accumulates them.
constexpr int kRowBatch = 8;

template <int VEC>
__device__ __forceinline__ void load_row_chunk(const float* p, float (&v)[VEC])
{
    if constexpr (VEC == 4) {
        const float4 q = __ldcs(reinterpret_cast<const float4*>(p));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
        v[0] = __ldcs(p);
    }
}

template <int VEC>
__global__ void __launch_bounds__(kThreads) consensus_kernel(const float* __restrict__ x, size_t ld, uint32_t N, int n,
                                                             double* partials)
{
    constexpr int U = kConsensusCols / (kThreads * VEC);
    __shared__ double s_part[kThreads / 32];
    const int tid = threadIdx.x;
    // the kernel that adds up the partial sums may be set up while this one still runs; it waits
    // for this grid to complete before it reads anything
    cudaTriggerProgrammaticLaunchCompletion();
    double acc = 0.0;
    const uint64_t col0 = (uint64_t)blockIdx.x * kConsensusCols;
    const uint32_t nfull = (VEC == 4) ? (N & ~3u) : N;
    const double inv_n = 1.0 / (double)n;
#pragma unroll 1
    for (int u = 0; u < U; ++u) {
        const uint64_t k = col0 + (uint64_t)(u * kThreads + tid) * VEC;
        if (k < nfull) {
            const float* col = x + k;
            float first[VEC];
            load_row_chunk<VEC>(col, first);
            double pivot[VEC], sd[VEC], sdd[VEC];
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                pivot[c] = (double)first[c];
                sd[c] = sdd[c] = 0.0;
            }
            int i = 1;
            for (; i + kRowBatch <= n; i += kRowBatch) {
                float v[kRowBatch][VEC];
#pragma unroll
                for (int b = 0; b < kRowBatch; ++b) load_row_chunk<VEC>(col + (size_t)(i + b) * ld, v[b]);
#pragma unroll
                for (int b = 0; b < kRowBatch; ++b) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        const double d = (double)v[b][c] - pivot[c];
                        sd[c] += d;
                        sdd[c] = __fma_rn(d, d, sdd[c]);
                    }
                }
            }
            for (; i < n; ++i) {
                float v[VEC];
                load_row_chunk<VEC>(col + (size_t)i * ld, v);
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    const double d = (double)v[c] - pivot[c];
                    sd[c] += d;
                    sdd[c] = __fma_rn(d, d, sdd[c]);
                }
            }
#pragma unroll
            for (int c = 0; c < VEC; ++c) acc += sdd[c] - sd[c] * sd[c] * inv_n;
        }
    }
    if constexpr (VEC == 4) {
        // the last (N mod 4) columns
        if ((uint32_t)tid < N - nfull && col0 <= nfull && nfull < col0 + kConsensusCols) {
            const uint32_t k = nfull + tid;  // cannot wrap: tid < N - nfull
            const double pivot = (double)x[k];
            double sd = 0.0, sdd = 0.0;
            for (int i = 1; i < n; ++i) {
                const double d = (double)x[(size_t)i * ld + k] - pivot;
                sd += d;
                sdd = __fma_rn(d, d, sdd);
            }
            acc += sdd - sd * sd * inv_n;
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if ((tid & 31) == 0) s_part[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) t += s_part[w];
        partials[blockIdx.x] = t;
    }
}

// Adds the partial sums in a fixed order (the result is reproducible).  Launched so that it may
// start before the kernel above has finished: everything it reads comes after the wait.
constexpr int kFinalThreads = 1024;
__global__ void __launch_bounds__(kFinalThreads) consensus_final_kernel(const double* partials, uint32_t count,
                                                                        double* out)
{
    __shared__ double s_sum[kFinalThreads];
    const uint32_t tid = threadIdx.x;
    cudaGridDependencySynchronize();
    // eight loads in flight per thread; the order of the additions is fixed all the same
    double sum = 0.0;
    uint32_t i = tid;
    for (; i + 7 * kFinalThreads < count; i += 8 * kFinalThreads) {
        double v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldcg(partials + i + j * kFinalThreads);
#pragma unroll
        for (int j = 0; j < 8; ++j) sum += v[j];
    }
    for (; i < count; i += kFinalThreads) sum += __ldcg(partials + i);
    s_sum[tid] = sum;
    __syncthreads();
    for (uint32_t d = kFinalThreads / 2; d > 0; d >>= 1) {
        if (tid < d) s_sum[tid] += s_sum[tid + d];
        __syncthreads();
    }
    if (tid == 0) *out = s_sum[0] < 0.0 ? 0.0 : s_sum[0];
}

}  // namespace

cudaError_t launch_unpack_avg(const UnpackArgs& a, cudaStream_t stream)
{
    if (a.cap == 0 || a.n == 0) return cudaSuccess;
    dim3 grid((a.cap + kThreads - 1) / kThreads, a.n, 1);
    unpack_avg_kernel<<<grid, kThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_consensus(const float* x, size_t ld, uint32_t N, int n, double* partials, double* out,
                             cudaStream_t stream)
{
    const uint32_t blocks = consensus_blocks(N);
    if (ld % 4 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0)
        consensus_kernel<4><<<blocks, kThreads, 0, stream>>>(x, ld, N, n, partials);
    else
        consensus_kernel<1><<<blocks, kThreads, 0, stream>>>(x, ld, N, n, partials);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // programmatic dependent launch: the one-block summation is scheduled while the first kernel
    // drains, which removes the launch gap between the two
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, 1, 1);
    cfg.blockDim = dim3(kFinalThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, consensus_final_kernel, (const double*)partials, blocks, out);
}

// Block size by the expected number of values a tile gathers (n workers x kept columns per tile).
static void launch_pack_kernel(const PackArgs& a, uint32_t ntiles, cudaStream_t stream)
{
    const double kept_per_tile = a.key.all ? (double)kTileCols : (double)kTileCols * a.key.thr32 / 4294967296.0;
    if ((double)a.n * kept_per_tile < 128.0)
        pack_kernel<true, 128><<<ntiles, 128, 0, stream>>>(a);
    else
        pack_kernel<true, kThreads><<<ntiles, kThreads, 0, stream>>>(a);
}

cudaError_t launch_pack(const PackArgs& a, cudaStream_t stream)
{
    const uint32_t ntiles = a.scratch.ntiles;
    cudaError_t e = cudaMemsetAsync(a.scratch.ticket, 0, scratch_clear_bytes(ntiles), stream);
    if (e != cudaSuccess) return e;
    launch_pack_kernel(a, ntiles, stream);
    return cudaGetLastError();
}

// In host code `g_static_scratch` names a host-side shadow of the device array, not device
// memory; the address a kernel may use has to be asked for, per device, with that device
// current.  It is looked up once per device and remembered.
cudaError_t static_scratch_address(void** out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex lock;
    static void* address[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> hold(lock);
    if (address[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        address[dev] = p;
    }
    *out = address[dev];
    return cudaSuccess;
}

cudaError_t launch_pack_static(PackArgs a, uint32_t ntiles, int* out_status, cudaStream_t stream)
{
    if (ntiles == 0 || ntiles > kStaticMaxTiles) return cudaErrorInvalidValue;
    void* base = nullptr;
    cudaError_t e = static_scratch_address(&base);
    if (e != cudaSuccess) return e;
    a.scratch = scratch_view(base, ntiles);
    // the area keeps whatever the previous call left: status, ticket and tile states restart at zero
    e = cudaMemsetAsync(base, 0, 4 + scratch_clear_bytes(ntiles), stream);
    if (e != cudaSuccess) return e;
    launch_pack_kernel(a, ntiles, stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (out_status != nullptr)
        e = cudaMemcpyAsync(out_status, a.scratch.status, sizeof(int), cudaMemcpyDeviceToDevice, stream);
    return e;
}

cudaError_t launch_mask_count(uint32_t N, uint32_t col_offset, RoundKey key, uint32_t ntiles, uint32_t* tile_cnt,
                              uint32_t* group_cnt, uint32_t group_shift, cudaStream_t stream)
{
    mask_count_kernel<<<ntiles, kThreads, 0, stream>>>(N, col_offset, key, tile_cnt, group_cnt, group_shift);
    return cudaGetLastError();
}

cudaError_t launch_mask(uint32_t N, uint32_t col_offset, RoundKey key, uint32_t* out_bits,
                        cudaStream_t stream)
{
    const uint32_t blocks = (uint32_t)(((uint64_t)N + kThreads - 1) / kThreads);
    mask_kernel<<<blocks, kThreads, 0, stream>>>(N, col_offset, key, out_bits);
    return cudaGetLastError();
}

}  // namespace saps
