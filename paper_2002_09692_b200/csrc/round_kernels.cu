// Fused gossip round: SGD step (Algorithm 2, SGD procedure), round mask (Section II-B,
// Eq. 3), pair average (Algorithm 2 merge with the weights of GenerateW; Eq. 7), and
// optionally the emission of the wire buffer (Eq. 2) from the same pass.
//
// One block serves one column tile of one row group (a matched pair, or a single worker).
// Every thread streams 128-bit vectors of x_i, g_i, x_j, g_j, hashes its columns once for
// both rows, and writes x_i and x_j back: 12 bytes of HBM traffic per worker-parameter,
// which is what bounds the kernel.  fp32 operations use the round-to-nearest intrinsics so
// that nothing is contracted into a fused multiply-add.
#include "internal.h"

namespace saps {
namespace {

__device__ __forceinline__ float sgd_step(float x, float g, float lr)
{
    return __fsub_rn(x, __fmul_rn(lr, g));
}

__device__ __forceinline__ float pair_mean(float a, float b)
{
    return __fmul_rn(0.5f, __fadd_rn(a, b));
}

template <int VEC>
struct Chunk {
    float v[VEC];
};

// Streaming (evict-first) accesses: every byte is touched once per round.
template <int VEC>
__device__ __forceinline__ Chunk<VEC> load_stream(const float* p)
{
    Chunk<VEC> c;
    if constexpr (VEC == 4) {
        float4 t = __ldcs(reinterpret_cast<const float4*>(p));
        c.v[0] = t.x; c.v[1] = t.y; c.v[2] = t.z; c.v[3] = t.w;
    } else if constexpr (VEC == 2) {
        float2 t = __ldcs(reinterpret_cast<const float2*>(p));
        c.v[0] = t.x; c.v[1] = t.y;
    } else {
        c.v[0] = __ldcs(p);
    }
    return c;
}

template <int VEC>
__device__ __forceinline__ void store_stream(float* p, const Chunk<VEC>& c)
{
    if constexpr (VEC == 4) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(c.v[0], c.v[1], c.v[2], c.v[3]));
    } else if constexpr (VEC == 2) {
        __stcs(reinterpret_cast<float2*>(p), make_float2(c.v[0], c.v[1]));
    } else {
        __stcs(p, c.v[0]);
    }
}

__device__ __forceinline__ uint32_t warp_inclusive_sum(uint32_t v, int lane)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// GOSSIP_FIRST selects the order of Eq. 7 (average the current models, then subtract the
// gradient step) instead of Algorithm 2's (SGD step first, then average).
template <int VEC, bool HAS_G, bool EMIT, bool GOSSIP_FIRST>
__global__ void __launch_bounds__(kThreads, VEC == 4 ? 5 : 1) round_kernel(const RoundArgs a)
{
    constexpr int U = kTileCols / (kThreads * VEC);
    constexpr int kWarps = kThreads / 32;
    const int tid = threadIdx.x;
    const uint32_t tile = a.tile_begin + blockIdx.x;
    const uint32_t ra = a.groups.a[blockIdx.y];
    const uint32_t rb_raw = a.groups.b[blockIdx.y];
    const bool paired = rb_raw != kNoPeer;
    const uint32_t rb = paired ? rb_raw : ra;

    float* __restrict__ xa = a.x + (size_t)ra * a.ld;
    float* __restrict__ xb = a.x + (size_t)rb * a.ld;
    const float* __restrict__ ga = HAS_G ? a.g + (size_t)ra * a.ld : nullptr;
    const float* __restrict__ gb = HAS_G ? a.g + (size_t)rb * a.ld : nullptr;

    // columns reachable by whole vectors; the (N mod VEC) leftovers are handled at the end
    const uint32_t nfull = a.N - a.N % VEC;
    const uint64_t col_tile = (uint64_t)tile * kTileCols;

    Chunk<VEC> va[U], vb[U], wa[U], wb[U];
    bool inb[U];
    uint32_t col[U];

#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t k = col_tile + (uint64_t)(u * kThreads + tid) * VEC;
        inb[u] = k < nfull;
        col[u] = (uint32_t)k;
        if (inb[u]) {
            va[u] = load_stream<VEC>(xa + k);
            if (HAS_G) wa[u] = load_stream<VEC>(ga + k);
            if (paired) {
                vb[u] = load_stream<VEC>(xb + k);
                if (HAS_G) wb[u] = load_stream<VEC>(gb + k);
            }
        }
    }

    // The rank offset of the tile = kept columns in all earlier tiles: whole groups of tiles from
    // the group sums, the rest tile by tile; every thread takes a share (one load, seldom more),
    // the block adds them up further down.  Placed behind the model loads, so that waiting for
    // these few values never delays them.
    uint32_t excl_part = 0;
    if constexpr (EMIT) {
        const uint32_t g = tile >> a.group_shift;
        for (uint32_t j = tid; j < g; j += kThreads) excl_part += __ldg(a.group_cnt + j);
        for (uint32_t j = (g << a.group_shift) + tid; j < tile; j += kThreads) excl_part += __ldg(a.tile_cnt + j);
    }

    uint32_t bits[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        bits[u] = 0;
        if (inb[u]) {
#pragma unroll
            for (int c = 0; c < VEC; ++c)
                bits[u] |= (column_kept(a.col_offset + col[u] + c, a.key) ? 1u : 0u) << c;
            if (HAS_G && !GOSSIP_FIRST) {
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                    if (paired) vb[u].v[c] = sgd_step(vb[u].v[c], wb[u].v[c], a.lr);
                }
            }
        }
    }

    uint32_t rank[U];       // EMIT only: rank of this thread's first kept column
    uint32_t total = 0;     // EMIT only: kept columns in the vector part of the tile
    uint32_t excl = 0;      // EMIT only: kept columns in all earlier tiles
    if constexpr (EMIT) {
        // Two counts travel in one word (16 bits each: a tile keeps at most 2048 columns), so one
        // warp scan and one pass over the warps' totals serve two of the thread's vectors.
        static_assert(U % 2 == 0, "vectors are ranked two at a time");
        constexpr int P = U / 2;
        __shared__ uint32_t s_warp[P][kWarps];
        __shared__ uint32_t s_excl[32];
        const int lane = tid & 31, warp = tid >> 5;
        {
            const uint32_t e = __reduce_add_sync(0xFFFFFFFFu, excl_part);
            if (lane == 0) s_excl[warp] = e;
        }
        uint32_t within[P];
#pragma unroll
        for (int j = 0; j < P; ++j) {
            const uint32_t c = __popc(bits[2 * j]) | (__popc(bits[2 * j + 1]) << 16);
            const uint32_t inc = warp_inclusive_sum(c, lane);
            within[j] = inc - c;
            if (lane == 31) s_warp[j][warp] = inc;
        }
        __syncthreads();
        excl = __reduce_add_sync(0xFFFFFFFFu, lane < kWarps ? s_excl[lane] : 0u);
        uint32_t running = excl;
#pragma unroll
        for (int j = 0; j < P; ++j) {
            uint32_t before = 0, all = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const uint32_t s = s_warp[j][w];
                before += (w < warp) ? s : 0u;
                all += s;
            }
            const uint32_t mine = before + within[j];
            rank[2 * j] = running + (mine & 0xFFFFu);
            running += all & 0xFFFFu;
            rank[2 * j + 1] = running + (mine >> 16);
            running += all >> 16;
        }
        total = running - excl;
        // the list of kept columns is the same for every row group: the first one writes it
        if (blockIdx.y == 0 && a.out_idx != nullptr) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                uint32_t r = rank[u];
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    if ((bits[u] >> c) & 1u) {
                        if (r < a.cap) a.out_idx[r] = a.col_offset + col[u] + c;
                        ++r;
                    }
                }
            }
        }
        // run-ahead: how many columns of this tile the next round's mask keeps
        if (blockIdx.y == 0 && a.next_cnt != nullptr) {
            __shared__ uint32_t s_next[kWarps];
            uint32_t c = 0;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (inb[u]) {
#pragma unroll
                    for (int q = 0; q < VEC; ++q) c += column_kept(a.col_offset + col[u] + q, a.next_key) ? 1u : 0u;
                }
            }
            if constexpr (VEC > 1) {
                // the (N mod VEC) leftover columns belong to the last tile; tid is compared with
                // their number first, so that nfull + tid cannot wrap for N close to 2^32
                if ((uint32_t)tid < a.N - nfull && col_tile <= nfull && nfull < col_tile + kTileCols)
                    c += column_kept(a.col_offset + nfull + tid, a.next_key) ? 1u : 0u;
            }
            c = __reduce_add_sync(0xFFFFFFFFu, c);
            if (lane == 0) s_next[warp] = c;
            __syncthreads();
            if (tid == 0) {
                uint32_t t = 0;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) t += s_next[w];
                a.next_cnt[tile] = t;
                atomicAdd(a.next_group_cnt + (tile >> a.group_shift), t);
            }
        }
        // what each worker sends: its value before the average (post-SGD in Algorithm 2's order)
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (bits[u]) {
                uint32_t r = rank[u];
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    if ((bits[u] >> c) & 1u) {
                        if (r < a.cap) {
                            a.out_vals[(size_t)ra * a.cap + r] = va[u].v[c];
                            if (paired) a.out_vals[(size_t)rb * a.cap + r] = vb[u].v[c];
                        }
                        ++r;
                    }
                }
            }
        }
    }

#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (inb[u]) {
            if (paired) {
                if (bits[u]) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        if ((bits[u] >> c) & 1u) {
                            const float m = pair_mean(va[u].v[c], vb[u].v[c]);
                            va[u].v[c] = m;
                            vb[u].v[c] = m;
                        }
                    }
                }
                if (HAS_G && GOSSIP_FIRST) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                        vb[u].v[c] = sgd_step(vb[u].v[c], wb[u].v[c], a.lr);
                    }
                }
                if (HAS_G || bits[u]) {
                    store_stream<VEC>(xa + col[u], va[u]);
                    store_stream<VEC>(xb + col[u], vb[u]);
                }
            } else if (HAS_G) {
                if (GOSSIP_FIRST) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                }
                store_stream<VEC>(xa + col[u], va[u]);
            }
        }
    }

    // the last (N mod VEC) columns of a row, one thread each
    if constexpr (VEC > 1) {
        const uint32_t ntail = a.N - nfull;
        if (ntail != 0 && tid < ntail && col_tile <= nfull && nfull < col_tile + kTileCols) {
            const uint32_t k = nfull + tid;
            float pa = xa[k], pb = 0.f;
            if (HAS_G && !GOSSIP_FIRST) pa = sgd_step(pa, ga[k], a.lr);
            if (paired) {
                pb = xb[k];
                if (HAS_G && !GOSSIP_FIRST) pb = sgd_step(pb, gb[k], a.lr);
            }
            const bool kept = column_kept(a.col_offset + k, a.key);
            if constexpr (EMIT) {
                if (kept) {
                    uint32_t r = excl + total;
                    for (uint32_t q = nfull; q < k; ++q) r += column_kept(a.col_offset + q, a.key) ? 1u : 0u;
                    if (r < a.cap) {
                        if (blockIdx.y == 0 && a.out_idx != nullptr) a.out_idx[r] = a.col_offset + k;
                        a.out_vals[(size_t)ra * a.cap + r] = pa;
                        if (paired) a.out_vals[(size_t)rb * a.cap + r] = pb;
                    }
                }
            }
            if (paired && kept) pa = pb = pair_mean(pa, pb);
            if (HAS_G && GOSSIP_FIRST) {
                pa = sgd_step(pa, ga[k], a.lr);
                if (paired) pb = sgd_step(pb, gb[k], a.lr);
            }
            if (paired) {
                if (HAS_G || kept) {
                    xa[k] = pa;
                    xb[k] = pb;
                }
            } else if (HAS_G) {
                xa[k] = pa;
            }
        }
    }

    // once per round, by the block of tile 0: the total of kept columns, the overflow report,
    // and clean group sums for the round after next
    if constexpr (EMIT) {
        if (tile == 0 && blockIdx.y == 0) {
            __shared__ uint32_t s_tot[kWarps];
            uint32_t t = 0;
            for (uint32_t j = tid; j < a.ngroups; j += kThreads) t += __ldg(a.group_cnt + j);
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, d);
            if ((tid & 31) == 0) s_tot[tid >> 5] = t;
            __syncthreads();
            if (tid == 0) {
                uint32_t sum = 0;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) sum += s_tot[w];
                if (a.out_count != nullptr) *a.out_count = sum;
                if (sum > a.cap) atomicCAS(a.status, 0, -4 /* SAPS_ERR_OVERFLOW */);
            }
            if (a.clear_group_cnt != nullptr)
                for (uint32_t j = tid; j < a.ngroups; j += kThreads) a.clear_group_cnt[j] = 0;
        }
    }
}

template <int VEC, bool HAS_G, bool EMIT, bool GOSSIP_FIRST>
cudaError_t launch_variant(const RoundArgs& a, cudaStream_t stream)
{
    dim3 grid(a.tile_count, a.groups.count, 1);
    round_kernel<VEC, HAS_G, EMIT, GOSSIP_FIRST><<<grid, kThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

template <int VEC>
cudaError_t launch_vec(const RoundArgs& a, bool emit, cudaStream_t stream)
{
    if (a.g == nullptr)  // without a gradient both orders are the same update
        return emit ? launch_variant<VEC, false, true, false>(a, stream)
                    : launch_variant<VEC, false, false, false>(a, stream);
    if (a.gossip_first)
        return emit ? launch_variant<VEC, true, true, true>(a, stream)
                    : launch_variant<VEC, true, false, true>(a, stream);
    return emit ? launch_variant<VEC, true, true, false>(a, stream)
                : launch_variant<VEC, true, false, false>(a, stream);
}

}  // namespace

cudaError_t launch_round(const RoundArgs& a, bool emit, cudaStream_t stream)
{
    if (a.groups.count == 0 || a.tile_count == 0) return cudaSuccess;
    // widest access that every row start allows: 128-bit, else 64-bit, else scalar
    const uintptr_t bits = reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.g) |
                           (uintptr_t)(a.ld * sizeof(float));
    if (bits % 16 == 0) return launch_vec<4>(a, emit, stream);
    if (bits % 8 == 0) return launch_vec<2>(a, emit, stream);
    return launch_vec<1>(a, emit, stream);
}

}  // namespace saps
