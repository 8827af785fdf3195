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


// ---- bulk asynchronous copies (global <-> shared memory, completion on an mbarrier) -------------
// Used by the 128-bit form of the round with gradients: one thread asks the copy engine for the
// block's four (or two) row pieces, everybody hashes the mask meanwhile, and the results leave the
// same way.  Addresses are 16-byte aligned and sizes multiples of 16 bytes by construction (the
// caller takes this path only for ld % 4 == 0 and 16-byte aligned bases; a tile starts at a
// multiple of 2048 columns and covers a multiple of 4).  No multicast, no other CTA involved.
__device__ __forceinline__ uint32_t shared_address(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_load(float* dst_shared, const float* src_global, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(shared_address(dst_shared)), "l"(src_global), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void bulk_store(float* dst_global, const float* src_shared, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(dst_global), "r"(shared_address(src_shared)), "r"(bytes) : "memory");
}

// Bounded wait for phase 0 of the barrier (every poll is itself a time-limited hardware wait).
constexpr uint32_t kBulkPolls = 1u << 20;
__device__ __forceinline__ bool bulk_wait(uint32_t bar)
{
    uint32_t done = 0;
    for (uint32_t it = 0; it < kBulkPolls && !done; ++it) {
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(bar), "r"(0u) : "memory");
    }
    return done != 0;
}

// Programmatic dependent launch: consecutive rounds in a stream are launched so that the next
// round's blocks may be set up, and hash their columns, while the last blocks of this round still
// run.  grid_dependents_may_start() lets the next launch begin once every block of this grid has
// started; wait_for_previous_grid() returns when the grid before this one in the stream (and with
// it every earlier one) has completed and its writes are visible.  A block touches global memory
// only behind that wait.  After any other kind of predecessor the wait returns at once.
__device__ __forceinline__ void grid_dependents_may_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_previous_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// GOSSIP_FIRST selects the order of Eq. 7 (average the current models, then subtract the
// gradient step) instead of Algorithm 2's (SGD step first, then average).
// BULK (VEC = 4 with gradients only): the row pieces travel through shared memory by bulk copies.
template <int VEC, bool HAS_G, bool EMIT, bool GOSSIP_FIRST, bool BULK>
__global__ void __launch_bounds__(kThreads, VEC == 4 ? 5 : 1) round_kernel(const RoundArgs a)
{
    static_assert(!BULK || (VEC == 4 && HAS_G), "bulk copies serve the 128-bit form with gradients");
    constexpr int U = kTileCols / (kThreads * VEC);
    constexpr int kWarps = kThreads / 32;
    const int tid = threadIdx.x;
    grid_dependents_may_start();
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

    // BULK: staging buffers x_a, g_a, x_b, g_b of the tile and the barrier their copies complete on
    __shared__ __align__(128) float s_stage[BULK ? 4 : 1][BULK ? kTileCols : 4];
    __shared__ __align__(8) unsigned long long s_bar;
    uint32_t bulk_bytes = 0;
    if constexpr (BULK) {
        const uint32_t bar = shared_address(&s_bar);
        const uint32_t cols = nfull > col_tile ? (uint32_t)(nfull - col_tile < kTileCols ? nfull - col_tile : kTileCols) : 0u;
        bulk_bytes = cols * (uint32_t)sizeof(float);
        if (tid == 0) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar));
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
        if (tid == 0 && bulk_bytes != 0) {
            wait_for_previous_grid();
            const uint32_t pieces = paired ? 4u : 2u;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(pieces * bulk_bytes) : "memory");
            bulk_load(s_stage[0], xa + col_tile, bulk_bytes, bar);
            bulk_load(s_stage[1], ga + col_tile, bulk_bytes, bar);
            if (paired) {
                bulk_load(s_stage[2], xb + col_tile, bulk_bytes, bar);
                bulk_load(s_stage[3], gb + col_tile, bulk_bytes, bar);
            }
        }
    }

    Chunk<VEC> va[U], vb[U], wa[U], wb[U];
    bool inb[U];
    uint32_t col[U];

    if constexpr (!BULK) wait_for_previous_grid();
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t k = col_tile + (uint64_t)(u * kThreads + tid) * VEC;
        inb[u] = k < nfull;
        col[u] = (uint32_t)k;
        if (!BULK && inb[u]) {
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
    // these few values never delays them.  (The counts may have been written by the previous
    // round's kernel while this one was already being set up: plain L2 loads, not the read-only path.)
    uint32_t excl_part = 0;
    auto load_rank_offset_share = [&]() {
        const uint32_t g = tile >> a.group_shift;
        for (uint32_t j = tid; j < g; j += kThreads) excl_part += __ldcg(a.group_cnt + j);
        for (uint32_t j = (g << a.group_shift) + tid; j < tile; j += kThreads) excl_part += __ldcg(a.tile_cnt + j);
    };
    if constexpr (EMIT && !BULK) load_rank_offset_share();

    uint32_t bits[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        bits[u] = 0;
        if (inb[u]) {
#pragma unroll
            for (int c = 0; c < VEC; ++c)
                bits[u] |= (column_kept(a.col_offset + col[u] + c, a.key) ? 1u : 0u) << c;
            if (!BULK && HAS_G && !GOSSIP_FIRST) {
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                    if (paired) vb[u].v[c] = sgd_step(vb[u].v[c], wb[u].v[c], a.lr);
                }
            }
        }
    }

    // BULK: the staged pieces have arrived (or, should the bounded wait ever run out, the thread
    // reads its vectors straight from global memory: same values, and the status word says so)
    bool staged = false;
    if constexpr (BULK) {
        // the columns are hashed by now; everything from here on reads or writes global memory
        wait_for_previous_grid();
        if constexpr (EMIT) load_rank_offset_share();
        staged = bulk_bytes != 0 && !a.staging_give_up && bulk_wait(shared_address(&s_bar));
        if (bulk_bytes != 0 && !staged && a.status != nullptr && *reinterpret_cast<volatile int*>(a.status) == 0)
            atomicCAS(a.status, 0, -5 /* SAPS_ERR_TIMEOUT */);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (inb[u]) {
                const int v = (u * kThreads + tid) * VEC;
                if (staged) {
                    const float4 p0 = *reinterpret_cast<const float4*>(&s_stage[0][v]);
                    const float4 p1 = *reinterpret_cast<const float4*>(&s_stage[1][v]);
                    va[u].v[0] = p0.x; va[u].v[1] = p0.y; va[u].v[2] = p0.z; va[u].v[3] = p0.w;
                    wa[u].v[0] = p1.x; wa[u].v[1] = p1.y; wa[u].v[2] = p1.z; wa[u].v[3] = p1.w;
                    if (paired) {
                        const float4 p2 = *reinterpret_cast<const float4*>(&s_stage[2][v]);
                        const float4 p3 = *reinterpret_cast<const float4*>(&s_stage[3][v]);
                        vb[u].v[0] = p2.x; vb[u].v[1] = p2.y; vb[u].v[2] = p2.z; vb[u].v[3] = p2.w;
                        wb[u].v[0] = p3.x; wb[u].v[1] = p3.y; wb[u].v[2] = p3.z; wb[u].v[3] = p3.w;
                    }
                } else {
                    va[u] = load_stream<VEC>(xa + col[u]);
                    wa[u] = load_stream<VEC>(ga + col[u]);
                    if (paired) {
                        vb[u] = load_stream<VEC>(xb + col[u]);
                        wb[u] = load_stream<VEC>(gb + col[u]);
                    }
                }
                if (!GOSSIP_FIRST) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                        if (paired) vb[u].v[c] = sgd_step(vb[u].v[c], wb[u].v[c], a.lr);
                    }
                }
            }
        }
    }

    uint32_t rank[U];       // EMIT only: rank of this thread's first kept column
    uint32_t total = 0;     // EMIT only: kept columns in the vector part of the tile
    uint32_t excl = 0;      // EMIT only: kept columns in all earlier tiles
    // EMIT only: where the two workers' packed values go.  Rows of one [n, cap] matrix, or, with
    // a table of destinations, any address this GPU can store to (a peer GPU's receive buffer,
    // for one: the stores then cross the link while the pass streams on); NULL = not wanted.
    float* dst_a = nullptr;
    float* dst_b = nullptr;
    if constexpr (EMIT) {
        if (a.out_rows != nullptr) {
            dst_a = a.out_rows[ra];
            dst_b = a.out_rows[rb];
        } else {
            dst_a = a.out_vals + (size_t)ra * a.cap;
            dst_b = a.out_vals + (size_t)rb * a.cap;
        }
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
                            if (dst_a != nullptr) dst_a[r] = va[u].v[c];
                            if (paired && dst_b != nullptr) dst_b[r] = vb[u].v[c];
                        }
                        ++r;
                    }
                }
            }
        }
    }

    // Without a gradient only vectors that hold a kept column change, so only those are stored.
    // Where every row starts on a 32-byte boundary (store_sectors), the threads that share a
    // 32-byte sector store together when any of them has a kept column: DRAM then receives whole
    // sectors and never has to merge a partial one with what it holds.
    uint32_t rewrite[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        rewrite[u] = bits[u];
        if constexpr (!HAS_G && VEC < 8) {
            if (a.store_sectors) {
#pragma unroll
                for (int d = 1; d < 8 / VEC; d <<= 1) rewrite[u] |= __shfl_xor_sync(0xFFFFFFFFu, rewrite[u], d);
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
                if (BULK) {
                    if (staged) {
                        const int v = (u * kThreads + tid) * VEC;
                        *reinterpret_cast<float4*>(&s_stage[0][v]) = make_float4(va[u].v[0], va[u].v[1], va[u].v[2], va[u].v[3]);
                        *reinterpret_cast<float4*>(&s_stage[2][v]) = make_float4(vb[u].v[0], vb[u].v[1], vb[u].v[2], vb[u].v[3]);
                    }
                } else if (HAS_G || a.store_all || rewrite[u]) {
                    // for dense masks (store_all) whole rows are written all the same, because many
                    // scattered stores cost more than one coalesced stream of unchanged values
                    store_stream<VEC>(xa + col[u], va[u]);
                    store_stream<VEC>(xb + col[u], vb[u]);
                }
            } else if (HAS_G) {
                if (GOSSIP_FIRST) {
#pragma unroll
                    for (int c = 0; c < VEC; ++c) va[u].v[c] = sgd_step(va[u].v[c], wa[u].v[c], a.lr);
                }
                if (BULK) {
                    if (staged) {
                        const int v = (u * kThreads + tid) * VEC;
                        *reinterpret_cast<float4*>(&s_stage[0][v]) = make_float4(va[u].v[0], va[u].v[1], va[u].v[2], va[u].v[3]);
                    }
                } else {
                    store_stream<VEC>(xa + col[u], va[u]);
                }
            }
        }
    }

    if constexpr (BULK) {
        // The results leave as two bulk stores when every thread had its inputs staged (so nothing
        // can still arrive in the buffers); otherwise every thread stores its own registers.
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const bool all_staged = __syncthreads_and(staged || bulk_bytes == 0) != 0;
        if (all_staged) {
            if (tid == 0 && bulk_bytes != 0) {
                bulk_store(xa + col_tile, s_stage[0], bulk_bytes);
                if (paired) bulk_store(xb + col_tile, s_stage[2], bulk_bytes);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the buffers are free again
            }
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (inb[u]) {
                    store_stream<VEC>(xa + col[u], va[u]);
                    if (paired) store_stream<VEC>(xb + col[u], vb[u]);
                }
            }
            // copies that were not seen to complete still target this block's buffers: give them
            // one more bounded wait before the block ends
            if (tid == 0) bulk_wait(shared_address(&s_bar));
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
                        if (dst_a != nullptr) dst_a[r] = pa;
                        if (paired && dst_b != nullptr) dst_b[r] = pb;
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
            for (uint32_t j = tid; j < a.ngroups; j += kThreads) t += __ldcg(a.group_cnt + j);
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

// A launch of fewer blocks than this serves a model that stays in L2, where the two extra block
// barriers of the staged form cost more than its better use of the memory system gains.
constexpr uint64_t kBulkMinBlocks = 4096;

// Launched as a programmatic dependent of whatever kernel precedes it in the stream: after another
// round kernel its blocks may start early (they wait for that grid before they touch memory),
// after anything else the launch is an ordinary one.
template <typename Kernel>
cudaError_t launch_dependent(Kernel kernel, dim3 grid, const RoundArgs& a, cudaStream_t stream)
{
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

template <int VEC, bool HAS_G, bool EMIT, bool GOSSIP_FIRST>
cudaError_t launch_variant(const RoundArgs& a, cudaStream_t stream)
{
    dim3 grid(a.tile_count, a.groups.count, 1);
    if constexpr (VEC == 4 && HAS_G) {
        // 128-bit accesses with gradients: staged through shared memory by bulk copies (32 KB a
        // block) for models that stream from HBM
        const bool bulk = a.staging == 2 || (a.staging == 0 && (uint64_t)a.tile_count * a.groups.count >= kBulkMinBlocks);
        if (bulk) {
            auto kernel = round_kernel<VEC, HAS_G, EMIT, GOSSIP_FIRST, true>;
            // once per process and kernel: let several blocks of 33 KB share an SM
            static const cudaError_t carve =
                cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (carve != cudaSuccess) return carve;
            return launch_dependent(kernel, grid, a, stream);
        }
    }
    return launch_dependent(round_kernel<VEC, HAS_G, EMIT, GOSSIP_FIRST, false>, grid, a, stream);
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
