// Internal declarations shared by the translation units of libsaps.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "mask_hash.cuh"

namespace saps {

// One column tile: the unit of the compaction scan and of a round-kernel block.
constexpr int kTileCols = 2048;
constexpr int kThreads = 256;
constexpr uint32_t kMaxWorkers = 64;
constexpr uint8_t kNoPeer = 0xFF;

// Rows served by one block row of the round kernel: a matched pair (a, b) or a single
// worker (b == kNoPeer).  Passed by value in the kernel parameter block, so a round needs
// no host-to-device copy and no staging buffer that a later round could overwrite.
struct RowGroups {
    int count;
    uint8_t a[kMaxWorkers];
    uint8_t b[kMaxWorkers];
};

// Device scratch of a context (also the layout of the static no-allocation area).
//   word 0            status (first device-found error, sticky until read)
//   word 1            tile ticket of the running scan
//   words 2..3        unused
//   then ntiles x u64 tile states {flag << 32 | value}
struct ScratchView {
    int* status;
    uint32_t* ticket;
    unsigned long long* tile_state;
    uint32_t ntiles;
};

inline size_t scratch_bytes(uint32_t ntiles)
{
    return 16 + (size_t)ntiles * 8;
}

inline ScratchView scratch_view(void* base, uint32_t ntiles)
{
    char* p = static_cast<char*>(base);
    ScratchView v;
    v.status = reinterpret_cast<int*>(p);
    v.ticket = reinterpret_cast<uint32_t*>(p + 4);
    v.tile_state = reinterpret_cast<unsigned long long*>(p + 16);
    v.ntiles = ntiles;
    return v;
}

// Bytes that must be zero before a scan starts: ticket + padding + tile states.
inline size_t scratch_clear_bytes(uint32_t ntiles) { return 12 + (size_t)ntiles * 8; }

// Poll budget of the look-back before it gives up (about a second with the back-off used).
constexpr uint32_t kSpinLimit = 1u << 21;

// ---- launchers (defined in the .cu files) ----------------------------------------------

struct RoundArgs {
    float* x;
    const float* g;
    size_t ld;
    uint32_t N;
    float lr;
    RowGroups groups;
    RoundKey key;
    uint32_t col_offset;   // global index of this shard's column 0 (mask hash input)
    uint32_t tile_begin;   // first column tile to process
    uint32_t tile_count;   // number of column tiles to process
    int gossip_first;      // 0: Algorithm 2's order (SGD, then average); 1: Eq. 7's order
    int staging;           // 0: chosen by size; 1: loads and stores from registers; 2: bulk copies through shared memory
    int staging_give_up;   // test hook: the staged form treats its wait for the copies as run out
    int store_all;         // round without gradient: write unchanged vectors too (dense masks)
    int store_sectors;     // round without gradient: rows start on 32-byte boundaries, store whole sectors
    // emission of the wire buffer (all NULL/0 when not emitting).  The ranks of a tile's kept
    // columns start at the number of kept columns in all earlier tiles.  That number is summed by
    // the block itself from two small arrays: the kept columns per tile, and their sums over
    // groups of 2^group_shift consecutive tiles.
    float* out_vals;             // [n, cap], or NULL when out_rows is given
    float* const* out_rows;      // device array of n destinations (NULL entries: not emitted), or NULL
    uint32_t cap;
    const uint32_t* tile_cnt;    // kept columns per tile, this round
    const uint32_t* group_cnt;   // the same summed over every group of tiles
    uint32_t group_shift;
    uint32_t ngroups;
    uint32_t* out_idx;           // kept columns, written by the first row group (may be NULL)
    uint32_t* out_count;         // total, written by the block of tile 0 (may be NULL)
    int* status;                 // receives SAPS_ERR_OVERFLOW when the total exceeds cap
    // run-ahead for the next round: the first row group also counts, per tile and per group, the
    // columns that the NEXT round's mask keeps (NULL = off), and clears the group sums that the
    // round after next will accumulate into
    uint32_t* next_cnt;
    uint32_t* next_group_cnt;
    uint32_t* clear_group_cnt;
    RoundKey next_key;
};

cudaError_t launch_round(const RoundArgs& a, bool emit, cudaStream_t stream);

struct PackArgs {
    const float* x;
    size_t ld;
    uint32_t N;
    int n;
    RoundKey key;
    uint32_t col_offset;  // added to k for the hash and in out_idx
    uint32_t cap;
    float* out_vals;      // NULL: scan only (indices, count and tile prefixes)
    uint32_t* out_idx;    // may be NULL
    uint32_t* out_count;  // may be NULL
    ScratchView scratch;
    uint32_t spin_limit;
    uint32_t skip_tile;   // test hook: this look-back tile never publishes (0xFFFFFFFF = none)
};

cudaError_t launch_pack(const PackArgs& a, cudaStream_t stream);

// Mask scan without model data: kept columns per tile, added up per group of 2^group_shift tiles
// as well (group_cnt must be zero before).
cudaError_t launch_mask_count(uint32_t N, uint32_t col_offset, RoundKey key, uint32_t ntiles, uint32_t* tile_cnt,
                              uint32_t* group_cnt, uint32_t group_shift, cudaStream_t stream);

cudaError_t launch_mask(uint32_t N, uint32_t col_offset, RoundKey key, uint32_t* out_bits,
                        cudaStream_t stream);

// Receiving side of the exchange: x[i][idx[r]] = (x[i][idx[r]] + recv[src[i]][r]) / 2.
struct UnpackArgs {
    float* x;
    size_t ld;
    int n;
    const float* recv;     // [n, cap]
    uint32_t cap;
    const uint32_t* idx;   // global columns
    const uint32_t* count; // device
    uint32_t col_offset;
    uint32_t N;
    uint8_t src[kMaxWorkers];  // row of recv that worker i received, kNoPeer = nothing received
};
cudaError_t launch_unpack_avg(const UnpackArgs& a, cudaStream_t stream);

// || X - mean over workers ||_F^2: one partial sum per block of kConsensusCols columns
// (consensus_blocks(N) doubles), then a one-block kernel adds them in a fixed order.
constexpr int kConsensusCols = 1024;
inline uint32_t consensus_blocks(uint32_t N) { return (uint32_t)(((uint64_t)N + kConsensusCols - 1) / kConsensusCols); }
cudaError_t launch_consensus(const float* x, size_t ld, uint32_t N, int n, double* partials, double* out,
                             cudaStream_t stream);

// Compaction on the library's static scratch area (no allocation anywhere on the path).
constexpr uint32_t kStaticMaxTiles = 65536;  // kTileCols columns each: N <= 134,217,728
cudaError_t launch_pack_static(PackArgs a, uint32_t ntiles, int* out_status, cudaStream_t stream);

// ---- host-side peer selection (select_peers.cpp) ------------------------------------------

struct SelectState {
    int n = 0;
    uint64_t seed = 0;
    double b_thres = 0.0;
    bool b_thres_default = true;
    int t_thres = 0;  // 0 = default
    uint64_t last_t = 0;
    std::vector<int64_t> R;  // n x n, kNever = never
    // what the last call derived from its bandwidth matrix, reused while the caller keeps passing
    // the same matrix and threshold setting (the usual case: one matrix for a whole run)
    std::vector<double> seen_bandwidth;   // the matrix as it was passed in
    std::vector<double> sym_bandwidth;    // min(B, B^T), zero diagonal
    double seen_b_thres_setting = 0.0;
    bool seen_b_thres_default = false;
    double derived_b_thres = 0.0;
    uint64_t any_link[kMaxWorkers] = {};    // row masks: links with B_ij > 0
    uint64_t fast_link[kMaxWorkers] = {};   // row masks: links of B* (B_ij >= B_thres)
    bool derived_valid = false;
};

constexpr int64_t kNever = -(1LL << 62);

int select_peers(SelectState& st, const double* bandwidth, uint64_t t, int32_t* out_pairs);

}  // namespace saps
