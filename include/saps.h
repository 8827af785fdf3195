/*
 * saps.h - C ABI of the SAPS-PSGD gossip-round library for NVIDIA B200 (sm_100a).
 *
 * The library runs the per-round sparsified pairwise model exchange of SAPS-PSGD
 * (Tang, Shi, Chu: "Communication-Efficient Decentralized Learning with
 * Sparsification and Adaptive Peer Selection") for n simulated workers whose
 * models are the rows of one [n, ld] fp32 matrix in the memory of ONE GPU:
 *
 *   1. local SGD step            a_i = x_i - lr * g_i            (Algorithm 2, SGD procedure)
 *   2. round mask                m_t[k] in {0,1}, Bernoulli(keep_frac), the same for
 *                                every worker                    (Section II-B, Eq. 3)
 *   3. pack                      the kept coordinates of every worker, contiguous, in
 *                                ascending k: the buffer "on the wire"   (Eq. 2, Section II-B)
 *   4. pair average              kept coordinates of a matched pair (i, j) both become
 *                                1/2 (a_i + a_j); all others stay a_i
 *                                                    (Algorithm 2 merge; GenerateW; Eq. 7)
 *   5. peer selection            the coordinator's bandwidth-aware matching
 *                                                    (Algorithm 3, GenerateGossipMatrix)
 *
 * The paper does not name the generator behind the mask.  This library defines it as a
 * counter-based hash of (seed, t, k) compared with keep_frac * 2^32 (see saps_round_key).
 *
 * Conventions
 *   - Every function returns an int status (0 = SAPS_OK, negative = error) unless stated;
 *     nothing throws, aborts or prints.
 *   - "device" pointers are CUDA device memory owned by the caller; the library neither
 *     allocates nor frees them.  "host" pointers are ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All device
 *     work is enqueued on it and the call returns without waiting.
 *   - Matrices are row-major fp32, row i = worker i, row stride `ld` elements (ld >= N).
 *     Elements k >= N of a row are never read or written.
 *   - n in [1, 64]; N in [1, 2^32 - 1]; t >= 1; keep_frac in [0, 1] (NaN rejected).
 *   - `pairs` (host, n entries): pairs[i] = peer of worker i, or i when it has none this
 *     round; it must be an involution (pairs[pairs[i]] == i).
 *   - fp32 arithmetic is IEEE round-to-nearest, one rounding per operation, never fused:
 *     a = x - fl(lr * g);  avg = fl(0.5f * fl(a_i + a_j)).  Subnormals are kept.
 *   - The context owns small device scratch areas, each allocated by the first call that
 *     needs it, on the device that is current then (so such a first call must not happen
 *     inside a stream capture): the status word and the tile states of the compaction scan
 *     (16 + 8 ceil(N/2048) bytes; saps_pack and every emitting entry point), the per-tile
 *     and per-group mask counts of the emitting round (about 8 ceil(N/2048) bytes), the partial sums of
 *     saps_consensus_distance (8 ceil(N/1024) bytes).  saps_round, saps_run_rounds,
 *     saps_mask, saps_unpack_avg* and saps_pack_noalloc allocate nothing.
 *   - Calls on one context must not overlap on the GPU (use one stream, or order streams
 *     with events): they share the scratch area.
 *   - Ordinary stream order is all a caller needs: work enqueued behind a call sees its results.
 *     One special case: the round kernels let a kernel that is launched behind them WITH the
 *     programmatic-stream-serialization launch attribute start early (consecutive rounds overlap
 *     at their edges that way).  A caller who launches own kernels with that attribute directly
 *     behind a round must, as always with that attribute, call cudaGridDependencySynchronize()
 *     in them before touching x or the wire buffers.  Kernels launched without it are unaffected.
 */
#ifndef SAPS_H_
#define SAPS_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SAPS_API __attribute__((visibility("default")))
#else
#define SAPS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define SAPS_OK            0
#define SAPS_ERR_INVALID  (-1)  /* bad argument; detected on the host before any launch   */
#define SAPS_ERR_PAIRS    (-2)  /* pairs is not an involution on 0..n-1                    */
#define SAPS_ERR_CUDA     (-3)  /* a CUDA runtime call failed (no device, launch error)    */
#define SAPS_ERR_OVERFLOW (-4)  /* more kept columns than the pack capacity (device-found) */
#define SAPS_ERR_TIMEOUT  (-5)  /* a bounded device-side wait ran out (device-found)       */
#define SAPS_ERR_NOMEM    (-6)  /* host or device allocation failed                        */
#define SAPS_ERR_TOO_LARGE (-7) /* N beyond the static scratch of saps_pack_noalloc        */

typedef struct saps_ctx saps_ctx;

/* ---- context ------------------------------------------------------------------------ */

/* Inputs of Algorithms 1-3: n workers, N parameters each, one library seed from which every
 * round's mask seed s is derived.  Row stride ld = N.  *out receives the context (host
 * object; no device work happens here). */
SAPS_API int saps_create(int n, uint64_t N, uint64_t seed, saps_ctx** out);

/* Same, with an explicit row stride ld >= N.  The round uses the widest access every row
 * start allows: 128-bit when ld % 4 == 0 and x, g are 16-byte aligned; 64-bit when ld % 2 == 0
 * and they are 8-byte aligned; scalar otherwise.  All three give the same bits. */
SAPS_API int saps_create_ld(int n, uint64_t N, uint64_t ld, uint64_t seed, saps_ctx** out);

/* Column sharding (one shard per GPU): this context's column 0 is column col_offset of the
 * whole model, so that every shard draws its part of the same round mask and a round needs
 * no exchange between shards.  col_offset + N <= 2^32.  out_idx then holds global columns. */
SAPS_API int saps_set_column_offset(saps_ctx* ctx, uint64_t col_offset);

/* Frees the context and its device scratch.  Pending work that uses it must have finished. */
SAPS_API int saps_destroy(saps_ctx* ctx);

/* ---- mask (Section II-B, Eq. 3; Algorithm 2, GenerateRandomMask) ---------------------- */

/* Host only.  The round key (k0, k1) replaces the coordinator's per-round random seed s
 * (Algorithm 1): a = mix(lo32(seed) ^ 0x243F6A88); a = mix(a ^ hi32(seed));
 * a = mix(a ^ lo32(t)); a = mix(a ^ hi32(t)); k0 = a; k1 = mix(a ^ 0x85A308D3), with
 * mix(v): v ^= v>>16; v *= 0x9E3779B9; v ^= v>>15; v *= 0x6A09E667; v ^= v>>16;
 *         v *= 0xBB67AE85; v ^= v>>15   (uint32, wrapping).
 * Column k is kept iff H(k) < threshold, where
 * H(k): v = k ^ k0; v ^= v>>16; v *= 0x9E3779B9; v ^= v>>15; v *= 0x6A09E667; v ^= k1;
 *       v ^= v>>16; v *= 0xBB67AE85; v ^= v>>15. */
SAPS_API void saps_round_key(uint64_t seed, uint64_t t, uint32_t* k0, uint32_t* k1);

/* Host only.  floor(keep_frac * 2^32) clamped to [0, 2^32]; 0 for NaN. */
SAPS_API uint64_t saps_threshold(double keep_frac);

/* Writes the round-t mask as a bitmap: bit (k & 31) of out_bits[k >> 5] is m_t[k]; bits at
 * and beyond N in the last word are zero.  out_bits: device, ceil(N/32) words. */
SAPS_API int saps_mask(saps_ctx* ctx, uint64_t t, double keep_frac, uint32_t* out_bits, void* stream);

/* ---- the round (Algorithm 2, SGD procedure and the mask / exchange / merge steps; Eq. 7) - */

/* One fused pass: SGD step, mask, pair average, in place on x.
 *   x      device [n, ld] fp32, updated in place
 *   g      device [n, ld] fp32 gradients, or NULL for a round without SGD step (then lr
 *          must be 0)
 *   pairs  host, n entries (see above); copied before the call returns
 * Reads x and g once and writes x once (12 bytes per worker-parameter). */
SAPS_API int saps_round(saps_ctx* ctx, float* x, const float* g, float lr, const int32_t* pairs,
               uint64_t t, double keep_frac, void* stream);

/* The same round that also emits the wire buffer of step 3 from the same pass: the packed
 * values are the post-SGD, pre-average a_i[k] (what worker i sends).  Outputs as saps_pack. */
SAPS_API int saps_round_pack(saps_ctx* ctx, float* x, const float* g, float lr, const int32_t* pairs,
                    uint64_t t, double keep_frac, float* out_vals, uint32_t* out_idx,
                    uint32_t* out_count, void* stream);

/* saps_round_pack with one destination per worker instead of one [n, cap] matrix (Algorithm 2,
 * ExchangeModelWithPeer, for workers spread over several GPUs): out_rows is a DEVICE array of n
 * pointers; worker i's packed values go to out_rows[i][0 .. count) (room for cap floats), and a
 * NULL entry means worker i's values are not wanted.  A destination may be any address this GPU
 * can store to: with peer access enabled, the receive buffer of the worker's peer on another GPU;
 * the kernel then writes the wire buffer straight into the receiver's memory with ordinary
 * stores while the same pass streams the model, and no separate transfer follows.  The receiver
 * may read it once this call's stream work has completed and that fact has reached it (a stream
 * synchronisation on this side followed by a host-side barrier, or an interprocess event).
 * out_idx, out_count as in saps_round_pack (local device memory).  The table is read by the
 * kernel: keep it unchanged until the call's stream work has completed. */
SAPS_API int saps_round_pack_rows(saps_ctx* ctx, float* x, const float* g, float lr,
                                  const int32_t* pairs, uint64_t t, double keep_frac,
                                  float* const* out_rows, uint32_t* out_idx, uint32_t* out_count,
                                  void* stream);

/* The emitting entry points need the number of kept columns per column tile before the fused
 * kernel runs (a block derives the ranks of its kept columns from the counts of all earlier
 * tiles).  By default that kernel also counts them for round t+1 while it streams round t (the
 * mask does not depend on the data, and the integer units are not the bottleneck of a
 * memory-bound kernel), so a following call for round t+1 with the same keep_frac is a single
 * kernel launch.  Any other call first counts in a small kernel of its own.
 * Results are identical either way; enabled = 0 switches the run-ahead off.
 * The counts are kept in the context and read by the next call's kernels, so consecutive
 * emitting calls on one context must run on one stream or be ordered by events (the general
 * rule above that calls on one context must not overlap covers it).  To capture a sequence of
 * emitting calls in a CUDA graph, call saps_set_run_ahead(ctx, 1) right before the capture: that
 * forgets counts taken by earlier kernels, so the first captured round counts its own mask inside
 * the graph and every replay is self-contained (make the context's first use before, outside
 * the capture, since it allocates). */
SAPS_API int saps_set_run_ahead(saps_ctx* ctx, int enabled);

/* Order of the two halves of the update.
 *   SAPS_ORDER_SGD_FIRST     Algorithm 2 (default): a = x - lr g, then the kept coordinates of
 *                            a matched pair become the mean of the two a's.
 *   SAPS_ORDER_GOSSIP_FIRST  Eq. 7, the form the convergence analysis uses:
 *                            X' = X o not M + (X o M) W - lr G(X): the kept coordinates of the
 *                            CURRENT models are averaged, then each worker subtracts its own
 *                            gradient step.  The emitted wire buffer then holds x (not a).
 * A per-round learning rate (gamma_t of Eq. 7) is simply the lr argument of each call. */
#define SAPS_ORDER_SGD_FIRST    0
#define SAPS_ORDER_GOSSIP_FIRST 1
SAPS_API int saps_set_update_order(saps_ctx* ctx, int order);

/* How the fused round moves its row pieces when rows allow 128-bit accesses and there is a
 * gradient.  SAPS_STAGING_BULK: bulk asynchronous copies global -> shared memory (completion on
 * an mbarrier, bounded wait), results back by bulk copies shared -> global; the fastest form for
 * models that stream from HBM.  SAPS_STAGING_REGISTERS: vector loads and stores from registers;
 * the better form for models that stay in L2 and the only one for other row alignments.
 * SAPS_STAGING_AUTO (default) chooses by the size of the launch.  Results are bit-identical. */
#define SAPS_STAGING_AUTO      0
#define SAPS_STAGING_REGISTERS 1
#define SAPS_STAGING_BULK      2
SAPS_API int saps_set_staging(saps_ctx* ctx, int staging);

/* ---- pack (Eq. 2; "sends the non-zero elements", Section II-B) -------------------------- */

/* Slots per worker that out_vals / out_idx must hold for this keep_frac:
 * min(N, round_up_32(ceil(N p + 8 sqrt(N p (1-p))) + 64)) with p = threshold / 2^32.
 * Returns 0 for a NULL context or an invalid keep_frac. */
SAPS_API uint64_t saps_pack_capacity(const saps_ctx* ctx, double keep_frac);

/* Fixes the capacity to `cap` slots (clamped to N) for every keep_frac, e.g. to a wire
 * buffer of a given size; 0 restores the formula above.  The paper's "less than N/c" is
 * loose: the count is Binomial(N, 1/c), so a hard cap can overflow (SAPS_ERR_OVERFLOW). */
SAPS_API int saps_set_pack_capacity(saps_ctx* ctx, uint64_t cap);

/* Compacts the kept columns of x (as it is now) for every worker.
 *   out_vals   device [n, cap] fp32, row stride cap = saps_pack_capacity(ctx, keep_frac):
 *              out_vals[i*cap + r] = x[i][idx[r]]
 *   out_idx    device [cap] uint32 or NULL: the kept columns in ascending order (one list,
 *              the mask being the same for every worker)
 *   out_count  device, one uint32: the number of kept columns
 * Selection is by mask position, not by value: a kept coordinate equal to 0.0 is sent.
 * If count > cap, writes stop at cap, out_count still holds the true count and the status
 * word is set to SAPS_ERR_OVERFLOW.  Slots r >= count are not written. */
SAPS_API int saps_pack(saps_ctx* ctx, const float* x, uint64_t t, double keep_frac, float* out_vals,
              uint32_t* out_idx, uint32_t* out_count, void* stream);

/* Receiving side of the exchange (Algorithm 2: ExchangeModelWithPeer and the merge), for a
 * deployment where the packed buffers really travel: every worker i averages its kept
 * coordinates with the buffer it received,
 *     x[i][idx[r]] = 1/2 (x[i][idx[r]] + recv_vals[src(i)][r]),  r < *count,
 * where src(i) = pairs[i] when pairs (host, n entries) is given - recv_vals is then simply
 * the senders' buffer [n, cap] as saps_pack wrote it, and a worker without a peer is left
 * alone - or src(i) = i when pairs is NULL (recv_vals already holds, in row i, what worker i
 * received).  idx, count: device, as written by saps_pack; cap = saps_pack_capacity(ctx,
 * keep_frac).  SGD-only round + saps_pack + saps_unpack_avg equals saps_round bit for bit. */
SAPS_API int saps_unpack_avg(saps_ctx* ctx, float* x, const float* recv_vals, const uint32_t* idx,
                             const uint32_t* count, double keep_frac, const int32_t* pairs,
                             void* stream);

/* The same with an explicit map: worker i averages with row src_rows[i] of recv_vals
 * (0 <= src_rows[i] < n), or is left alone when src_rows[i] == -1.  This is the form a
 * row-sharded deployment needs (the workers of one job spread over several GPUs: only the
 * rows whose peer lives elsewhere receive a buffer).  src_rows: host, n entries. */
SAPS_API int saps_unpack_avg_rows(saps_ctx* ctx, float* x, const float* recv_vals, const uint32_t* idx,
                                  const uint32_t* count, double keep_frac, const int32_t* src_rows,
                                  void* stream);

/* saps_pack for callers that must not allocate device memory.  (The paper has no counterpart:
 * this entry point exists for integration only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a serving or training
 * process whose framework has already claimed the whole GPU for its own memory pool, a
 * latency-critical loop that cannot afford the device-wide synchronisation an allocation
 * implies, or a plug-in that is only handed buffers and a stream.  saps_pack would allocate
 * the context's scratch area on its first use; this variant never does: it calls neither
 * cudaMalloc nor cudaFree nor any library routine that does.
 *
 * Instead the tile states of the compaction scan live in a fixed array inside the library
 * image (524,304 bytes).  The CUDA runtime creates that array on a GPU when it loads the
 * library's device code there (at the latest on the first launch of one of its kernels on
 * that GPU), not on demand from this call, and keeps it until the process exits.  That array
 * covers N <= SAPS_NOALLOC_MAX_N columns; a larger context is refused with SAPS_ERR_TOO_LARGE
 * before anything is launched.
 *
 * Arguments and results are those of saps_pack (same capacity rule, same overflow
 * behaviour), plus
 *   out_status  device, one int, or NULL: receives SAPS_OK, SAPS_ERR_OVERFLOW or
 *               SAPS_ERR_TIMEOUT for this call (saps_status does not cover this entry point).
 *
 * The first call on each device looks up the array's device address (once per device, with
 * that device current); make that first call outside any stream capture.  All calls, from
 * all contexts, share the one array: it is cleared at the start of every call, and two
 * calls that overlap on the same GPU (different streams, no ordering) race and give
 * undefined results.  Calls on one stream, or ordered by events, are safe. */
#define SAPS_NOALLOC_MAX_N 134217728ull
SAPS_API int saps_pack_noalloc(saps_ctx* ctx, const float* x, uint64_t t, double keep_frac,
                               float* out_vals, uint32_t* out_idx, uint32_t* out_count,
                               int* out_status, void* stream);

/* ---- peer selection (Algorithm 3; GetNewConnectedGraph of Algorithm 1) -------------------- */

/* b_thres: links with min(B_ij, B_ji) >= b_thres form B*.  NaN selects the default, the
 * median of the symmetrised off-diagonal bandwidths of each call's matrix.  +INFINITY selects,
 * per call, the largest threshold for which B* still lets as many workers pair up as the
 * link graph allows, so that the first matching maximises the slowest chosen link (the
 * bandwidth utilisation measured in Section IV-D).
 * t_thres: an edge is "recently connected" iff R_ij > t - t_thres.  0 selects the default
 * max(2, 2 ceil(log2 n)). */
SAPS_API int saps_set_select_params(saps_ctx* ctx, double b_thres, int t_thres);

/* Host only; no device needed.  One run of GenerateGossipMatrix for round t:
 *   bandwidth  host n x n row-major doubles (symmetrised by min inside; diagonal ignored;
 *              0 = no link)
 *   out_pairs  host n entries: the matching as an involution (out_pairs[i] == i only when
 *              worker i could not be matched: odd n or missing links)
 * Records the chosen pairs in the context's timestamp matrix R.  t must not decrease
 * between calls (SAPS_ERR_INVALID).  Any maximum matching of the candidate edges is a
 * valid answer; which one is returned depends on (seed, t) only.
 * Round numbers are kept as signed 64-bit timestamps: 1 <= t <= SAPS_SELECT_MAX_T, else
 * SAPS_ERR_INVALID (the same limit holds for the rounds of saps_run_rounds* when they select
 * peers, and for last_t and the entries of R given to saps_set_select_state). */
#define SAPS_SELECT_MAX_T ((1ull << 62) - 1)
SAPS_API int saps_select_peers(saps_ctx* ctx, const double* bandwidth, uint64_t t, int32_t* out_pairs);

/* Forgets every recorded exchange (R = "never") and the last t. */
SAPS_API int saps_select_reset(saps_ctx* ctx);

/* Checkpoint / resume of the selection state: R is n x n int64 row-major, INT64_MIN-like
 * SAPS_NEVER marks "never".  Either pointer may be NULL. */
#define SAPS_NEVER (-(1LL << 62))
SAPS_API int saps_get_select_state(const saps_ctx* ctx, int64_t* out_R, uint64_t* out_last_t);
SAPS_API int saps_set_select_state(saps_ctx* ctx, const int64_t* R, uint64_t last_t);

/* ---- round scheduler (Algorithm 1, the coordinator's loop) --------------------------------- */

/* Enqueues rounds t_first .. t_first + T - 1 on `stream` without any host-device
 * synchronisation in between.  The matching of each round is
 *   pairs_list != NULL : pairs_list[r*n .. r*n+n-1] (host, T x n), else
 *   bandwidth  != NULL : saps_select_peers(ctx, bandwidth, t) (runs on the host ahead of
 *                        the GPU; it never depends on device data).
 * out_pairs_log (host, T x n) receives the matchings used, or may be NULL.
 * lr_list (host, T floats) gives a learning rate per round (gamma_t), or NULL to use lr. */
SAPS_API int saps_run_rounds(saps_ctx* ctx, float* x, const float* g, float lr, uint64_t t_first,
                    uint64_t T, double keep_frac, const float* lr_list, const int32_t* pairs_list,
                    const double* bandwidth, int32_t* out_pairs_log, void* stream);

/* The same loop with the wire buffer of every round (as saps_round_pack): round r writes its
 * packed values to out_vals [n, cap] and its kept columns to out_idx [cap] (may be NULL), each
 * round over the previous one, and its count to out_counts[r] (device, T words).  After the
 * call the buffers hold the last round's wire data and out_counts the traffic of every round
 * (Table 1: a worker moves 2 count values per round). */
SAPS_API int saps_run_rounds_pack(saps_ctx* ctx, float* x, const float* g, float lr, uint64_t t_first,
                                  uint64_t T, double keep_frac, const float* lr_list,
                                  const int32_t* pairs_list, const double* bandwidth,
                                  int32_t* out_pairs_log, float* out_vals, uint32_t* out_idx,
                                  uint32_t* out_counts, void* stream);

/* ---- host-buffer entry point ----------------------------------------------------------------- */

/* One round on HOST matrices: copies x_host and g_host ([n, N] fp32, row stride N; pinned
 * memory recommended) to the device staging buffers, runs the round, copies x back, all in
 * column chunks pipelined over internal streams, and waits for completion.
 *   d_x, d_g  device staging, [n, ld] fp32 with the context's row stride ld (create the
 *             context with saps_create_ld and ld a multiple of 32 for 128-bit accesses);
 *             caller-owned.  g_host may be NULL (then lr = 0, d_g unused).
 * The first call creates the internal streams and events (not inside a stream capture). */
SAPS_API int saps_round_host(saps_ctx* ctx, float* x_host, const float* g_host, float lr,
                    const int32_t* pairs, uint64_t t, double keep_frac, float* d_x, float* d_g);

/* In both host-buffer entry points x_host may be NULL: the model then stays resident in d_x
 * from call to call (as in training, where the weights live on the GPU) and only the
 * gradients travel in and, for saps_round_pack_host, the wire buffer travels out. */

/* The same with the wire buffer of step 3 (as saps_round_pack): out_vals_host [n, cap],
 * out_idx_host [cap] or NULL, out_count_host (one word) are HOST buffers filled before the
 * call returns; d_vals [n, cap], d_idx [cap], d_count are device staging (d_idx may be NULL
 * when out_idx_host is).  cap = saps_pack_capacity(ctx, keep_frac). */
SAPS_API int saps_round_pack_host(saps_ctx* ctx, float* x_host, const float* g_host, float lr,
                                  const int32_t* pairs, uint64_t t, double keep_frac, float* d_x,
                                  float* d_g, float* out_vals_host, uint32_t* out_idx_host,
                                  uint32_t* out_count_host, float* d_vals, uint32_t* d_idx,
                                  uint32_t* d_count);

/* Tuning of the copy/compute pipeline behind the two host-buffer entry points: columns per
 * chunk (rounded up to whole 2048-column tiles; default 1,048,576; the last chunks of a row halve
 * down to 65,536 columns, so that little is left to do once the last copy-in has landed) and the
 * number of streams that copy chunks in and run the round on them (1..6, default 3; results
 * always leave on one further stream).  0 leaves a setting as it is.  Results do not depend on either. */
SAPS_API int saps_set_host_pipeline(saps_ctx* ctx, uint64_t chunk_columns, int lanes);

/* ---- consensus and communication metrics -------------------------------------------------------- */

/* Consensus distance of Theorem 1 / Lemma 2: *out = || X - Xbar 1^T ||_F^2, the sum over all
 * coordinates of the squared deviations of the n workers from their mean, accumulated in
 * fp64 in a fixed order (the result is reproducible).  x: device [n, ld]; out: device, one
 * double.  Reads x once: every block of 1024 columns leaves a partial sum, and a one-block kernel,
 * launched so that it is already in place when the first one ends, adds them up.  The first call
 * allocates ceil(N/1024) doubles. */
SAPS_API int saps_consensus_distance(saps_ctx* ctx, const float* x, double* out, void* stream);

/* Host only.  Communication figures of one round (Table 1; the bandwidth utilisation of
 * Section IV-D is the bottleneck bandwidth of the chosen pairs): out5[0] = values a matched
 * worker sends + receives (2 count), out5[1] = the same in bytes, out5[2] = smallest and
 * out5[3] = mean symmetrised bandwidth over the chosen pairs, out5[4] = time in seconds to
 * move one buffer over the slowest chosen link, 32 count / (out5[2] * bits_per_s_per_unit)
 * (bits_per_s_per_unit = 1e6 when the matrix is in Mb/s). */
SAPS_API int saps_comm_stats(const saps_ctx* ctx, const double* bandwidth, const int32_t* pairs,
                             uint64_t count, double bits_per_s_per_unit, double* out5);

/* ---- measurement ------------------------------------------------------------------------------- */

/* Optional cudaEvent_t pair (as void*; NULL, NULL switches it off).  When set, saps_round
 * and saps_round_pack record `before` just ahead of the fused round kernel and `after`
 * just behind it, on the call's stream, so that a benchmark can time that one kernel inside
 * a longer step.  The events stay owned by the caller. */
SAPS_API int saps_set_timing_events(saps_ctx* ctx, void* before, void* after);

/* Test hook for the bounded wait of the compaction scan: look-back tile `skip_tile` never
 * publishes its state, so its successors run out of polls after `spin_limit` tries (0 = the
 * default budget) and the kernel ends with SAPS_ERR_TIMEOUT in the status word instead of
 * hanging.  skip_tile = 0xFFFFFFFF switches the hook off.  Nothing faults or traps. */
SAPS_API int saps_debug_inject(saps_ctx* ctx, uint32_t skip_tile, uint32_t spin_limit);

/* Test hook for the bounded wait of the staged form of the fused round (SAPS_STAGING_BULK):
 * with give_up != 0 every block treats the wait for its bulk copies as run out.  Its threads
 * then load their vectors straight from global memory and store their results themselves (same
 * bits), the block still waits, bounded, for its copies to land before it ends, and the status
 * word receives SAPS_ERR_TIMEOUT when the context has its scratch (any earlier saps_pack or
 * emitting call creates it).  Every access stays in bounds; nothing faults, traps or hangs. */
SAPS_API int saps_debug_staging_wait(saps_ctx* ctx, int give_up);

/* ---- errors ----------------------------------------------------------------------------------- */

/* Waits for `stream`, then returns in *out_device_status the first error a kernel of this
 * context recorded since the last call (SAPS_OK, SAPS_ERR_OVERFLOW or SAPS_ERR_TIMEOUT)
 * and clears it. */
SAPS_API int saps_status(saps_ctx* ctx, void* stream, int* out_device_status);

/* Static string for a status code. */
SAPS_API const char* saps_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SAPS_H_ */
