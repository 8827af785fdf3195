/*
 * CPU oracle for one SAPS-PSGD gossip round.  TEST INFRASTRUCTURE ONLY: it is
 * called by the test-suite, by the smoke check and by the benchmark's CPU
 * baseline leg, never by the product path, and it shares no code with the CUDA
 * library.
 *
 * Plain single-threaded C.  Every fp32 operation is rounded on its own: build
 * with -ffp-contract=off and without -ffast-math so that no multiply-add is
 * fused and subnormals are kept.
 *
 * What it follows
 *   - worker loop of Algorithm 2 (SGD step, mask, sparsify, exchange, merge);
 *   - Section II-B, Eq. 2 (x~ = x o m) and Eq. 3 (Bernoulli(p = 1/c) mask that
 *     is the same on every worker in a round);
 *   - GenerateW of Algorithm 3 (weights 1/2 on a matched pair and on its
 *     diagonal) together with Eq. 7, which make the merge an average.
 *
 * Readings taken where the paper is silent or at odds with itself
 *   - The merge line of Algorithm 2 prints a replacement; the prose of
 *     Section II-A says "averages", GenerateW puts 1/2 on both entries and
 *     Eq. 7 multiplies by W.  The oracle averages.
 *   - Order: Algorithm 2's (SGD first, then exchange the updated model).
 *   - The paper does not name the random generator behind the mask.  Here the
 *     mask is a counter-based hash of (seed, t, k) compared with
 *     keep_frac * 2^32; this is a stated substitution.
 *   - "Send the non-zero elements": packing goes by mask position, not by
 *     value, so a kept coordinate that is exactly 0.0 is still sent.
 *
 * Parity pins: see tests/test_oracle_*.py (golden hash values, the worked
 * 4x8 example, dense W*X product, axpy, hypercube consensus, Lemma 1,
 * Lemma 2 contraction factor, binomial density).
 */
#include <stddef.h>
#include <stdint.h>
#include <math.h>

/* ---- mask hash (defined here, not by the paper; arithmetic wraps mod 2^32) -- */

#define ORC_M1 0x9E3779B9u
#define ORC_M2 0x6A09E667u
#define ORC_M3 0xBB67AE85u
#define ORC_P0 0x243F6A88u
#define ORC_P1 0x85A308D3u

uint32_t orc_mix(uint32_t v)
{
    v ^= v >> 16;
    v *= ORC_M1;
    v ^= v >> 15;
    v *= ORC_M2;
    v ^= v >> 16;
    v *= ORC_M3;
    v ^= v >> 15;
    return v;
}

/* Round key: the coordinator's per-round seed s of Algorithm 1 is replaced by
 * a pure function of one library seed and the round counter t. */
void orc_round_key(uint64_t seed, uint64_t t, uint32_t *k0, uint32_t *k1)
{
    uint32_t a;
    a = orc_mix((uint32_t)(seed & 0xFFFFFFFFu) ^ ORC_P0);
    a = orc_mix(a ^ (uint32_t)(seed >> 32));
    a = orc_mix(a ^ (uint32_t)(t & 0xFFFFFFFFu));
    a = orc_mix(a ^ (uint32_t)(t >> 32));
    *k0 = a;
    *k1 = orc_mix(a ^ ORC_P1);
}

uint32_t orc_hash(uint32_t k, uint32_t k0, uint32_t k1)
{
    uint32_t v = k ^ k0;
    v ^= v >> 16;
    v *= ORC_M1;
    v ^= v >> 15;
    v *= ORC_M2;
    v ^= k1;
    v ^= v >> 16;
    v *= ORC_M3;
    v ^= v >> 15;
    return v;
}

/* keep_frac -> integer threshold in [0, 2^32]; coordinate k is kept iff
 * hash(k) < threshold.  (Eq. 3 with p = keep_frac.) */
uint64_t orc_threshold(double keep_frac)
{
    double s = floor(keep_frac * 4294967296.0);
    if (!(s > 0.0))
        return 0;
    if (s >= 4294967296.0)
        return 4294967296ull;
    return (uint64_t)s;
}

/* m[k] in {0,1} for k = 0..N-1: GenerateRandomMask of Algorithm 2, Eq. 3. */
void orc_mask(uint64_t seed, uint64_t t, double keep_frac, uint64_t N, uint8_t *m)
{
    uint32_t k0, k1;
    uint64_t thr = orc_threshold(keep_frac);
    orc_round_key(seed, t, &k0, &k1);
    for (uint64_t k = 0; k < N; ++k)
        m[k] = ((uint64_t)orc_hash((uint32_t)k, k0, k1) < thr) ? 1 : 0;
}

/* ---- the round ----------------------------------------------------------- */

/* SGD procedure of Algorithm 2: x = x - lr * g, every worker, every
 * coordinate.  x and g are [n, N] row-major (row = worker).  g == NULL means
 * "no gradient" (pure gossip) and leaves x as it is. */
void orc_sgd(int n, uint64_t N, float *x, const float *g, float lr)
{
    if (!g)
        return;
    for (int i = 0; i < n; ++i)
        for (uint64_t k = 0; k < N; ++k) {
            float step = lr * g[(size_t)i * N + k];
            x[(size_t)i * N + k] = x[(size_t)i * N + k] - step;
        }
}

/* Sparsify and "send": x~ = x o m (Eq. 2); the wire buffer holds the kept
 * coordinates in ascending order of k.  idx[r] = r-th kept column (one list
 * for all workers, the mask being the same for all), vals[i*cap + r] =
 * a[i][idx[r]].  Entries with r >= cap are not written; the return value is
 * the full number of kept columns. */
uint64_t orc_pack(int n, uint64_t N, const float *a, const uint8_t *m, uint64_t cap,
                  float *vals, uint32_t *idx)
{
    uint64_t r = 0;
    for (uint64_t k = 0; k < N; ++k) {
        if (!m[k])
            continue;
        if (r < cap) {
            if (idx)
                idx[r] = (uint32_t)k;
            if (vals)
                for (int i = 0; i < n; ++i)
                    vals[(size_t)i * cap + r] = a[(size_t)i * N + k];
        }
        ++r;
    }
    return r;
}

/* Exchange + merge: for each matched pair (i, j = pairs[i]) and each kept k,
 * both workers end with 1/2 (a_i[k] + a_j[k]); everything else is untouched
 * (the "o not m" term).  pairs[i] == i means worker i has no peer this round. */
void orc_pair_average(int n, uint64_t N, float *a, const int32_t *pairs, const uint8_t *m)
{
    for (int i = 0; i < n; ++i) {
        int j = pairs[i];
        if (j <= i)
            continue;
        for (uint64_t k = 0; k < N; ++k) {
            if (!m[k])
                continue;
            float s = a[(size_t)i * N + k] + a[(size_t)j * N + k];
            float v = 0.5f * s;
            a[(size_t)i * N + k] = v;
            a[(size_t)j * N + k] = v;
        }
    }
}

/* One whole round in Algorithm 2's order.  m is caller-provided scratch of N
 * bytes and holds the round's mask on return. */
void orc_round(int n, uint64_t N, float *x, const float *g, float lr, const int32_t *pairs,
               uint64_t seed, uint64_t t, double keep_frac, uint8_t *m)
{
    orc_sgd(n, N, x, g, lr);
    orc_mask(seed, t, keep_frac, N, m);
    orc_pair_average(n, N, x, pairs, m);
}

/* ---- variants and companions of the round ------------------------------------ */

/* The update in the order of Eq. 7 (the form the convergence analysis uses):
 * X_{t+1} = X_t o not M_t + (X_t o M_t) W_t - gamma G(X_t).  The kept coordinates of the
 * CURRENT models are averaged first, then every worker subtracts its own gradient step. */
void orc_round_eq7(int n, uint64_t N, float *x, const float *g, float lr, const int32_t *pairs,
                   uint64_t seed, uint64_t t, double keep_frac, uint8_t *m)
{
    orc_mask(seed, t, keep_frac, N, m);
    orc_pair_average(n, N, x, pairs, m);
    orc_sgd(n, N, x, g, lr);
}

/* Receiving side of the exchange (Algorithm 2, merge): worker i holds its own model x_i and
 * the buffer recv[i*cap + r] it received, whose r-th entry belongs to column idx[r]; the kept
 * coordinates become the mean of the local and the received value. */
void orc_unpack_avg(int n, uint64_t N, float *x, const float *recv, uint64_t cap,
                    const uint32_t *idx, uint64_t count)
{
    for (int i = 0; i < n; ++i)
        for (uint64_t r = 0; r < count && r < cap; ++r) {
            float s = x[(size_t)i * N + idx[r]] + recv[(size_t)i * cap + r];
            x[(size_t)i * N + idx[r]] = 0.5f * s;
        }
}

/* Consensus distance of Theorem 1 / Lemma 2: || X - Xbar 1^T ||_F^2, the sum over all
 * coordinates of the squared deviations of the n workers from their mean.  fp64. */
double orc_consensus_distance(int n, uint64_t N, const float *x)
{
    double total = 0.0;
    for (uint64_t k = 0; k < N; ++k) {
        double mean = 0.0;
        for (int i = 0; i < n; ++i)
            mean += (double)x[(size_t)i * N + k];
        mean /= (double)n;
        for (int i = 0; i < n; ++i) {
            double d = (double)x[(size_t)i * N + k] - mean;
            total += d * d;
        }
    }
    return total;
}
