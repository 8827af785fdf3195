// Counter-based mask hash: the stand-in for the unnamed generator behind the
// Bernoulli mask of Section II-B (Eq. 3).  Pure 32-bit wrapping arithmetic.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define SAPS_HD __host__ __device__ __forceinline__
#else
#define SAPS_HD inline
#endif

namespace saps {

constexpr uint32_t kMul1 = 0x9E3779B9u;
constexpr uint32_t kMul2 = 0x6A09E667u;
constexpr uint32_t kMul3 = 0xBB67AE85u;
constexpr uint32_t kSeedPad = 0x243F6A88u;
constexpr uint32_t kKeyPad = 0x85A308D3u;

SAPS_HD uint32_t mix32(uint32_t v)
{
    v ^= v >> 16; v *= kMul1;
    v ^= v >> 15; v *= kMul2;
    v ^= v >> 16; v *= kMul3;
    v ^= v >> 15;
    return v;
}

// Key of round t: what the coordinator would broadcast as the seed s (Algorithm 1).
// k0f and k1f are the key words folded with their own upper halves, k ^ (k >> 16): the hash
// xors a key word into v and then applies v ^= v >> 16, which equals xoring the folded word
// into v ^ (v >> 16), one operation less per column.
struct RoundKey {
    uint32_t k0f, k1f;
    uint32_t thr32;   // low 32 bits of the threshold
    uint32_t all;     // 1 when the threshold is 2^32 (every column kept)
};

SAPS_HD uint32_t fold16(uint32_t w) { return w ^ (w >> 16); }

// H(k): v = k ^ k0; v ^= v >> 16; v *= M1; v ^= v >> 15; v *= M2; v ^= k1; v ^= v >> 16;
//       v *= M3; v ^= v >> 15, written with the folded key words.
SAPS_HD uint32_t column_hash(uint32_t k, uint32_t k0f, uint32_t k1f)
{
    uint32_t v = k ^ (k >> 16) ^ k0f;
    v *= kMul1;
    v ^= v >> 15; v *= kMul2;
    v = v ^ (v >> 16) ^ k1f;
    v *= kMul3;
    v ^= v >> 15;
    return v;
}

SAPS_HD bool column_kept(uint32_t k, const RoundKey& key)
{
    return (column_hash(k, key.k0f, key.k1f) < key.thr32) | (key.all != 0);
}

}  // namespace saps
