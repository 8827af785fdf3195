"""Regenerates tests/golden/mask_hash.txt from the CPU oracle alone (it imports nothing else).

    python tests/golden/make_mask_golden.py > tests/golden/mask_hash.txt

The numbers in the committed file were first obtained by evaluating the written definition of
the hash by hand-driven integer arithmetic, outside both implementations; this script
reproduces them from oracle/ and is what any later regeneration must use.
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

import numpy as np  # noqa: E402

import oracle  # noqa: E402

HEADER = '''# Golden values of the mask hash (the counter-based stand-in for the unnamed
# generator of Section II-B / Eq. 3).  They were evaluated once, by hand-driven
# integer arithmetic outside both implementations, from the written definition
#   mix(v):  v^=v>>16; v*=0x9E3779B9; v^=v>>15; v*=0x6A09E667; v^=v>>16; v*=0xBB67AE85; v^=v>>15
#   key(seed,t): a=mix(lo(seed)^0x243F6A88); a=mix(a^hi(seed)); a=mix(a^lo(t)); a=mix(a^hi(t));
#                k0=a; k1=mix(a^0x85A308D3)
#   H(k): v=k^k0; v^=v>>16; v*=M1; v^=v>>15; v*=M2; v^=k1; v^=v>>16; v*=M3; v^=v>>15
# and both the CPU oracle and the CUDA library must reproduce them.
#'''

KEYS = [("0x0", 1), ("0x0", 2), ("0x1", 1), ("0x2", 20), ("0xDEADBEEFCAFEF00D", 4294967301)]
COLUMNS = [0, 1, 2, 3, 65535, 272473, 14728265, 124439807, 4294967295]
COUNTS = [(0, 1, 65536, "0.1"), (0, 2, 65536, "0.1"), (0, 3, 65536, "0.1"), (1, 1, 272474, "0.01"),
          (0, 1, 14728266, "0.01"), (0, 1, 14728266, "0.001"), (2, 1, 25557032, "0.1"),
          (2, 1, 25557032, "0.03"), (2, 1, 25557032, "0.01"), (2, 1, 25557032, "0.003"),
          (2, 1, 25557032, "0.001"), (0, 1, 124439808, "0.01")]
FIRST = [(0, 1, 8), (0, 2, 4), (0, 3, 4)]


def main():
    out = [HEADER, "# mix  <v> <mix(v)>"]
    for v in (0, 1, 0xFFFFFFFF):
        out.append(f"mix 0x{v:08x} 0x{oracle.mix(v):08x}")
    out.append("# key  <seed> <t> <k0> <k1>")
    for seed, t in KEYS:
        k0, k1 = oracle.round_key(int(seed, 0), t)
        out.append(f"key {seed} {t} 0x{k0:08x} 0x{k1:08x}")
    out.append("# hash <seed> <t> <k> <H(k)>")
    for seed, t in KEYS:
        k0, k1 = oracle.round_key(int(seed, 0), t)
        cols = COLUMNS[:4] + ([4, 5, 6, 7] if (seed, t) == ("0x0", 1) else []) + COLUMNS[4:]
        for k in cols:
            out.append(f"hash {seed} {t} {k} 0x{oracle.hash_k(k, k0, k1):08x}")
    out.append("# thr <keep_frac> <floor(keep_frac * 2^32) clamped to [0, 2^32]>")
    for p in ("1.0", "0.1", "0.03", "0.01", "0.003", "0.001", "0.0"):
        out.append(f"thr {p} {oracle.threshold(float(p))}")
    out.append("# count <seed> <t> <N> <keep_frac> <number of kept columns>")
    for seed, t, N, p in COUNTS:
        out.append(f"count {seed} {t} {N} {p} {int(oracle.mask(seed, t, float(p), N).sum(dtype=np.int64))}")
    out.append("# first <seed> <t> <N> <keep_frac> <the first kept columns ...>")
    masks = {t: np.nonzero(oracle.mask(seed, t, 0.1, 65536))[0] for seed, t, _ in FIRST}
    for seed, t, k in FIRST:
        out.append(f"first {seed} {t} 65536 0.1 " + " ".join(str(int(v)) for v in masks[t][:k]))
    out.append("# last <seed> <t> <N> <keep_frac> <the last kept column>")
    for seed, t, _ in FIRST:
        out.append(f"last {seed} {t} 65536 0.1 {int(masks[t][-1])}")
    print("\n".join(out))


if __name__ == "__main__":
    main()
