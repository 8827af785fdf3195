"""Helpers for the GPU parity tests: device buffers with canaries, oracle-side mirrors."""
from __future__ import annotations

import numpy as np

CANARY = np.float32(-7.25e33)


def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch


def round_up(v, m):
    return (v + m - 1) // m * m


class DeviceMatrix:
    """[n, N] fp32 on the GPU inside a larger allocation: row stride ld, `lead` floats before
    the first row (to shift the alignment), canary values everywhere outside the matrix."""

    def __init__(self, host: np.ndarray, ld: int | None = None, lead: int = 0):
        torch = torch_cuda()
        n, N = host.shape
        self.n, self.N = n, N
        self.ld = N if ld is None else ld
        self.lead = lead
        total = lead + n * self.ld + 64
        self.buf = torch.full((total,), float(CANARY), dtype=torch.float32, device="cuda")
        self.view = self.buf[lead:lead + n * self.ld].view(n, self.ld)
        self.view[:, :N].copy_(torch.from_numpy(host))

    @property
    def ptr(self):
        return self.buf.data_ptr() + 4 * self.lead

    def host(self) -> np.ndarray:
        return self.view[:, :self.N].cpu().numpy()

    def canaries_intact(self) -> bool:
        buf = self.buf.cpu().numpy()
        inside = np.zeros(buf.shape, dtype=bool)
        for i in range(self.n):
            s = self.lead + i * self.ld
            inside[s:s + self.N] = True
        return bool((buf[~inside] == CANARY).all())


def bits_from_mask(m: np.ndarray) -> np.ndarray:
    """uint8 0/1 vector -> little-endian 32-bit words, zero padded."""
    N = m.shape[0]
    padded = np.zeros(round_up(N, 32), dtype=np.uint8)
    padded[:N] = m
    return np.packbits(padded.reshape(-1, 32), axis=1, bitorder="little").view("<u4").ravel()


def assert_bits_equal(got: np.ndarray, want: np.ndarray, what: str = ""):
    g, w = got.view(np.uint32), want.view(np.uint32)
    if not (g == w).all():
        bad = np.argwhere(g != w)
        first = tuple(int(v) for v in bad[0])
        raise AssertionError(f"{what}: {len(bad)} of {g.size} words differ, first at {first}: "
                             f"{got[first]!r} != {want[first]!r}")


def force_staging(monkeypatch, mode: str) -> None:
    """Make every context created through the binding use the given staging of the fused round
    ("auto" leaves the default).  Small test sizes would otherwise never reach the bulk-copy form,
    which the library only picks for launches of several thousand blocks."""
    if mode == "auto":
        return
    from paper_2002_09692_b200 import binding
    value = {"registers": binding.SAPS_STAGING_REGISTERS, "bulk": binding.SAPS_STAGING_BULK}[mode]
    for name in ("saps_create", "saps_create_ld"):
        original = getattr(binding, name)

        def wrapped(*args, _original=original):
            ctx = _original(*args)
            binding.saps_set_staging(ctx, value)
            return ctx

        monkeypatch.setattr(binding, name, wrapped)
