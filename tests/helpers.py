"""Shared helpers of the GPU parity tests: move seeded inputs to the device, run the
oracle on the same values, compare."""
import numpy as np
import torch

from oracle import quantizers as OQ
from oracle.quantizers import QParams as OQP
from paper_2506_04985_b200 import synth

DEV = "cuda"


def dev(t):
    return t.to(DEV) if isinstance(t, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(t)).to(DEV)


def host(t):
    return t.detach().cpu().numpy()


def bf16_host(t):
    """device bf16 tensor -> numpy float32 with the same values"""
    return t.detach().cpu().to(torch.float32).numpy()


def oqp(bqp):
    """binding QParams -> oracle QParams"""
    return OQP(bqp.bits, bool(bqp.symmetric), float(np.float32(bqp.scale)), bqp.zero_point)


def random_codes(rng, shape, symmetric=True):
    lo, hi = (-8, 8) if symmetric else (0, 16)
    return rng.integers(lo, hi, shape).astype(np.int8 if symmetric else np.uint8)


def packed_dev(codes):
    return dev(OQ.pack_int4(codes))


def bf16_ulp_diff(a, b):
    """distance in bf16 ulps between two float32 arrays holding bf16 values"""
    def key(x):
        bits = (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.int64)
        return np.where(bits & 0x8000, 0x8000 - bits, bits)          # monotone integer key
    return np.abs(key(a) - key(b))


def assert_bf16_close(got, want, what=""):
    """spec tolerance for bf16 outputs: within 1 bf16 ulp or 1e-2 relative"""
    got = np.asarray(got, dtype=np.float32)
    want = np.asarray(want, dtype=np.float32)
    ulp = bf16_ulp_diff(got, want)
    rel = np.abs(got - want) <= 1e-2 * np.abs(want)
    bad = ~((ulp <= 1) | rel)
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outputs off; worst ulp {ulp.max()}"
    return int((ulp > 0).sum())


# ------------------------------------------------------------------------------------------
# guard bands: every buffer the binding allocates (outputs, codes, per-token vectors, workspaces)
# sits between two bands of a known pattern, and starts out poisoned, so that a write past either
# end, or an output the kernel never wrote, is seen even though the comparison itself only covers
# the valid region
# ------------------------------------------------------------------------------------------
GUARD_BYTES = 4096
GUARD_PATTERN = 0xA5
POISON = 0xFF               # bf16 / f32: a NaN; int32: -1; codes: 0xFF


class GuardedAllocator:
    def __init__(self):
        self.live = []          # (raw uint8 tensor, payload bytes)

    def __call__(self, shape, dtype, device):
        shape = (int(shape),) if isinstance(shape, (int, np.integer)) else tuple(int(s) for s in shape)
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        padded = (n + 255) // 256 * 256
        raw = torch.empty((2 * GUARD_BYTES + padded,), dtype=torch.uint8, device=device)
        raw[:GUARD_BYTES] = GUARD_PATTERN
        raw[GUARD_BYTES:GUARD_BYTES + n] = POISON
        raw[GUARD_BYTES + n:] = GUARD_PATTERN
        self.live.append((raw, n))
        return raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)

    def check(self, release=True):
        """Asserts that no band was written; with `release`, forgets the buffers (frees their memory once
        the test drops its own references)."""
        for raw, n in self.live:
            lo = raw[:GUARD_BYTES]
            hi = raw[GUARD_BYTES + n:]
            assert bool((lo == GUARD_PATTERN).all()), f"write BEFORE a {n}-byte buffer"
            assert bool((hi == GUARD_PATTERN).all()), f"write PAST the end of a {n}-byte buffer"
        if release:
            self.live = []


GUARDS = GuardedAllocator()


def guarded_empty(shape, dtype, device=DEV):
    """A poisoned buffer between guard bands for outputs a test allocates itself."""
    return GUARDS(shape, dtype, device)


def check_guards():
    GUARDS.check(release=True)
