"""Helpers shared by the GPU parity tests (comparison utilities and scenario setup)."""
import numpy as np
import torch

from oracle import q4d_oracle as orc
from workload import gen


def bits(t):
    """torch bf16 tensor -> numpy uint16 bit patterns (host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def bf16_ulp_distance(a_bits, b_bits):
    """Distance in bf16 steps between two arrays of bf16 bit patterns (sign-magnitude aware)."""
    def key(b):
        b = b.astype(np.int64)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(np.asarray(a_bits)) - key(np.asarray(b_bits)))


def assert_bf16_close(got_bits, want_bits, max_ulp=1, max_mismatch_frac=0.01, what=""):
    """All elements within max_ulp bf16 steps and at most max_mismatch_frac of them different at all.

    Both sides round a value computed in different precision (fp32 on the GPU, fp64 in the oracle) to bf16,
    so a small fraction of elements that sit next to a rounding boundary may land one step apart.
    """
    d = bf16_ulp_distance(got_bits, want_bits)
    frac = float((d > 0).mean()) if d.size else 0.0
    assert d.max(initial=0) <= max_ulp, f"{what}: max bf16 step distance {d.max()} > {max_ulp}"
    assert frac <= max_mismatch_frac, f"{what}: {frac:.4%} of elements differ (> {max_mismatch_frac:.2%})"
    return frac


class Scenario:
    """Weights, pool and requests on the GPU, mirrored on the host for the oracle."""

    def __init__(self, shape, lens, seed=0, extra_blocks=8, device="cuda"):
        self.shape, self.device = shape, device
        self.weights = gen.make_weights(shape, seed, device)
        need = sum((l + 1 + 64 + 15) // 16 for l in lens) + extra_blocks
        self.pool = gen.make_pool(shape, need, device)
        self.alloc = gen.BlockAllocator(need, seed)
        self.lens = list(lens)
        self.blocks = []
        for r, l in enumerate(lens):
            blk = self.alloc.alloc((l + 1 + 15) // 16)
            gen.fill_blocks(self.pool, blk, seed, "kv", r)
            self.blocks.append(blk)
        rng = np.random.default_rng(seed + 1000)
        self.tokens = rng.integers(0, shape.vocab, size=len(lens)).astype(np.int32)
        self.oracle = orc.OracleModel(shape, self.weights)
        self.host_pool = orc.to_np(self.pool).copy()

    def block_tables(self):
        for r, l in enumerate(self.lens):
            need = (l + 1 + 15) // 16
            if need > len(self.blocks[r]):
                self.blocks[r].extend(self.alloc.alloc(need - len(self.blocks[r])))
        mb = max(len(b) for b in self.blocks)
        bt = np.zeros((len(self.lens), mb), dtype=np.int32)
        for r, b in enumerate(self.blocks):
            bt[r, :len(b)] = b
        return bt
