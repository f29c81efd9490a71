"""Model shapes of the synthetic workloads (no arithmetic of the decode step lives here).

The paper measures Qwen3 and Llama-3.2 checkpoints and a 30B-class MoE (Table 1);
the checkpoints are not available, so only their shapes are reproduced.
"""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Shape:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    mlp_inter: int
    vocab: int
    qk_norm: int
    tie_embeddings: int
    rms_eps: float
    rope_base: float
    head_dim: int = 128
    group_size: int = 64
    bits: int = 4
    n_experts: int = 0
    top_k: int = 0
    expert_inter: int = 0
    norm_topk_prob: int = 0
    max_batch: int = 16
    max_positions: int = 8192 + 1024

    def with_(self, **kw):
        return replace(self, **kw)

    @property
    def qkv_out(self):
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def kv_bytes_per_token(self):
        """K and V bytes one token occupies over all layers (bf16)."""
        return self.n_layers * 2 * self.n_kv_heads * self.head_dim * 2


QWEN3_0P6B = Shape("qwen3-0.6b-shaped", 28, 1024, 16, 8, 3072, 151936, 1, 1, 1e-6, 1e6)
LLAMA32_3B = Shape("llama-3.2-3b-shaped", 28, 3072, 24, 8, 8192, 128256, 0, 1, 1e-5, 5e5)
QWEN3_8B = Shape("qwen3-8b-shaped", 36, 4096, 32, 8, 12288, 151936, 1, 0, 1e-6, 1e6)
MOE_30B = Shape("moe-30b-a3b-shaped", 48, 2048, 32, 4, 0, 151936, 1, 0, 1e-6, 1e6,
                n_experts=128, top_k=8, expert_inter=768, norm_topk_prob=1)

PRESETS = {s.name: s for s in (QWEN3_0P6B, LLAMA32_3B, QWEN3_8B, MOE_30B)}


def toy(name="toy", n_layers=2, hidden=128, n_q_heads=4, n_kv_heads=2, mlp_inter=256, vocab=512,
        qk_norm=1, tie_embeddings=0, rms_eps=1e-6, rope_base=1e4, max_positions=512, **kw):
    """A small shape of the same structure for tests (head_dim stays 128)."""
    return Shape(name, n_layers, hidden, n_q_heads, n_kv_heads, mlp_inter, vocab, qk_norm, tie_embeddings,
                 rms_eps, rope_base, max_positions=max_positions, **kw)


def q4_bytes(N, K):
    """Bytes of one 4-bit group-64 tensor: packed codes + bf16 scale + bf16 bias."""
    return N * K // 2 + 2 * (N * (K // 64) * 2)


def weight_bytes(shape, experts_touched_per_layer=None):
    """Packed-weight bytes one decode step streams (every projection once)."""
    H, d = shape.hidden, shape.head_dim
    per_layer = q4_bytes(shape.qkv_out, H) + q4_bytes(H, shape.n_q_heads * d)
    if shape.n_experts:
        e = shape.n_experts if experts_touched_per_layer is None else experts_touched_per_layer
        per_layer += shape.n_experts * H * 2  # bf16 router
        per_layer += e * (q4_bytes(2 * shape.expert_inter, H) + q4_bytes(H, shape.expert_inter))
    else:
        per_layer += q4_bytes(2 * shape.mlp_inter, H) + q4_bytes(H, shape.mlp_inter)
    return shape.n_layers * per_layer + q4_bytes(shape.vocab, H)
