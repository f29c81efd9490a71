"""GPU parity of the single operations against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_util import assert_bf16_close, bits
from oracle import q4d_oracle as orc
from workload import gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4d():
    from paper_2601_19139_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _np_triple(w):
    return orc.to_np(w[0], np.uint32), orc.to_np(w[1]), orc.to_np(w[2])


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(*shape, generator=g, device="cuda") * scale).to(torch.bfloat16)


# ------------------------------------------------------------ bit-exact exports

@pytest.mark.parametrize("N,K", [(48, 256), (1000, 1024), (96, 3072)])
def test_dequant_is_bit_exact(q4d, N, K):
    w = gen.random_q4(N, K, "cuda", "gpu-dequant", N, K)
    got = q4d.debug_dequant(w).cpu().numpy()
    want = orc.dequant_q4(*_np_triple(w))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_dequant_is_bit_exact_on_edge_scales(q4d):
    q = torch.randint(-2 ** 31, 2 ** 31 - 1, (16, 32), dtype=torch.int64, device="cuda").to(torch.int32)
    vals = torch.tensor([0.0, 1.0, -0.5, 1e-3, 2.0 ** -126, 2.0 ** -130, 1e30, 0.00665283203125, 3.140625, -0.0,
                         255.0, 7.5e29, -3.0, 2.0 ** -127, 1e-38, 65280.0], device="cuda")
    s = vals.to(torch.bfloat16).view(16, 1).repeat(1, 4).contiguous()
    b = vals.flip(0).to(torch.bfloat16).view(16, 1).repeat(1, 4).contiguous()
    got = q4d.debug_dequant((q, s, b)).cpu().numpy()
    want = orc.dequant_q4(orc.to_np(q, np.uint32), orc.to_np(s), orc.to_np(b))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_embed_is_bit_exact(q4d):
    table = gen.random_q4(5000, 1024, "cuda", "gpu-embed")
    toks = torch.tensor([0, 4999, 17, 17, 2500], dtype=torch.int32, device="cuda")
    got = bits(q4d.embed(table, toks))
    W = orc.dequant_q4(*_np_triple(table))
    want = orc.bf16_round(W[toks.cpu().numpy()].astype(np.float64))
    assert np.array_equal(got, want)


# ---------------------------------------------------------------------- GEMM

GEMM_CASES = [
    # N, K, n  -- several row blocks and K slices, ragged N, every batch size class
    (4096, 1024, 1), (4096, 1024, 16), (1024, 2048, 3), (1024, 3072, 16), (6144, 1024, 8), (6144, 4096, 9),
    (272, 256, 5), (5000, 512, 16), (4096, 12288, 2), (130, 768, 16),
    # K in three parts at the full batch; many rounds per CTA with a ragged last tile; a single tile
    (4096, 12288, 16), (40010, 512, 12), (16, 256, 16), (48, 1024, 4),
]


@pytest.mark.parametrize("N,K,n", GEMM_CASES)
def test_q4_gemm_f32_matches_oracle(q4d, N, K, n):
    w = gen.random_q4(N, K, "cuda", "gpu-gemm", N, K)
    x = _rand_bf16((n, K), N + K + n)
    got = q4d.q4_gemm(w, x, n, epilogue=2).cpu().numpy().astype(np.float64)
    want = orc.q4_matmul(*_np_triple(w), bits(x))
    rms = np.sqrt((want ** 2).mean())
    # fp32 accumulation of exact products vs fp64: error ~ 1e-7 * sqrt(terms) * partial-sum magnitude
    assert np.abs(got - want).max() <= 3e-5 * rms, np.abs(got - want).max() / rms


def _assert_residual_close(got_bits, res_in_bits, want):
    """out = bf16(res + bf16(v)) against the oracle's.  bf16(v) may land one step of v apart (fp32 vs fp64 sums next
    to a rounding boundary); where the residual cancels v that step is several steps of the sum, so the bound is a
    step of v plus a step of the sum, and at most 1 % of the elements may differ at all."""
    v = orc.bf16_to_f64(orc.bf16_round(want))
    want_res = orc.bf16_to_f64(orc.bf16_round(orc.bf16_to_f64(res_in_bits) + v))
    got_res = orc.bf16_to_f64(got_bits)
    step = lambda a: 2.0 ** (np.floor(np.log2(np.maximum(np.abs(a), 1e-30))) - 7)
    err = np.abs(got_res - want_res)
    assert (err <= step(v) + step(want_res)).all(), float((err / (step(v) + step(want_res))).max())
    assert (got_res != want_res).mean() <= 0.01


def test_q4_gemm_bf16_and_residual_epilogues(q4d):
    N, K, n = 2048, 1024, 16
    w = gen.random_q4(N, K, "cuda", "gpu-gemm-epi")
    x = _rand_bf16((n, K), 5)
    want = orc.q4_matmul(*_np_triple(w), bits(x))
    got = bits(q4d.q4_gemm(w, x, n, epilogue=0))
    assert_bf16_close(got, orc.bf16_round(want), what="bf16 epilogue")
    res = _rand_bf16((n, N), 6, 0.5)
    res_in = bits(res).copy()
    q4d.q4_gemm(w, x, n, epilogue=1, out=res)
    _assert_residual_close(bits(res), res_in, want)


def _random_gemm_shapes(count, seed):
    """Seeded shapes that land in every branch of the projection kernels' planning: one tile or thousands, spans
    shorter than a stage or several tiles long, one to twelve K-slices (K up to three parts), both batch classes."""
    rng = np.random.default_rng(seed)
    shapes_ = []
    for _ in range(count):
        N = int(rng.choice([rng.integers(1, 64), rng.integers(64, 2400), rng.integers(2400, 30000)]))
        K = 256 * int(rng.choice([1, 2, 3, 4, 5, 8, 12, 16, 20, 48]))
        if N * K > 40_000_000:
            N = 40_000_000 // K
        shapes_.append((N, K, int(rng.integers(1, 17)), int(rng.integers(0, 3))))
    return shapes_


@pytest.mark.parametrize("N,K,n,epi", _random_gemm_shapes(14, 2024))
def test_q4_gemm_random_shapes_every_epilogue(q4d, N, K, n, epi):
    w = gen.random_q4(N, K, "cuda", "gpu-gemm-rand", N, K)
    x = _rand_bf16((n, K), N + 3 * K + n)
    want = orc.q4_matmul(*_np_triple(w), bits(x))
    if epi == 2:
        got = q4d.q4_gemm(w, x, n, epilogue=2).cpu().numpy().astype(np.float64)
        rms = np.sqrt((want ** 2).mean())
        assert np.abs(got - want).max() <= 3e-5 * rms, np.abs(got - want).max() / rms
    elif epi == 0:
        assert_bf16_close(bits(q4d.q4_gemm(w, x, n, epilogue=0)), orc.bf16_round(want), what="bf16 epilogue")
    else:
        res = _rand_bf16((n, N), N + K, 0.5)
        res_in = bits(res).copy()
        q4d.q4_gemm(w, x, n, epilogue=1, out=res)
        _assert_residual_close(bits(res), res_in, want)


def test_q4_gemm_silu_mul_prologue(q4d):
    N, K, n = 1024, 3072, 16
    w = gen.random_q4(N, K, "cuda", "gpu-gemm-silu")
    gu = _rand_bf16((n, 2 * K), 7, 1.5)
    gub = bits(gu)
    h = orc.silu_mul(gub[:, :K], gub[:, K:])
    want = orc.q4_matmul(*_np_triple(w), h)
    got = q4d.q4_gemm(w, gu, n, prologue=1, epilogue=2).cpu().numpy().astype(np.float64)
    rms = np.sqrt((want ** 2).mean())
    # a handful of h elements may round one bf16 step differently (fp32 vs fp64 silu)
    assert np.abs(got - want).max() <= 2e-3 * rms


def test_q4_gemm_is_deterministic_and_batch_invariant_at_fixed_n(q4d):
    N, K, n = 4096, 4096, 16
    w = gen.random_q4(N, K, "cuda", "gpu-gemm-det")
    x = _rand_bf16((n, K), 8)
    a = q4d.q4_gemm(w, x, n, epilogue=2)
    b = q4d.q4_gemm(w, x, n, epilogue=2)
    assert torch.equal(a, b)
    x2 = x.clone()
    x2[3:] = _rand_bf16((n - 3, K), 9)
    c = q4d.q4_gemm(w, x2, n, epilogue=2)
    assert torch.equal(a[:3], c[:3])          # other requests in the batch do not change a request's result


# ------------------------------------------------------------------- RMSNorm

@pytest.mark.parametrize("n,H", [(1, 1024), (16, 4096), (5, 3072)])
def test_rmsnorm_matches_oracle(q4d, n, H):
    x = _rand_bf16((n, H), H + n, 0.3)
    w = gen.norm_weight(H, "cuda", "gpu-norm", H)
    got = bits(q4d.rmsnorm(x, w, 1e-6))
    want = orc.rmsnorm(bits(x), bits(w), 1e-6)
    assert_bf16_close(got, want, what="rmsnorm")


# -------------------------------------------------------------------- argmax

def test_argmax_matches_oracle_with_ties(q4d):
    g = torch.Generator(device="cuda").manual_seed(3)
    lg = torch.randn(16, 151936, generator=g, device="cuda")
    lg[1, 17] = lg[1, 90000] = 50.0
    lg[2] = 0.25
    lg[3, 151935] = 60.0
    lg[4, 0] = 60.0
    got = q4d.argmax(lg).cpu().numpy()
    assert np.array_equal(got, orc.argmax(lg.cpu().numpy()))
    assert got[1] == 17 and got[2] == 0 and got[3] == 151935 and got[4] == 0


# ------------------------------------------------- rope + append, paged attention

def _pool_layer(nblocks, nkv, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return torch.randn(2, nblocks, nkv, 16, 128, generator=g, device="cuda").to(torch.bfloat16)


def _tables(lens, nblocks, seed):
    rng = np.random.default_rng(seed)
    perm = rng.permutation(nblocks)
    mb = max((l + 1 + 15) // 16 for l in lens)
    bt = np.zeros((len(lens), mb), dtype=np.int32)
    cur = 0
    for r, l in enumerate(lens):
        nb = (l + 1 + 15) // 16
        bt[r, :nb] = perm[cur:cur + nb]
        cur += nb
    return bt


def _close_after_two_roundings(got_bits, want_bits, what):
    """The head is rounded to bf16 after the norm and again after the rotation.  A one-step difference after the
    first rounding moves the rotated value by up to one step of the larger input, which can be several steps of a
    small output, so the bound is absolute: one bf16 step of the head's largest element; and few elements differ."""
    got, want = orc.bf16_to_f64(got_bits), orc.bf16_to_f64(want_bits)
    assert np.abs(got - want).max() <= 2.0 ** -7 * np.abs(want).max(), what
    assert (got_bits != want_bits).mean() <= 0.05, what


@pytest.mark.parametrize("nq,nkv,qk_norm", [(16, 8, True), (24, 8, False), (32, 4, True)])
def test_rope_append_matches_oracle(q4d, nq, nkv, qk_norm):
    lens = [0, 15, 16, 100, 257]
    n = len(lens)
    nblocks = 64
    pool = _pool_layer(nblocks, nkv, 11)
    before = bits(pool).copy()
    bt = _tables(lens, nblocks, 12)
    qkv = _rand_bf16((n, (nq + 2 * nkv) * 128), 13)
    qn = gen.norm_weight(128, "cuda", "gpu-qn") if qk_norm else None
    kn = gen.norm_weight(128, "cuda", "gpu-kn") if qk_norm else None
    rope = gen.rope_table(512, 128, 1e6, "cuda")
    q_out = q4d.rope_append(qkv, qn, kn, 1e-6, rope, nq, nkv, torch.tensor(lens, dtype=torch.int32, device="cuda"),
                            torch.from_numpy(bt).cuda(), pool[0], pool[1])
    torch.cuda.synchronize()
    after = bits(pool)
    tab = rope.cpu().numpy()
    qb = bits(qkv).reshape(n, nq + 2 * nkv, 128)
    touched = np.zeros_like(before, dtype=bool)
    for r, l in enumerate(lens):
        for hd in range(nq + nkv):
            head = qb[r, hd]
            if qk_norm:
                head = orc.rmsnorm(head[None], bits(qn if hd < nq else kn), 1e-6)[0]
            want = orc.rope(head, tab[l])
            if hd < nq:
                _close_after_two_roundings(bits(q_out)[r, hd], want, "q")
            else:
                blk, slot = bt[r, l // 16], l % 16
                _close_after_two_roundings(after[0, blk, hd - nq, slot], want, "k")
                touched[0, blk, hd - nq, slot] = True
        for hv in range(nkv):
            blk, slot = bt[r, l // 16], l % 16
            assert np.array_equal(after[1, blk, hv, slot], qb[r, nq + nkv + hv])     # v is copied verbatim
            touched[1, blk, hv, slot] = True
    assert np.array_equal(after[~touched], before[~touched])                         # nothing else was written


@pytest.mark.parametrize("nq,nkv,lens,chunk", [
    (16, 8, [0, 1, 15, 16, 17, 255, 256, 1000], 0),
    (32, 8, [2047, 300, 64, 63], 64),
    (24, 8, [700, 33], 256),
    (32, 4, [513, 129, 4000], 0),
    (8, 8, [50], 0),
    (32, 2, [333, 90], 128),
    # more than eight chunks per request: eleven 12-tile chunks with a 3-tile tail, and nine planner-sized chunks
    (32, 4, [1953, 194, 1036], 192),
    (32, 8, [9000, 40], 0),
    # a full batch on four kv heads: the planner's one-wave chunking gives a request dozens of chunks across the
    # three resident CTAs per SM; and a group of five query heads (columns 5..7 of the token-major MMA stay empty)
    (32, 4, [8191, 5003, 3100, 2047, 1500, 1024, 1023, 777, 512, 300, 255, 129, 64, 17, 1, 0], 0),
    (40, 8, [1200, 31, 640], 0),
])
def test_paged_attention_matches_oracle(q4d, nq, nkv, lens, chunk):
    n = len(lens)
    nblocks = sum((l + 1 + 15) // 16 for l in lens) + 5
    pool = _pool_layer(nblocks, nkv, 21)
    bt = _tables(lens, nblocks, 22)
    q = _rand_bf16((n, nq, 128), 23)
    out = q4d.paged_attention(q, pool[0], pool[1], lens, torch.from_numpy(bt).cuda(), chunk_tokens=chunk)
    host_pool = bits(pool)[None]        # one layer: [1][2][blocks][nkv][16][128]
    want = orc.attention_paged(bits(q), host_pool, nq, nkv, 16, 128, 0, lens, bt)
    assert_bf16_close(bits(out), want, what="attention")


def test_paged_attention_split_choice_does_not_matter_beyond_rounding(q4d):
    lens = [1500, 77]
    nq, nkv = 16, 8
    nblocks = 120
    pool = _pool_layer(nblocks, nkv, 31)
    bt = torch.from_numpy(_tables(lens, nblocks, 32)).cuda()
    q = _rand_bf16((2, nq, 128), 33)
    outs = [bits(q4d.paged_attention(q, pool[0], pool[1], lens, bt, chunk_tokens=c)) for c in (64, 256, 4096)]
    for o in outs[1:]:
        assert_bf16_close(o, outs[0], what="split choice")


def test_kv_gather_is_bit_exact(q4d):
    from workload import shapes
    shape = shapes.toy("toy-gather", hidden=256, mlp_inter=512, n_layers=3)
    weights = gen.make_weights(shape, 0, "cuda")
    pool_t = gen.make_pool(shape, 40, "cuda")
    gen.fill_blocks(pool_t, range(40), "gather")
    model = q4d.Model(shape, weights)
    pool = q4d.KVPool(model, pool_t)
    bt = np.random.default_rng(5).permutation(40)[:9].astype(np.int32)
    host = bits(pool_t)
    for layer in (0, 2):
        k, v = q4d.debug_kv_gather(pool, layer, torch.from_numpy(bt).cuda(), 131)
        for h in range(shape.n_kv_heads):
            ko, vo = orc.kv_gather(host, shape.n_kv_heads, 16, 128, layer, h, bt, 131)
            assert np.array_equal(bits(k)[:, h], ko) and np.array_equal(bits(v)[:, h], vo)
    pool.close()
    model.close()
