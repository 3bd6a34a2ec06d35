"""FF blocks without a gate (Eq. 2 of the paper: FF_1(x) = sigma(W_1 x + b_1), as in OPT) through
the C ABI against the CPU oracle: prompt phase with the statistic, slicing, both decode paths and
one block end to end.  There is no W_g: the gate pointers are NULL on the GPU side and None in the
oracle."""
import numpy as np
import pytest
import torch

from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G
from gpu_util import check_expert_set, dev, np64, rand, assert_output, score_tol
from test_gpu_kernels import TD, h64, make_layer

pytestmark = pytest.mark.gpu

ACTS = ["relu", "gelu_tanh", "gelu_erf", "silu"]

# S, d, d_ff: fp32-FMA kernels (small or odd shapes; d_ff = 1408 is a multiple of 128 but not of 256), then
# tensor-core shapes (tiles of 256 neurons), the last one with a cut last round of tiles (160 tiles on 148 SMs)
PREFILL_SHAPES = [(64, 256, 688), (1, 64, 96), (37, 72, 200), (130, 512, 1408), (130, 512, 1024), (256, 1024, 2816 + 256),
                  (300, 1024, 4096), (256, 1024, 20480)]


# (the largest case is there for the tensor-core tiling, which is bf16 only)
@pytest.mark.parametrize("dtype,S,d,d_ff", [(dt, *shape) for dt in ("f32", "bf16") for shape in PREFILL_SHAPES
                                            if not (dt == "f32" and shape[2] > 5000)])
def test_prefill_score_without_a_gate_matches_oracle(dtype, S, d, d_ff):
    act = ACTS[(S + d_ff // 8) % 4]
    L, host = make_layer(d, d_ff, dtype, act=act, bias=(S in (37, 130, 256)), seed=S + d, S_max=S)
    x = rand((S, d), TD[dtype], 5) + rand((1, d), TD[dtype], 6, 4.0 / d ** 0.5)
    y, s = L.prefill(x)
    ref_y, ref_z = O.ff_dense(np64(x), None, h64(host, "wu"), h64(host, "wd"), act, None, h64(host, "bu"), h64(host, "bd"))
    ref_s = O.flock_score(ref_z)
    assert L.status() == G.OK
    assert_output(np64(y), ref_y, dtype)
    s = np64(s)
    assert np.all(np.abs(s - ref_s) <= score_tol(dtype) * ref_s + 1e-6 * np.sqrt(S / d_ff))
    assert abs(float(np.sum(s * s)) - S) < 1e-5 * S     # rows of Zbar are unit vectors
    _, s2 = L.prefill(x, want_y=False)
    assert np.array_equal(np64(s2), s)


@pytest.mark.parametrize("dtype,pieces,d,d_ff", [("bf16", (100, 37, 119), 512, 1024), ("bf16", (300, 1, 211), 1024, 4096),
                                                 ("f32", (1, 1, 62), 256, 688)])
def test_prefill_without_a_gate_fed_piece_by_piece(dtype, pieces, d, d_ff):
    """The statistic's sums of squares carried across the pieces of a prompt (Eq. 6) for a block without a gate."""
    S, act = sum(pieces), "gelu_tanh"
    L, host = make_layer(d, d_ff, dtype, act=act, bias=True, seed=S + d, S_max=S)
    x = rand((S, d), TD[dtype], 25) + rand((1, d), TD[dtype], 26, 4.0 / d ** 0.5)
    xd = x.to(dev())
    y = torch.empty((S, d), device=dev(), dtype=TD[dtype])
    sumsq = torch.full((d_ff,), float("nan"), device=dev())        # the first piece must not read it
    score = torch.empty((d_ff,), device=dev())
    at = 0
    for i, n in enumerate(pieces):
        last = i == len(pieces) - 1
        G.griffin_ff_prefill_score_chunk(L.desc, L.weights, xd[at:at + n], y[at:at + n], sumsq, score if last else None,
                                         i == 0, L.ws)
        at += n
    assert L.status() == G.OK
    ref_y, ref_z = O.ff_dense(np64(x), None, h64(host, "wu"), h64(host, "wd"), act, None, h64(host, "bu"), h64(host, "bd"))
    ref_s = O.flock_score(ref_z)
    assert_output(np64(y), ref_y, dtype)
    s = np64(score)
    assert np.all(np.abs(s - ref_s) <= score_tol(dtype) * ref_s + 1e-6 * np.sqrt(S / d_ff))
    assert abs(float(np.sum(s * s)) - S) < 1e-5 * S


@pytest.mark.parametrize("act", ACTS)
def test_prefill_sigma_of_each_block_without_a_gate(act):
    L, host = make_layer(512, 1024, "bf16", act=act, bias=True, seed=11, S_max=96)
    x = rand((96, 512), torch.bfloat16, 7)
    y, s = L.prefill(x)
    ref_y, ref_z = O.ff_dense(np64(x), None, h64(host, "wu"), h64(host, "wd"), act, None, h64(host, "bu"), h64(host, "bd"))
    assert_output(np64(y), ref_y, "bf16")
    ref_s = O.flock_score(ref_z)
    assert np.all(np.abs(np64(s) - ref_s) <= score_tol("bf16") * ref_s + 1e-6 * np.sqrt(96 / 1024))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_compact_without_a_gate_is_exact(dtype):
    d, d_ff, k = 520, 1032, 517
    L, host = make_layer(d, d_ff, dtype, act="relu", bias=True, seed=3)
    e_np = np.sort(np.random.default_rng(1).choice(d_ff, size=k, replace=False)).astype(np.int32)
    cs = L.compact(torch.from_numpy(e_np).to(dev()))
    assert L.status() == G.OK
    wu_c, wd_c, bu_c = cs._keep[1], cs._keep[2], cs._keep[4]
    assert cs._keep[0] is None and cs._keep[3] is None
    ref = O.compact_experts(e_np, None, host["wu"].view(torch.int16 if dtype == "bf16" else torch.int32).numpy(),
                            host["wd"].view(torch.int16 if dtype == "bf16" else torch.int32).numpy(), None,
                            host["bu"].view(torch.int16 if dtype == "bf16" else torch.int32).numpy())
    bits = lambda t: t.cpu().view(torch.int16 if dtype == "bf16" else torch.int32).numpy()
    assert np.array_equal(bits(wu_c), ref["w_up"])
    assert np.array_equal(bits(wd_c)[:, :k], ref["w_down"]) and not bits(wd_c)[:, k:].any()
    assert np.array_equal(bits(bu_c), ref["b_up"])


DECODE_SHAPES = [
    # d, d_ff, k, B
    (256, 688, 344, 1),
    (64, 96, 37, 3),         # odd k: padded ldk, a last pair with one row
    (1000, 1504, 751, 2),
    (2048, 5632, 2815, 1),
    (4096, 16384, 8192, 1),  # OPT-6.7B shape
    (5120, 2048, 1024, 8),
    (8192, 1024, 512, 1),
    (512, 9008, 9008, 1),    # k = d_ff, rows of W_2_hat of two chunks
    (3136, 9504, 9473, 8),   # 16 pairs of rows per warp: the run-time pool of the register stream, ending in a pair of one row
]


@pytest.mark.parametrize("dtype,kernel", [("f32", 0), ("bf16", G.DECODE_RING), ("bf16", G.DECODE_STREAM)])
@pytest.mark.parametrize("d,d_ff,k,B", DECODE_SHAPES)
def test_decode_without_a_gate_matches_oracle(dtype, kernel, d, d_ff, k, B):
    act = ACTS[(d // 8 + k) % 4]
    L, host = make_layer(d, d_ff, dtype, act=act, bias=(d_ff < 6000), seed=d + k, n_seq=B)
    rs = np.random.default_rng(d + k)
    x = rand((B, d), TD[dtype], 98)
    sets, refs = [], []
    for b in range(B):
        e_np = np.sort(rs.choice(d_ff, size=k, replace=False)).astype(np.int32)
        sets.append(L.compact(torch.from_numpy(e_np).to(dev())))
        c = O.compact_experts(e_np, None, h64(host, "wu"), h64(host, "wd"), None, h64(host, "bu"))
        refs.append(O.ff_pruned(np64(x[b]), c, act, h64(host, "bd")))
    y = L.decode(sets, x, kernel)
    y2 = L.decode(sets, x, kernel | G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    y3 = L.decode(sets, x, kernel | G.DECODE_OVERLAP_WEIGHT_PREFETCH | G.DECODE_TCGEN05)   # (the flag falls back here)
    assert L.status() == G.OK
    for b in range(B):
        assert_output(np64(y[b]), refs[b], dtype, b)
    assert torch.equal(y, y2) and torch.equal(y, y3)


INDEXED_SHAPES = [
    (256, 688, 344, 1, True),
    (64, 96, 37, 3, True),
    (1000, 1504, 751, 2, True),
    (4096, 16384, 8192, 1, False),   # OPT-6.7B shape
    (4096, 16384, 8191, 4, False),
    (5120, 2048, 1024, 8, True),
    (8192, 1024, 512, 2, False),
    (512, 1536, 1536, 2, True),
]


@pytest.mark.parametrize("d,d_ff,k,B,bias", INDEXED_SHAPES)
def test_decode_indexed_without_a_gate_matches_oracle_and_compact_path(d, d_ff, k, B, bias):
    act = ACTS[(d // 8 + k + B) % 4]
    L, host = make_layer(d, d_ff, "bf16", act=act, bias=bias, seed=5 * d + k, n_seq=B)
    rs = np.random.default_rng(d + k + B)
    x = rand((B, d), torch.bfloat16, 96)
    idx = np.empty((B, k), dtype=np.int32)
    refs = []
    for b in range(B):
        e_np = rs.choice(d_ff, size=k, replace=False).astype(np.int32)
        idx[b] = e_np if b % 2 else np.sort(e_np)
        c = O.compact_experts(idx[b], None, h64(host, "wu"), h64(host, "wd"), None, h64(host, "bu"))
        refs.append(O.ff_pruned(np64(x[b]), c, act, h64(host, "bd")))
    e = torch.from_numpy(idx).to(dev())
    y = L.decode_indexed(e, x)
    y2 = L.decode_indexed(e, x, G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    assert L.status() == G.OK
    assert torch.equal(y, y2)
    for b in range(B):
        assert_output(np64(y[b]), refs[b], "bf16", b)
    if B <= 2:
        y_c = L.decode([L.compact(e[b]) for b in range(B)], x)
        assert_output(np64(y), np64(y_c), "bf16", scale=2.0)


@pytest.mark.parametrize("dtype,d,d_ff,S,T", [("f32", 256, 688, 64, 4), ("bf16", 1024, 4096, 200, 3)])
def test_one_block_without_a_gate_end_to_end(dtype, d, d_ff, S, T):
    """Prompt phase, top-k, slicing and decode in the paper's order, every intermediate against the oracle."""
    act, k = "relu", d_ff // 2
    L, host = make_layer(d, d_ff, dtype, act=act, bias=True, seed=77, S_max=S)
    shared = rand((1, d), TD[dtype], 8, 4.0 / d ** 0.5)
    x, xd = rand((S, d), TD[dtype], 9) + shared, rand((T, d), TD[dtype], 10) + shared
    ref = O.griffin_layer(np64(x), np64(xd), None, h64(host, "wu"), h64(host, "wd"), act, k, None, h64(host, "bu"),
                          h64(host, "bd"))
    y, s = L.prefill(x)
    e = L.select(s, k)
    cs = L.compact(e)
    yd = torch.cat([L.decode([cs], xd[t:t + 1]) for t in range(T)])
    assert L.status() == G.OK
    assert_output(np64(y), ref["y"], dtype)
    e_np = e.cpu().numpy()
    check_expert_set(e_np, ref["s"], k)
    c = O.compact_experts(e_np, None, h64(host, "wu"), h64(host, "wd"), None, h64(host, "bu"))
    assert_output(np64(yd), O.ff_pruned(np64(xd), c, act, h64(host, "bd")), dtype)


def test_gate_pointers_must_match_the_kind_of_block():
    L, host = make_layer(256, 512, "bf16", act="relu", seed=1, S_max=8)
    fake_gate = torch.zeros((512, 256), device=dev(), dtype=torch.bfloat16)
    w_bad = G.make_weights(fake_gate, L.t["wu"], L.t["wd"])
    x = rand((8, 256), torch.bfloat16, 2).to(dev())
    y, s = torch.empty_like(x), torch.empty((512,), device=dev(), dtype=torch.float32)
    with pytest.raises(G.GriffinError) as err:
        G.griffin_ff_prefill_score(L.desc, w_bad, x, y, s, L.ws)      # a gate for a block that has none
    assert err.value.status == G.ERR_INVALID_ARG
    gated = G.make_desc(256, 512, "swiglu", "bf16")
    with pytest.raises(G.GriffinError) as err:
        G.griffin_ff_prefill_score(gated, L.weights, x, y, s, L.ws)   # no gate for a block that needs one
    assert err.value.status == G.ERR_INVALID_ARG
