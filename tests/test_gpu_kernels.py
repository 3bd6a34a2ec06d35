"""Per-kernel parity of the CUDA path (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G
from gpu_util import (GpuLayer, check_expert_set, dev, np64, rand, assert_output, score_tol)

pytestmark = pytest.mark.gpu

TD = {"f32": torch.float32, "bf16": torch.bfloat16}


def make_layer(d, d_ff, dtype, act="swiglu", bias=False, seed=0, S_max=0, n_seq=1):
    td = TD[dtype]
    gated = G.act_is_gated(act)     # a block without a gate (Eq. 2) has no W_g, b_g
    wg, wu = rand((d_ff, d), td, seed + 1, d ** -0.5) if gated else None, rand((d_ff, d), td, seed + 2, d ** -0.5)
    wd = rand((d, d_ff), td, seed + 3, d_ff ** -0.5)
    bg = rand((d_ff,), td, seed + 4, 0.3) if bias and gated else None
    bu = rand((d_ff,), td, seed + 5, 0.3) if bias else None
    bd = rand((d,), td, seed + 6, 0.3) if bias else None
    host = dict(wg=wg, wu=wu, wd=wd, bg=bg, bu=bu, bd=bd)
    return GpuLayer(d, d_ff, act, dtype, wg, wu, wd, bg, bu, bd, S_max=S_max, n_seq=n_seq), host


def h64(host, name):
    return None if host[name] is None else np64(host[name])


# ------------------------------------------------------------------ top-k ---

@pytest.mark.parametrize("d_ff,k", [(8, 1), (8, 8), (688, 344), (1000, 999), (11008, 5504), (24576, 12288),
                                    (24576, 1), (4099, 2000)])
def test_topk_exact(d_ff, k):
    g = torch.Generator().manual_seed(d_ff + k)
    s = torch.rand((3, d_ff), generator=g)
    s[1] = torch.round(s[1] * 8) / 8          # many exact ties
    s[2] = 0.5                                 # all equal -> lowest indices
    s[2, -1] = 0.0
    e = torch.empty((3, k), device=dev(), dtype=torch.int32)
    G.griffin_select_topk(s.to(dev()), k, e)
    e = e.cpu().numpy()
    for i in range(3):
        assert np.array_equal(e[i], O.select_topk(s[i].double().numpy(), k)), i


def test_topk_negative_and_zero_scores():
    s = torch.tensor([[-1.0, 0.0, -0.0, 2.0, -3.0, 0.0, 1e-30, -1e-30]])
    for k in range(1, 9):
        e = torch.empty((1, k), device=dev(), dtype=torch.int32)
        G.griffin_select_topk(s.to(dev()), k, e)
        assert np.array_equal(e.cpu().numpy()[0], O.select_topk(s[0].double().numpy(), k)), k


def test_combine_scores():
    g = torch.Generator().manual_seed(5)
    s = torch.rand((5, 1000), generator=g)
    lens = [3, 64, 512, 7, 1]
    out = torch.empty((1000,), device=dev())
    G.griffin_combine_scores(s.to(dev()), lens, out)
    ref = O.combine_scores([r for r in s.double().numpy()], lens)
    assert np.max(np.abs(np64(out) - ref) / ref) < 1e-6


# ------------------------------------------------------------- compaction ---

@pytest.mark.parametrize("source", ["row_major", "neuron_major"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,d_ff,k", [(64, 96, 37), (256, 688, 344), (1024, 2816, 1408), (520, 1032, 1032),
                                      (72, 200, 1), (136, 30008, 15001),   # rows of W_2 too long for shared memory
                                      (4096, 11008, 5504)])
def test_compact_exact(dtype, d, d_ff, k, source):
    """Slicing (Section 4.2) is indexing: raw-bit equality with W[E, :] and W[:, E], from the row-major W_2 and
    from its transpose.  The index list is unsorted for the small shapes and starts at an address that is not a
    multiple of 8 bytes when k is odd."""
    L, host = make_layer(d, d_ff, dtype, bias=True, seed=d + k)
    rs = np.random.default_rng(k)
    e_np = rs.choice(d_ff, size=k, replace=False).astype(np.int32)
    if d_ff > 1100:
        e_np = np.sort(e_np)
    e = torch.from_numpy(np.concatenate([[0], e_np]).astype(np.int32)).to(dev())[1:]   # 4 bytes off an aligned address
    cs = L.compact(e) if source == "row_major" else L.compact_nm(e)
    assert L.status() == G.OK
    g, u, dn, bg, bu = cs._keep
    ref = O.compact_experts(e_np, host["wg"].numpy() if dtype == "f32" else host["wg"].view(torch.int16).numpy(),
                            host["wu"].numpy() if dtype == "f32" else host["wu"].view(torch.int16).numpy(),
                            host["wd"].numpy() if dtype == "f32" else host["wd"].view(torch.int16).numpy(),
                            host["bg"].numpy() if dtype == "f32" else host["bg"].view(torch.int16).numpy(),
                            host["bu"].numpy() if dtype == "f32" else host["bu"].view(torch.int16).numpy())
    bits = (lambda t: t.cpu().numpy()) if dtype == "f32" else (lambda t: t.cpu().view(torch.int16).numpy())
    assert np.array_equal(bits(g), ref["w_gate"])
    assert np.array_equal(bits(u), ref["w_up"])
    assert np.array_equal(bits(dn)[:, :k], ref["w_down"])
    assert np.all(bits(dn)[:, k:] == 0)                       # padding columns are zero
    assert np.array_equal(bits(bg), ref["b_gate"]) and np.array_equal(bits(bu), ref["b_up"])


@pytest.mark.parametrize("source,d_ff", [("row_major", 96), ("neuron_major", 96), ("row_major", 40000)])
def test_compact_out_of_range_index_is_reported_not_read(source, d_ff):
    L, host = make_layer(64, d_ff, "bf16")
    e = torch.tensor([0, 5, d_ff, 7, -1], dtype=torch.int32, device=dev())   # d_ff and -1 are out of range
    cs = L.compact(e) if source == "row_major" else L.compact_nm(e)
    assert L.status() == G.ERR_INVALID_ARG
    g, dn = cs._keep[0].cpu(), cs._keep[2].cpu()
    assert torch.all(g[2] == 0) and torch.all(g[4] == 0) and torch.equal(g[1], host["wg"][5])
    assert torch.all(dn[:, 2] == 0) and torch.all(dn[:, 4:] == 0) and torch.equal(dn[:, 3], host["wd"][:, 7])
    G.griffin_workspace_init(L.ws)
    assert L.status() == G.OK


# ----------------------------------------------------------------- decode ---

DECODE_SHAPES = [
    # d, d_ff, k, B
    (256, 688, 344, 1),      # the tiny workload
    (64, 96, 37, 3),         # odd k -> padded ldk, several sequences
    (1000, 1504, 751, 2),    # d not a multiple of the vector tiling
    (2048, 5632, 2816, 1),
    (3072, 4096, 4096, 1),   # k = d_ff
    (4096, 11008, 5504, 1),  # Llama-2-7B shape
    (5120, 2048, 1024, 8),   # widest d of the workloads, batch 8
    (8192, 1024, 512, 1),    # largest supported d
    (512, 9008, 9008, 1),    # rows of W_2_hat longer than one stage chunk (two chunks)
    (256, 20000, 16400, 2),  # three chunks per row, two sequences
    (5120, 13824, 6912, 3),  # Llama-2-13B shape; with 3 sequences the CTAs' ranges of the register stream straddle them
    (256, 688, 344, 32),     # the largest batch
    (128, 64, 1, 2),         # one expert: most CTAs have nothing to do in the first half
    (136, 200, 9, 5),        # rows shorter than one step, odd k, more sequences than pairs per CTA
    (3136, 4800, 4736, 8),   # 16 pairs per warp in the first half: the register stream hands the last 8 % out at run time
]

# The two warp-level kernels for sequences with their own sets (bf16), and the choice by size.
DECODE_KERNELS = {"by_size": 0, "ring": G.DECODE_RING, "stream": G.DECODE_STREAM}


@pytest.mark.parametrize("dtype,kernel", [("f32", "by_size"), ("bf16", "by_size"), ("bf16", "ring"), ("bf16", "stream")])
@pytest.mark.parametrize("d,d_ff,k,B", DECODE_SHAPES)
def test_decode_matches_oracle(dtype, kernel, d, d_ff, k, B):
    kf = DECODE_KERNELS[kernel]
    act = {3072: "geglu_tanh", 2048: "geglu_erf", 1000: "reglu"}.get(d, "swiglu")
    L, host = make_layer(d, d_ff, dtype, act=act, bias=(d_ff < 2000), seed=d + k, n_seq=B)
    rs = np.random.default_rng(d + k)
    x = rand((B, d), TD[dtype], 99)
    sets, refs = [], []
    for b in range(B):
        e_np = np.sort(rs.choice(d_ff, size=k, replace=False)).astype(np.int32)
        sets.append(L.compact(torch.from_numpy(e_np).to(dev())))
        c = O.compact_experts(e_np, h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), h64(host, "bg"), h64(host, "bu"))
        refs.append(O.ff_pruned(np64(x[b]), c, act, h64(host, "bd")))
    y = L.decode(sets, x, kf)
    y2 = L.decode(sets, x, kf | G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    y3 = L.decode(sets, x, kf | G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    assert L.status() == G.OK
    for b in range(B):
        assert_output(np64(y[b]), refs[b], dtype, b)
    assert torch.equal(y, y2) and torch.equal(y, y3)   # deterministic, launch mode does not matter


def test_decode_kernels_take_turns_on_one_workspace():
    """The ring kernel and the register-streaming kernel keep separate meeting-point counters in the
    workspace header, so calls of the two may alternate in any order."""
    d, d_ff, k, B = 1024, 2816, 1408, 3
    L, host = make_layer(d, d_ff, "bf16", seed=21, n_seq=B)
    rs = np.random.default_rng(21)
    sets = [L.compact(torch.from_numpy(np.sort(rs.choice(d_ff, size=k, replace=False)).astype(np.int32)).to(dev()))
            for _ in range(B)]
    x = rand((B, d), torch.bfloat16, 22)
    first = {}
    for kernel in ["ring", "stream", "stream", "ring", "stream", "ring", "ring", "stream"]:
        y = L.decode(sets, x, DECODE_KERNELS[kernel] | G.DECODE_OVERLAP_WEIGHT_PREFETCH)
        assert torch.equal(first.setdefault(kernel, y), y)
    assert L.status() == G.OK
    # the two sum in different orders: close, not equal
    assert_output(np64(first["stream"]), np64(first["ring"]), "bf16")


def test_decode_rejects_both_kernel_flags_at_once():
    L, host = make_layer(256, 688, "bf16")
    cs = L.compact(torch.arange(0, 688, 2, dtype=torch.int32, device=dev()))
    with pytest.raises(G.GriffinError) as err:
        L.decode([cs], rand((1, 256), torch.bfloat16, 1), G.DECODE_RING | G.DECODE_STREAM)
    assert err.value.status == G.ERR_INVALID_ARG


# Shapes that the opt-in tcgen05 kernel takes (d and ldk multiples of 128) and two that it hands
# back to the warp-level kernel (ldk = 344; d = 1000).
TCGEN05_SHAPES = [
    # d, d_ff, k, B
    (128, 256, 128, 1),      # a single 256-byte window per row of W_g_hat; fewer rows than CTAs
    (2048, 5632, 2816, 1),
    (3072, 4096, 4096, 1),   # k = d_ff, GEGLU
    (4096, 11008, 5504, 1),  # Llama-2-7B shape: rows of W_2_hat end in a short piece
    (5120, 2048, 1024, 8),   # batch 8: several work items per CTA, the vector changes between them
    (8192, 1024, 512, 3),    # largest supported d; rows of W_2_hat shorter than a batch of windows
    (1024, 3000, 1500, 2),   # k not a multiple of 8: ldk = 1504 is not a multiple of 128 either -> warp-level kernel
    (256, 688, 344, 1),      # falls back as well
]


@pytest.mark.parametrize("d,d_ff,k,B", TCGEN05_SHAPES)
def test_decode_tcgen05_kernel_matches_oracle_and_default_kernel(d, d_ff, k, B):
    act = "geglu_tanh" if d == 3072 else "swiglu"
    L, host = make_layer(d, d_ff, "bf16", act=act, bias=(d_ff < 2500), seed=3 * d + k, n_seq=B)
    rs = np.random.default_rng(d + k)
    x = rand((B, d), torch.bfloat16, 98)
    sets, refs = [], []
    for b in range(B):
        e_np = np.sort(rs.choice(d_ff, size=k, replace=False)).astype(np.int32)
        sets.append(L.compact(torch.from_numpy(e_np).to(dev())))
        c = O.compact_experts(e_np, h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), h64(host, "bg"), h64(host, "bu"))
        refs.append(O.ff_pruned(np64(x[b]), c, act, h64(host, "bd")))
    y_tc = L.decode(sets, x, G.DECODE_TCGEN05)
    y_tc2 = L.decode(sets, x, G.DECODE_TCGEN05 | G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    y_warp = L.decode(sets, x)
    y_tc3 = L.decode(sets, x, G.DECODE_TCGEN05 | G.DECODE_OVERLAP_WEIGHT_PREFETCH)   # after the other kernel used the workspace
    assert L.status() == G.OK
    for b in range(B):
        assert_output(np64(y_tc[b]), refs[b], "bf16", b)
        assert_output(np64(y_tc[b]), np64(y_warp[b]), "bf16", b, scale=2.0)
    assert torch.equal(y_tc, y_tc2) and torch.equal(y_tc, y_tc3)   # deterministic, launch mode does not matter


# One expert set for all sequences of a call (Eq. 7): d, d_ff, k, B, activation, biases
SHARED_SET_SHAPES = [
    (512, 1536, 768, 2, "geglu_tanh", True),
    (4096, 11008, 5504, 3, "swiglu", False),   # an odd number of vectors
    (4096, 11008, 5504, 8, "swiglu", False),   # the most that one call streams together
    (2048, 5632, 2816, 5, "reglu", True),
    (1024, 2816, 1408, 2, "geglu_erf", True),
    (8192, 1024, 512, 8, "swiglu", False),     # the widest rows: shorter chunks make room for the eight vectors
    (1000, 1504, 751, 4, "swiglu", False),     # rows that end inside a block of four units; odd k
    (4096, 11008, 11008, 8, "swiglu", False),  # the unpruned block: eight vectors of 22 KB, taken in two passes of four
    (1024, 2816, 1408, 11, "swiglu", True),    # more than eight sequences: a pass of eight and a pass of three
    (64, 96, 37, 2, "reglu", True),            # fewer neurons than CTAs: most work items are empty
    (2048, 8192, 4000, 6, "relu", True),       # a block without a gate (Eq. 2)
    (1024, 4096, 2048, 8, "gelu_tanh", False),  # ... and another
    (5120, 13824, 6912, 8, "swiglu", False),   # Llama-2-13B shape: rows of 10 KB and 13.5 KB in three and four chunks
    (3072, 24576, 12288, 8, "geglu_tanh", False),  # Gemma shape: eight vectors of 24 KB do not fit, two passes of four
    (4096, 14336, 3584, 4, "swiglu", False),   # Mistral shape at keep 0.25
]


@pytest.mark.parametrize("d,d_ff,k,B,act,bias", SHARED_SET_SHAPES)
def test_decode_with_one_shared_set_matches_oracle_and_separate_calls(d, d_ff, k, B, act, bias):
    L, host = make_layer(d, d_ff, "bf16", act=act, bias=bias, seed=7 * d + k, n_seq=B)
    rs = np.random.default_rng(d + k + B)
    x = rand((B, d), torch.bfloat16, 97)
    e_np = np.sort(rs.choice(d_ff, size=k, replace=False)).astype(np.int32)
    cs = L.compact(torch.from_numpy(e_np).to(dev()))
    c = O.compact_experts(e_np, h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), h64(host, "bg"), h64(host, "bu"))
    ref = O.ff_pruned(np64(x), c, act, h64(host, "bd"))
    y = L.decode([cs] * B, x)
    y2 = L.decode([cs] * B, x, G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    y3 = L.decode([cs] * B, x)
    assert L.status() == G.OK
    assert torch.equal(y, y2) and torch.equal(y, y3)     # bitwise reproducible
    for b in range(B):
        assert_output(np64(y[b]), ref[b], "bf16", b)
        y1 = L.decode([cs], x[b:b + 1])   # the same sequence on its own
        assert_output(np64(y[b]), np64(y1[0]), "bf16", b, scale=2.0)
    # the opt-in tcgen05 kernel has a shared-set mode of its own (gated blocks, 2..8 sequences, whole windows);
    # where it does not apply the flag changes nothing
    yt = L.decode([cs] * B, x, G.DECODE_TCGEN05)
    assert L.status() == G.OK
    for b in range(B):
        assert_output(np64(yt[b]), ref[b], "bf16", ("tcgen05", b))


# Decode straight from the full weights through the index list: d, d_ff, k, B, activation, biases
INDEXED_SHAPES = [
    (256, 688, 344, 1, "swiglu", True),        # the tiny workload's shape
    (64, 96, 37, 3, "reglu", True),            # fewer experts than CTAs: most slices are empty
    (1000, 1504, 751, 2, "geglu_erf", True),   # rows that end inside a block of 32 units
    (2048, 5632, 2816, 1, "swiglu", False),
    (256, 20000, 16400, 2, "geglu_tanh", False),   # two work items per CTA and sequence
    (4096, 11008, 5504, 1, "swiglu", False),   # Llama-2-7B shape
    (4096, 11008, 5504, 4, "swiglu", False),   # the final sum takes four columns per lane
    (5120, 2048, 1024, 8, "swiglu", True),     # one pair per stage, batch 8
    (8192, 1024, 512, 2, "swiglu", False),     # largest supported d
    (512, 1536, 1536, 2, "geglu_tanh", True),  # every neuron, in a shuffled order
]


@pytest.mark.parametrize("d,d_ff,k,B,act,bias", INDEXED_SHAPES)
def test_decode_indexed_matches_oracle_and_compact_path(d, d_ff, k, B, act, bias):
    L, host = make_layer(d, d_ff, "bf16", act=act, bias=bias, seed=5 * d + k, n_seq=B)
    rs = np.random.default_rng(d + k + B)
    x = rand((B, d), torch.bfloat16, 96)
    idx = np.empty((B, k), dtype=np.int32)
    refs = []
    for b in range(B):
        e_np = rs.choice(d_ff, size=k, replace=False).astype(np.int32)
        idx[b] = e_np if b % 2 else np.sort(e_np)       # the order of the list must not matter
        c = O.compact_experts(idx[b], h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), h64(host, "bg"), h64(host, "bu"))
        refs.append(O.ff_pruned(np64(x[b]), c, act, h64(host, "bd")))
    e = torch.from_numpy(idx).to(dev())
    y = L.decode_indexed(e, x)
    y2 = L.decode_indexed(e, x, G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    y3 = L.decode_indexed(e, x, G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    assert L.status() == G.OK
    assert torch.equal(y, y2) and torch.equal(y, y3)    # deterministic, launch mode does not matter
    for b in range(B):
        assert_output(np64(y[b]), refs[b], "bf16", b)
    if B <= 2:   # the compact-set kernels on the same indices
        y_c = L.decode([L.compact(e[b]) for b in range(B)], x)
        assert_output(np64(y), np64(y_c), "bf16", scale=2.0)


def test_decode_indexed_out_of_range_index_is_reported_not_read():
    d, d_ff = 256, 688
    L, host = make_layer(d, d_ff, "bf16", seed=77)
    good = np.arange(0, 600, 2, dtype=np.int32)
    bad = good.copy()
    bad[7], bad[100] = d_ff, -3
    x = rand((1, d), torch.bfloat16, 95)
    y = L.decode_indexed(torch.from_numpy(bad).to(dev()), x)
    assert L.status() == G.ERR_INVALID_ARG
    G.griffin_workspace_init(L.ws)
    # the two bad entries contribute nothing: the result is that of the list without them
    keep = np.delete(good, [7, 100])
    c = O.compact_experts(keep, h64(host, "wg"), h64(host, "wu"), h64(host, "wd"))
    assert_output(np64(y[0]), O.ff_pruned(np64(x[0]), c, "swiglu"), "bf16")
    assert L.status() == G.OK


def test_decode_indexed_rejects_fp32_storage():
    L, _ = make_layer(64, 96, "f32")
    e = torch.arange(8, dtype=torch.int32, device=dev())
    with pytest.raises(G.GriffinError) as err:
        L.decode_indexed(e, rand((1, 64), torch.float32, 1))
    assert err.value.status == G.ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_decode_with_all_neurons_is_the_dense_ff(dtype):
    d, d_ff = 512, 1536
    L, host = make_layer(d, d_ff, dtype, act="geglu_tanh", bias=True, n_seq=2)
    x = rand((2, d), TD[dtype], 3)
    y = L.decode([L.dense_set(), L.dense_set()], x)
    ref, _ = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), "geglu_tanh",
                        h64(host, "bg"), h64(host, "bu"), h64(host, "bd"))
    assert_output(np64(y), ref, dtype)
    # and the compacted copy of E = everything gives the same bits as the aliased weights
    cs = L.compact(torch.arange(d_ff, dtype=torch.int32, device=dev()))
    assert torch.equal(L.decode([cs, cs], x), y)


@pytest.mark.parametrize("kernel", ["ring", "stream"])
def test_decode_many_steps_back_to_back_with_overlap(kernel):
    d, d_ff, k = 1024, 2816, 1408
    L, host = make_layer(d, d_ff, "bf16")
    e_np = np.arange(0, d_ff, 2, dtype=np.int32)
    cs = L.compact(torch.from_numpy(e_np).to(dev()))
    xs = rand((16, d), torch.bfloat16, 11).to(dev())
    ys = torch.empty_like(xs)
    arr = G.compact_array([cs])
    torch.cuda.synchronize()
    for t in range(16):
        G.griffin_ff_decode(L.desc, arr, None, xs[t:t + 1], ys[t:t + 1], L.ws,
                            G.DECODE_OVERLAP_WEIGHT_PREFETCH | DECODE_KERNELS[kernel])
    assert L.status() == G.OK
    c = O.compact_experts(e_np, h64(host, "wg"), h64(host, "wu"), h64(host, "wd"))
    ref = O.ff_pruned(np64(xs), c, "swiglu")
    assert_output(np64(ys), ref, "bf16")


@pytest.mark.parametrize("kernel", ["ring", "stream"])
def test_decode_calls_replayed_from_a_cuda_graph_give_the_same_bits(kernel):
    """bench.py captures the decode calls of a step once and replays them: same kernels, same
    launch attributes (the overlapped-launch edges included), so the same bits."""
    d, d_ff, k, n = 1024, 2816, 1408, 6
    L, host = make_layer(d, d_ff, "bf16", seed=5)
    cs = L.compact(torch.arange(0, d_ff, 2, dtype=torch.int32, device=dev()))
    arr = G.compact_array([cs])
    xs = rand((n, d), torch.bfloat16, 12).to(dev())
    y_direct, y_graph = torch.empty_like(xs), torch.zeros_like(xs)

    def calls(out):
        for t in range(n):
            G.griffin_ff_decode(L.desc, arr, None, xs[t:t + 1], out[t:t + 1], L.ws,
                                (G.DECODE_OVERLAP_WEIGHT_PREFETCH if t > 0 else G.DECODE_DEFAULT) | DECODE_KERNELS[kernel])

    calls(y_direct)
    torch.cuda.synchronize()
    g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            calls(y_graph)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        y_graph.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(y_graph, y_direct)
    assert L.status() == G.OK


# ---------------------------------------------------------------- prefill ---

PREFILL_SHAPES = [(64, 256, 688), (1, 64, 96), (37, 72, 200), (130, 512, 1032), (256, 1024, 2816)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("act", ["swiglu", "geglu_tanh", "reglu", "geglu_erf"])
@pytest.mark.parametrize("S,d,d_ff", PREFILL_SHAPES)
def test_prefill_score_matches_oracle(dtype, act, S, d, d_ff):
    L, host = make_layer(d, d_ff, dtype, act=act, bias=(S == 37), seed=S + d, S_max=S)
    x = rand((S, d), TD[dtype], 5) + rand((1, d), TD[dtype], 6, 4.0 / d ** 0.5)
    y, s = L.prefill(x)
    ref_y, ref_z = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), act,
                              h64(host, "bg"), h64(host, "bu"), h64(host, "bd"))
    ref_s = O.flock_score(ref_z)
    assert_output(np64(y), ref_y, dtype)
    s = np64(s)
    assert np.all(np.abs(s - ref_s) <= score_tol(dtype) * ref_s + 1e-6 * np.sqrt(S / d_ff))
    assert abs(float(np.sum(s * s)) - S) < 1e-5 * S     # rows of Zbar are unit vectors
    _, s2 = L.prefill(x, want_y=False)
    assert np.array_equal(np64(s2), s)                   # deterministic; y is optional


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("pieces,d,d_ff", [((100, 37, 119), 512, 1032), ((1, 1, 62), 256, 688), ((300,), 1024, 2816),
                                           ((128, 128, 128, 128, 50), 1024, 2816)])
def test_prefill_fed_piece_by_piece_gives_the_statistic_of_the_whole_prompt(dtype, pieces, d, d_ff):
    """s_j^2 is a sum over tokens (Eq. 6): the pieces' sums of squares add up to the whole prompt's."""
    S = sum(pieces)
    L, host = make_layer(d, d_ff, dtype, act="swiglu", bias=(d == 512), seed=S + d, S_max=S)
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
    ref_y, ref_z = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), "swiglu",
                              h64(host, "bg"), h64(host, "bu"), h64(host, "bd"))
    ref_s = O.flock_score(ref_z)
    assert_output(np64(y), ref_y, dtype)
    s = np64(score)
    assert np.all(np.abs(s - ref_s) <= score_tol(dtype) * ref_s + 1e-6 * np.sqrt(S / d_ff))
    assert abs(float(np.sum(s * s)) - S) < 1e-5 * S
    assert np.allclose(np64(sumsq), s * s, rtol=1e-6, atol=0)
    _, s_whole = L.prefill(x)                                       # one call on the whole prompt
    assert np.allclose(np64(s_whole), s, rtol=2 * score_tol(dtype), atol=1e-6 * np.sqrt(S / d_ff))


@pytest.mark.parametrize("S,d,d_ff", [(256, 1024, 10240), (200, 2048, 9728)])
def test_prefill_with_a_cut_last_round_of_tiles(S, d, d_ff):
    """160 (152) tiles of the first GEMM on 148 SMs: the last 12 (4) are cut along K into parts
    whose partial accumulators meet in the finishing kernel."""
    L, host = make_layer(d, d_ff, "bf16", act="geglu_tanh", bias=True, seed=S + d_ff, S_max=S)
    x = rand((S, d), torch.bfloat16, 15) + rand((1, d), torch.bfloat16, 16, 4.0 / d ** 0.5)
    y, s = L.prefill(x)
    ref_y, ref_z = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), "geglu_tanh",
                              h64(host, "bg"), h64(host, "bu"), h64(host, "bd"))
    ref_s = O.flock_score(ref_z)
    assert L.status() == G.OK
    assert_output(np64(y), ref_y, "bf16")
    s = np64(s)
    assert np.all(np.abs(s - ref_s) <= score_tol("bf16") * ref_s + 1e-6 * np.sqrt(S / d_ff))
    assert abs(float(np.sum(s * s)) - S) < 1e-5 * S
    _, s2 = L.prefill(x, want_y=False)
    assert np.array_equal(np64(s2), s)


def test_prefill_down_projection_with_a_cut_last_round_of_tiles():
    """160 tiles of the second GEMM (5 row blocks x 32 blocks of 256 outputs) on 148 SMs: the last 12 are
    cut along K into four parts whose partial accumulators meet in a finishing kernel."""
    S, d, d_ff = 640, 8192, 1024
    L, host = make_layer(d, d_ff, "bf16", act="swiglu", bias=True, seed=S + d_ff, S_max=S)
    x = rand((S, d), torch.bfloat16, 17) + rand((1, d), torch.bfloat16, 18, 4.0 / d ** 0.5)
    y, s = L.prefill(x)
    ref_y, ref_z = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), "swiglu",
                              h64(host, "bg"), h64(host, "bu"), h64(host, "bd"))
    assert L.status() == G.OK
    y = np64(y)
    assert_output(y, ref_y, "bf16")
    for r0, c0 in ((0, 0), (512, 7936), (639, 8191 - 255)):      # whole tiles and cut ones, corner by corner
        blk = (slice(r0, min(S, r0 + 128)), slice(c0, c0 + 256))
        assert_output(y[blk], ref_y[blk], "bf16")
    ref_s = O.flock_score(ref_z)
    assert np.all(np.abs(np64(s) - ref_s) <= score_tol("bf16") * ref_s + 1e-6 * np.sqrt(S / d_ff))


def test_prefill_zero_row_contributes_nothing():
    S, d, d_ff = 16, 64, 96
    L, host = make_layer(d, d_ff, "f32", S_max=S)
    x = rand((S, d), torch.float32, 8)
    x[3] = 0.0
    y, s = L.prefill(x)
    s = np64(s)
    assert np.all(np.isfinite(s)) and abs(float(np.sum(s * s)) - (S - 1)) < 1e-4 * S
    _, z = O.ff_dense(np64(x), h64(host, "wg"), h64(host, "wu"), h64(host, "wd"), "swiglu")
    assert np.max(np.abs(s - O.flock_score(z))) < 1e-5
    assert torch.all(y[3] == 0)


def test_device_status_word_is_decoded():
    # what a kernel leaves in the workspace header after a bounded wait gave up, or after it met a
    # bad expert index, comes back as a status code; re-initialising the workspace clears it
    L, _ = make_layer(64, 96, "bf16")
    hdr = L.ws[:16].view(torch.int32)
    assert L.status() == G.OK
    hdr[0] = 1
    assert L.status() == G.ERR_TIMEOUT
    hdr[0] = 2
    assert L.status() == G.ERR_INVALID_ARG
    hdr[0] = 77
    assert L.status() == G.ERR_CUDA
    G.griffin_workspace_init(L.ws)
    assert L.status() == G.OK and int(hdr[2]) == 0 and int(hdr[3]) == 0
