"""End-to-end parity of the whole path (prompt FF + statistic -> top-k -> compaction -> decode)
against the CPU oracle, driven through the same runner and launch configuration bench.py
times (decode calls with overlapped weight prefetch after the first step).

Small versions of every workload are checked in full; the full-size workloads are checked on
one block each (first, middle or last), all prompt rows, and decode steps {0, 1, T/2, T-1}.
"""
import numpy as np
import pytest
import torch

from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G, synth
from paper_2404_01365_b200.runner import FFStack
from gpu_util import check_expert_set, dev, np64, assert_output, score_tol

pytestmark = pytest.mark.gpu


def run_block(w, layer, keep, n_seq, oracle_seqs, steps):
    """One block of workload `w`: n_seq sequences on the GPU; the oracle follows the sequences
    in `oracle_seqs` through the prompt phase, and every sequence through the decode steps
    (with the expert set the GPU selected, so that decode is judged on its own)."""
    k = G.griffin_k_from_keep_ratio(w.d_ff, keep)
    assert k == O.k_from_keep_ratio(w.d_ff, keep)
    wg, wu, wd = synth.make_weights(w, layer)
    stack = FFStack(w.d, w.d_ff, w.act, w.dtype, 1, n_seq, w.S, k, dev())
    wg_d, wu_d, wd_d = None if wg is None else wg.to(dev()), wu.to(dev()), wd.to(dev())   # (no W_g without a gate)
    stack.add_block(wg_d, wu_d, wd_d)
    X = [synth.make_prompt(w, layer, q) for q in range(n_seq)]
    XD = torch.stack([synth.make_decode_inputs(w, layer, q) for q in range(n_seq)], 1)  # [T, n_seq, d]
    Y = torch.empty((n_seq, w.S, w.d), device=dev(), dtype=w.torch_dtype)
    for q in range(n_seq):
        stack.prefill_score(0, q, X[q].to(dev()), Y[q])
    stack.select_all()
    for q in range(n_seq):
        stack.compact(0, q)
    xd_dev = XD.to(dev())
    yd = torch.empty_like(xd_dev)
    for t in range(w.T):
        stack.decode(0, xd_dev[t], yd[t], overlap=t > 0)
    yd_ix = None
    if w.dtype == "bf16":   # the same steps without the compact sets: rows read in place through the index lists
        wn = G.make_weights_nm(wg_d, wu_d, wd_d.t().contiguous())
        yd_ix = torch.empty_like(xd_dev)
        for t in range(w.T):
            G.griffin_ff_decode_indexed(stack.desc, wn, stack.idx[0], xd_dev[t], yd_ix[t], stack.ws,
                                        G.DECODE_OVERLAP_WEIGHT_PREFETCH if t > 0 else G.DECODE_DEFAULT)
    assert stack.status() == G.OK
    E = stack.idx[0].cpu().numpy()
    S_gpu = np64(stack.score[0])

    wg64, wu64, wd64 = None if wg is None else np64(wg), np64(wu), np64(wd)
    swaps = 0
    for q in oracle_seqs:
        y_ref, z_ref = O.ff_dense(np64(X[q]), wg64, wu64, wd64, w.act)
        s_ref = O.flock_score(z_ref)
        assert_output(np64(Y[q]), y_ref, w.dtype, ("prefill output", q))
        tol = score_tol(w.dtype)
        assert np.all(np.abs(S_gpu[q] - s_ref) <= tol * s_ref + 1e-6 * np.sqrt(w.S / w.d_ff)), ("statistic", q)
        assert abs(float(np.sum(S_gpu[q] ** 2)) - w.S) < 1e-4 * w.S
        swaps += check_expert_set(E[q], s_ref, k)
    for q in range(n_seq):
        assert np.all(np.diff(E[q]) > 0) and E[q].min() >= 0 and E[q].max() < w.d_ff
        c = O.compact_experts(E[q], wg64, wu64, wd64)
        for t in steps:
            ref = O.ff_pruned(np64(XD[t, q]), c, w.act)
            assert_output(np64(yd[t, q]), ref, w.dtype, ("decode", q, t))
            if yd_ix is not None:
                assert_output(np64(yd_ix[t, q]), ref, w.dtype, ("index-direct decode", q, t))
    if n_seq > 1 and k < w.d_ff:   # each sequence picked its own experts
        assert any(not np.array_equal(E[0], E[q]) for q in range(1, n_seq))
    return swaps


def test_tiny_workload_in_full():
    w = synth.WORKLOADS["tiny_swiglu_f32"]
    swaps = run_block(w, 0, 0.5, 1, [0], range(w.T))
    assert swaps == 0      # fp32 end to end: the expert set is the oracle's


SMALL = {
    "llama2_7b": dict(d=512, d_ff=1376, S=96, T=6),
    "gemma_7b": dict(d=384, d_ff=3072, S=128, T=6),
    "llama2_13b": dict(d=640, d_ff=1728, S=160, T=4),
    "mistral_7b": dict(d=512, d_ff=1792, S=200, T=4),
    "opt_6p7b": dict(d=512, d_ff=2048, S=96, T=6),     # a ReLU block without a gate (Eq. 2)
}


@pytest.mark.parametrize("name", list(SMALL))
def test_small_versions_of_every_workload(name):
    base = synth.WORKLOADS[name]
    w = synth.scaled(base, **SMALL[name])
    for keep in base.keeps:
        for layer in (0, base.L - 1):
            run_block(w, layer, keep, base.B, range(base.B), range(w.T))


def test_stack_without_compact_sets():
    """The runner's index-direct mode: prompt phase, top-k, then decode straight from the full weights."""
    base = synth.WORKLOADS["llama2_7b"]
    w = synth.scaled(base, **SMALL["llama2_7b"])
    k = G.griffin_k_from_keep_ratio(w.d_ff, 0.5)
    wg, wu, wd = synth.make_weights(w, 0)
    stack = FFStack(w.d, w.d_ff, w.act, w.dtype, 1, 2, w.S, k, dev(), indexed=True)
    stack.add_block(wg.to(dev()), wu.to(dev()), wd.to(dev()))
    assert stack.sets == []
    X = [synth.make_prompt(w, 0, q) for q in range(2)]
    XD = torch.stack([synth.make_decode_inputs(w, 0, q) for q in range(2)], 1).to(dev())
    Y = torch.empty((2, w.S, w.d), device=dev(), dtype=w.torch_dtype)
    for q in range(2):
        stack.prefill_score(0, q, X[q].to(dev()), Y[q])
    stack.select_all()
    yd = torch.empty_like(XD)
    for t in range(w.T):
        stack.decode_indexed(0, XD[t], yd[t], overlap=t > 0)
    assert stack.status() == G.OK
    E = stack.idx[0].cpu().numpy()
    for q in range(2):
        c = O.compact_experts(E[q], np64(wg), np64(wu), np64(wd))
        for t in range(w.T):
            assert_output(np64(yd[t, q]), O.ff_pruned(np64(XD[t, q]), c, w.act), w.dtype, (q, t))


def _steps(T):
    return sorted({0, 1, T // 2, T - 1})


def test_full_size_llama2_7b_blocks():
    w = synth.WORKLOADS["llama2_7b"]
    for layer in (0, w.L // 2, w.L - 1):
        run_block(w, layer, 0.5, 1, [0], _steps(w.T))


def test_full_size_opt_6p7b_block_without_a_gate():
    w = synth.WORKLOADS["opt_6p7b"]
    run_block(w, 1, 0.5, 1, [0], _steps(w.T))


def test_full_size_gemma_7b_block():
    w = synth.WORKLOADS["gemma_7b"]
    run_block(w, w.L - 1, 0.5, 1, [0], _steps(w.T))


def test_full_size_llama2_13b_block_batch8():
    w = synth.WORKLOADS["llama2_13b"]
    # 8 sequences with 8 distinct expert sets decoded together; the oracle follows the prompt
    # phase of two of them (0.87 TFLOP of fp64 each) and the decode of all eight
    run_block(w, w.L // 2, 0.5, w.B, [0, w.B - 1], _steps(w.T))


@pytest.mark.parametrize("keep", [0.25, 0.5, 0.75, 1.0])
def test_full_size_mistral_7b_block_keep_sweep(keep):
    w = synth.WORKLOADS["mistral_7b"]
    run_block(w, 0, keep, w.B, [0] if keep != 0.5 else [0, 3], _steps(w.T))


def test_shared_expert_set_for_a_batch():
    """Batched GRIFFIN as the paper extends it (Eq. 7): the samples' statistics are combined into
    s_bar = sum_i s_i / sqrt(S_i), ONE expert set is selected and every sequence decodes with
    it (the same compact set passed for each sequence of the decode call)."""
    w = synth.scaled(synth.WORKLOADS["mistral_7b"], d=512, d_ff=1792, T=3)
    lengths = [200, 64, 131, 17]
    n_seq, k = len(lengths), G.griffin_k_from_keep_ratio(w.d_ff, 0.5)
    wg, wu, wd = synth.make_weights(w, 0)
    stack = FFStack(w.d, w.d_ff, w.act, w.dtype, 1, n_seq, max(lengths), k, dev())
    wg_d, wu_d, wd_d = wg.to(dev()), wu.to(dev()), wd.to(dev())
    stack.add_block(wg_d, wu_d, wd_d)
    wg64, wu64, wd64 = np64(wg), np64(wu), np64(wd)
    s_ref = []
    for q, S in enumerate(lengths):
        x = synth.make_prompt(w, 0, q, S=S)
        y = torch.empty((S, w.d), device=dev(), dtype=w.torch_dtype)
        stack.prefill_score(0, q, x.to(dev()), y)
        _, z = O.ff_dense(np64(x), wg64, wu64, wd64, w.act)
        s_ref.append(O.flock_score(z))
    s_bar = torch.empty((w.d_ff,), device=dev(), dtype=torch.float32)
    G.griffin_combine_scores(stack.score[0], lengths, s_bar)
    s_bar_ref = O.combine_scores(s_ref, lengths)
    assert np.max(np.abs(np64(s_bar) - s_bar_ref) / s_bar_ref) < 1e-4
    e = torch.empty((k,), device=dev(), dtype=torch.int32)
    G.griffin_select_topk(s_bar, k, e)
    check_expert_set(e.cpu().numpy(), s_bar_ref, k)
    shared = stack.sets[0][0]
    G.griffin_compact_experts(stack.desc, stack.weights[0], e, shared, stack.ws)
    xd = torch.stack([synth.make_decode_inputs(w, 0, q)[0] for q in range(n_seq)])
    yd = torch.empty((n_seq, w.d), device=dev(), dtype=w.torch_dtype)
    G.griffin_ff_decode(stack.desc, [shared] * n_seq, None, xd.to(dev()), yd, stack.ws)
    assert stack.status() == G.OK
    c = O.compact_experts(e.cpu().numpy(), wg64, wu64, wd64)
    ref = O.ff_pruned(np64(xd), c, w.act)
    for q in range(n_seq):
        assert_output(np64(yd[q]), ref[q], w.dtype)
