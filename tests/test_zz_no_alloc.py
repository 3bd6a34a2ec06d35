"""griffin_ff_decode_static: the decode call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: a plug-in inside a server that
owns the whole memory budget, or a latency-critical loop that must not take the allocator's
lock or the device-wide synchronisation that comes with it.  For them the library carries its
own fixed scratch array.  This test drives that entry point through the C ABI and checks that
it gives what griffin_ff_decode gives with a caller-owned workspace -- and what the CPU oracle
gives -- on two calls in a row (the second call finds the first call's leftovers in the shared
array and must not care), and that the device's free memory is the same before and after.
The file is named so that pytest collects it last.
"""
import ctypes as C

import pytest
import torch

from oracle import griffin_oracle as O
from out_check import assert_output
from paper_2404_01365_b200 import binding as G

pytestmark = pytest.mark.gpu


def _layer(d, d_ff, k, B, dtype, seed, act="swiglu", shared=False):
    """Weights of one block, B compact expert sets cut from them (one set named B times when `shared`), two
    batches of inputs, and the float64 copies the oracle needs."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(seed)
    host = lambda shape, s: (torch.randn(shape, generator=g) * s).to(dtype)
    gated = G.act_is_gated(act)
    wg = host((d_ff, d), d ** -0.5) if gated else None
    wu, wd = host((d_ff, d), d ** -0.5), host((d, d_ff), d_ff ** -0.5)
    desc = G.make_desc(d, d_ff, act, "f32" if dtype == torch.float32 else "bf16")
    up = lambda t: None if t is None else t.to(dev)
    weights = G.make_weights(up(wg), up(wu), up(wd))
    ws = G.alloc_workspace(desc, 0, B, dev)
    sets, experts = [], []
    for b in range(1 if shared else B):
        e = torch.sort(torch.randperm(d_ff, generator=g)[:k]).values.to(torch.int32)
        cs = G.alloc_compact(desc, k, dev, dtype)
        G.griffin_compact_experts(desc, weights, e.to(dev), cs, ws)
        sets.append(cs)
        experts.append(e.numpy())
    if shared:
        sets, experts = sets * B, experts * B
    xs = [host((B, d), 1.0) for _ in range(2)]
    f64 = lambda t: None if t is None else t.double().numpy()
    refs = [[O.ff_pruned(f64(x[b]), O.compact_experts(experts[b], f64(wg), f64(wu), f64(wd)), act) for b in range(B)]
            for x in xs]
    return desc, sets, ws, [x.to(dev) for x in xs], refs


def _two_calls_in_a_row(desc, sets, ws, xs, refs, dtype, flags=G.DECODE_DEFAULT):
    name = "f32" if dtype == torch.float32 else "bf16"
    arr = G.compact_array(sets)
    for i, x in enumerate(xs):                      # two calls in a row on the shared array
        y_ref, y = torch.empty_like(x), torch.empty_like(x)
        G.griffin_ff_decode(desc, arr, None, x, y_ref, ws, flags & ~G.DECODE_OVERLAP_WEIGHT_PREFETCH)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]  # cudaMemGetInfo: what the driver itself reports as free
        G.griffin_ff_decode_static(desc, arr, None, x, y, flags if i > 0 else flags & ~G.DECODE_OVERLAP_WEIGHT_PREFETCH)
        torch.cuda.synchronize()
        if i > 0:   # (a process's very first call may make the driver load the library's image, array included)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        for b in range(x.shape[0]):
            assert_output(y[b].double().cpu().numpy(), refs[i][b], name, ("oracle", i, b))
            assert_output(y[b].double().cpu().numpy(), y_ref[b].double().cpu().numpy(), name, ("workspace call", i, b),
                          scale=2.0)
    assert G.griffin_check_device_status(ws) == G.OK
    assert G.griffin_ff_decode_static_status() == G.OK


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_decode_matches_workspace_decode_twice(dtype):
    desc, sets, ws, xs, refs = _layer(1024, 2816, 1401, 3, dtype, seed=5)   # odd k: padded ldk
    _two_calls_in_a_row(desc, sets, ws, xs, refs, dtype)


@pytest.mark.parametrize("B", [2, 5, 8])
def test_static_scratch_decode_with_one_expert_set_for_the_batch(B):
    # every sequence names the same buffers: the weights are streamed once for all of them, and the CTAs of
    # that kernel meet through the counters in front of the static array
    desc, sets, ws, xs, refs = _layer(1024, 2816, 1408, B, torch.bfloat16, seed=11 + B, shared=True)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16)


def test_static_scratch_decode_through_the_tcgen05_kernel_and_with_overlapped_launches():
    desc, sets, ws, xs, refs = _layer(1024, 2816, 1408, 2, torch.bfloat16, seed=21)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16, flags=G.DECODE_TCGEN05)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16, flags=G.DECODE_OVERLAP_WEIGHT_PREFETCH)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16, flags=G.DECODE_TCGEN05 | G.DECODE_OVERLAP_WEIGHT_PREFETCH)


@pytest.mark.parametrize("kernel", [G.DECODE_RING, G.DECODE_STREAM])
def test_static_scratch_decode_through_either_warp_level_kernel(kernel):
    # both keep their meeting-point counter in the header in front of the static array
    desc, sets, ws, xs, refs = _layer(1024, 2816, 1401, 3, torch.bfloat16, seed=41)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16, flags=kernel)
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16, flags=kernel | G.DECODE_OVERLAP_WEIGHT_PREFETCH)


def test_static_scratch_decode_of_a_block_without_a_gate():
    desc, sets, ws, xs, refs = _layer(512, 2048, 1000, 2, torch.bfloat16, seed=31, act="relu")
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.bfloat16)


def test_static_scratch_decode_that_fills_the_array_exactly():
    # B * ldk * 4 bytes == GRIFFIN_STATIC_SCRATCH_BYTES: the largest call that is accepted
    B, k = 32, G.STATIC_SCRATCH_BYTES // (32 * 4)
    desc, sets, ws, xs, refs = _layer(128, k, k, B, torch.float32, seed=41, shared=True)
    assert B * sets[0].ldk * 4 == G.STATIC_SCRATCH_BYTES
    _two_calls_in_a_row(desc, sets, ws, xs, refs, torch.float32)


def test_static_scratch_rejects_what_does_not_fit():
    # B * ldk * 4 bytes beyond the array: refused on the host, nothing is launched
    desc = G.make_desc(256, 16384, "swiglu", "bf16")
    fake = C.c_void_p(0x10000)
    big = G.FFCompact(fake, fake, fake, None, None, 16384, 16384)
    sets = (G.FFCompact * 32)(*([big] * 32))
    assert 32 * 16384 * 4 > G.STATIC_SCRATCH_BYTES
    st = G.load().griffin_ff_decode_static(C.byref(desc), 32, sets, None, fake, fake, 0, None)
    assert st == G.ERR_UNSUPPORTED
    assert G.load().griffin_ff_decode_static(C.byref(desc), 0, sets, None, fake, fake, 0, None) == G.ERR_INVALID_ARG
