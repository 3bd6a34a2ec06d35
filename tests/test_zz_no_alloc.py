"""griffin_ff_decode_static: the decode call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: a plug-in inside a server that
owns the whole memory budget, or a latency-critical loop that must not take the allocator's
lock or the device-wide synchronisation that comes with it.  For them the library carries its
own fixed scratch array.  This test drives that entry point through the C ABI and checks that
it gives what griffin_ff_decode gives with a caller-owned workspace, on two calls in a row
(the second call finds the first call's leftovers in the shared array and must not care).
The file is named so that pytest collects it last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2404_01365_b200 import binding as G

pytestmark = pytest.mark.gpu


def _layer(d, d_ff, k, B, dtype, seed):
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(seed)
    rnd = lambda shape, s: (torch.randn(shape, generator=g) * s).to(dtype).to(dev)
    wg, wu, wd = rnd((d_ff, d), d ** -0.5), rnd((d_ff, d), d ** -0.5), rnd((d, d_ff), d_ff ** -0.5)
    desc = G.make_desc(d, d_ff, "swiglu", "f32" if dtype == torch.float32 else "bf16")
    weights = G.make_weights(wg, wu, wd)
    ws = G.alloc_workspace(desc, 0, B, dev)
    sets = []
    for b in range(B):
        e = torch.sort(torch.randperm(d_ff, generator=g)[:k]).values.to(torch.int32).to(dev)
        cs = G.alloc_compact(desc, k, dev, dtype)
        G.griffin_compact_experts(desc, weights, e, cs, ws)
        sets.append(cs)
    xs = [rnd((B, d), 1.0) for _ in range(2)]
    return desc, sets, ws, xs


@pytest.mark.parametrize("dtype,tol", [(torch.bfloat16, 2e-2), (torch.float32, 1e-4)])
def test_static_scratch_decode_matches_workspace_decode_twice(dtype, tol):
    desc, sets, ws, xs = _layer(1024, 2816, 1401, 3, dtype, seed=5)   # odd k: padded ldk
    arr = G.compact_array(sets)
    for x in xs:                                   # two calls in a row on the shared array
        y_ref, y = torch.empty_like(x), torch.empty_like(x)
        G.griffin_ff_decode(desc, arr, None, x, y_ref, ws)
        G.griffin_ff_decode_static(desc, arr, None, x, y)
        torch.cuda.synchronize()
        a, b = y.double().cpu().numpy(), y_ref.double().cpu().numpy()
        assert np.all(np.isfinite(a))
        assert np.linalg.norm(a - b) <= tol * np.linalg.norm(b)
    assert G.griffin_check_device_status(ws) == G.OK


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
