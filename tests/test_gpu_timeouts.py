"""What happens when a bounded device-side wait runs out (no healthy run ever gets there).

Every wait inside the kernels -- on a shared-memory barrier, on the grid-wide meeting counter -- gives up after
a fixed number of SM clock cycles, raises the workspace's status word and lets the kernel return; the host
then reads GRIFFIN_ERR_TIMEOUT from griffin_check_device_status.  The library exports a small self-test
(not in the public header) that drives the very primitive the kernels use to that give-up: a barrier on which
nobody arrives, with a limit of a fraction of a millisecond.  Nothing here hangs or faults the GPU: the wait
is bounded by construction, which is the property under test."""
import ctypes as C

import numpy as np
import pytest
import torch

from gpu_util import GpuLayer, assert_output, dev, np64, rand
from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G

pytestmark = pytest.mark.gpu


def _selftest(ws, limit_cycles):
    lib = G.load()
    fn = lib.griffin_selftest_wait_gives_up
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p]
    out = torch.zeros(2, dtype=torch.int64, device=dev())
    st = fn(C.c_void_p(ws.data_ptr()), limit_cycles, C.c_void_p(out.data_ptr()),
            C.c_void_p(torch.cuda.current_stream().cuda_stream))
    return st, out


def test_a_wait_that_nobody_ends_gives_up_reports_a_timeout_and_the_workspace_works_again_after_init():
    d, d_ff, k = 1024, 2816, 1408
    wg, wu, wd = rand((d_ff, d), torch.bfloat16, 1, d ** -0.5), rand((d_ff, d), torch.bfloat16, 2, d ** -0.5), \
        rand((d, d_ff), torch.bfloat16, 3, d_ff ** -0.5)
    L = GpuLayer(d, d_ff, "swiglu", "bf16", wg, wu, wd)
    assert L.status() == G.OK
    limit = 200_000                                        # about 0.1 ms of SM clocks
    st, out = _selftest(L.ws, limit)
    assert st == G.OK
    torch.cuda.synchronize()                               # the kernel returned: the wait was bounded
    gave_up, cycles = (int(v) for v in out.cpu())
    assert gave_up == 1
    # it waited the limit out, and not much more: the clock is only read between rounds of a few thousand
    # polls (each of which the hardware may hold for microseconds), so the give-up comes tens of milliseconds late
    assert limit < cycles < 400_000_000
    assert L.status() == G.ERR_TIMEOUT
    assert L.status() == G.ERR_TIMEOUT                     # the word stays raised until the workspace is initialised
    G.griffin_workspace_init(L.ws)
    assert L.status() == G.OK
    # the context is intact and the workspace serves a decode call as before
    e = torch.arange(0, 2 * k, 2, dtype=torch.int32, device=dev())
    cs = L.compact(e)
    x = rand((1, d), torch.bfloat16, 4)
    y = L.decode([cs], x)
    c = O.compact_experts(e.cpu().numpy(), np64(wg), np64(wu), np64(wd))
    assert_output(np64(y[0]), O.ff_pruned(np64(x[0]), c, "swiglu"), "bf16")
    assert L.status() == G.OK


def test_the_selftest_refuses_limits_that_could_hold_the_gpu_for_long():
    ws = torch.zeros(256, dtype=torch.uint8, device=dev())
    assert _selftest(ws, 0)[0] == G.ERR_INVALID_ARG
    assert _selftest(ws, 10 ** 10)[0] == G.ERR_INVALID_ARG
    torch.cuda.synchronize()
