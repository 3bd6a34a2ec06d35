"""The C ABI without a GPU: the library builds, loads, exports every declared symbol, and
validates its arguments on the host before it touches CUDA."""
import ctypes as C
import os
import re

import pytest

from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return G.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "griffin_ff.h")).read()
    declared = set(re.findall(r"\b(griffin_[a-z_0-9]+)\s*\(", header))
    assert declared == set(G.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert G.griffin_version() == 1
    texts = [G.status_string(i) for i in range(7)]
    assert len(set(texts)) == 7 and texts[0] == "ok"
    assert "unknown" in G.status_string(99)


def test_k_from_keep_ratio_agrees_with_oracle(lib):
    for d_ff in (8, 688, 11008, 24576, 13824, 14336, 7):
        for keep in (0.0, 0.1, 0.25, 0.5, 0.75, 1.0, 1.7, 0.333):
            assert G.griffin_k_from_keep_ratio(d_ff, keep) == O.k_from_keep_ratio(d_ff, keep)
    assert G.griffin_k_from_keep_ratio(16, float("nan")) == 1
    assert [G.griffin_compact_ldk(k) for k in (1, 8, 9, 5504, 37)] == [8, 8, 16, 5504, 40]


def test_workspace_bytes(lib):
    desc = G.make_desc(4096, 11008, "swiglu", "bf16")
    n = G.griffin_workspace_bytes(desc, 512, 1)
    assert n >= 256 + 512 * 11008 * 2
    assert G.griffin_workspace_bytes(desc, 0, 8) >= 256 + 8 * 11008 * 4
    assert G.griffin_workspace_bytes(G.make_desc(4097, 11008, "swiglu", "bf16"), 512, 1) == 0
    assert G.griffin_workspace_bytes(desc, 1024, 1) > n


def test_host_validation_rejects_before_any_launch(lib):
    desc = G.make_desc(256, 688, "swiglu", "f32")
    fake = C.c_void_p(0x10000)      # aligned, never dereferenced: validation fails first
    odd = C.c_void_p(0x10004)
    w = G.FFWeights(fake, fake, fake, None, None, None)
    # prefill
    f = lib.griffin_ff_prefill_score
    assert f(None, C.byref(w), fake, 4, fake, fake, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert f(C.byref(desc), C.byref(w), fake, 0, fake, fake, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert f(C.byref(desc), C.byref(w), odd, 4, fake, fake, fake, 1 << 30, None) == G.ERR_ALIGNMENT
    assert f(C.byref(desc), C.byref(w), fake, 4, fake, fake, None, 0, None) == G.ERR_WORKSPACE
    assert f(C.byref(desc), C.byref(w), fake, 4, fake, fake, fake, 1000, None) == G.ERR_WORKSPACE
    bad = G.make_desc(256, 688, 8, "f32")   # beyond the last activation code
    assert f(C.byref(bad), C.byref(w), fake, 4, fake, fake, fake, 1 << 30, None) == G.ERR_UNSUPPORTED
    bad = G.make_desc(250, 688, "swiglu", "f32")
    assert f(C.byref(bad), C.byref(w), fake, 4, fake, fake, fake, 1 << 30, None) == G.ERR_ALIGNMENT
    # a block without a gate (Eq. 2) must not name W_g or b_g, a gated one (Eq. 3) must name W_g
    relu = G.make_desc(256, 688, "relu", "f32")
    w_ng = G.FFWeights(None, fake, fake, None, None, None)
    assert f(C.byref(relu), C.byref(w), fake, 4, fake, fake, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert f(C.byref(relu), C.byref(G.FFWeights(None, fake, fake, fake, None, None)), fake, 4, fake, fake, fake,
             1 << 30, None) == G.ERR_INVALID_ARG
    assert f(C.byref(desc), C.byref(w_ng), fake, 4, fake, fake, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert f(C.byref(relu), C.byref(w_ng), fake, 4, fake, fake, fake, 1000, None) == G.ERR_WORKSPACE  # passes the gate check
    cs_g = G.FFCompact(fake, fake, fake, None, None, 344, 344)
    cs_ng = G.FFCompact(None, fake, fake, None, None, 344, 344)
    fd = lib.griffin_ff_decode
    assert fd(C.byref(relu), 1, C.byref(cs_g), None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_INVALID_ARG
    assert fd(C.byref(desc), 1, C.byref(cs_ng), None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_INVALID_ARG
    assert fd(C.byref(relu), 1, C.byref(cs_ng), None, fake, fake, fake, 100, 0, None) == G.ERR_WORKSPACE
    # prompt phase, piece by piece
    fc = lib.griffin_ff_prefill_score_chunk
    assert fc(C.byref(desc), C.byref(w), fake, 4, fake, None, fake, 1, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert fc(C.byref(desc), C.byref(w), fake, 0, fake, fake, None, 1, fake, 1 << 30, None) == G.ERR_INVALID_ARG
    assert fc(C.byref(desc), C.byref(w), fake, 4, fake, odd, None, 1, fake, 1 << 30, None) == G.ERR_ALIGNMENT
    assert fc(C.byref(desc), C.byref(w), fake, 4, fake, fake, None, 0, fake, 1000, None) == G.ERR_WORKSPACE
    # top-k
    t = lib.griffin_select_topk
    assert t(fake, 1, 688, 0, fake, None) == G.ERR_INVALID_ARG
    assert t(fake, 1, 688, 689, fake, None) == G.ERR_INVALID_ARG
    assert t(None, 1, 688, 3, fake, None) == G.ERR_INVALID_ARG
    # compaction
    c = lib.griffin_compact_experts
    out = G.FFCompact(fake, fake, fake, None, None, 344, 344)
    assert c(C.byref(desc), C.byref(w), None, C.byref(out), None, None) == G.ERR_INVALID_ARG
    out_bad = G.FFCompact(fake, fake, fake, None, None, 689, 696)
    assert c(C.byref(desc), C.byref(w), fake, C.byref(out_bad), None, None) == G.ERR_INVALID_ARG
    out_bad = G.FFCompact(fake, fake, fake, None, None, 37, 37)
    assert c(C.byref(desc), C.byref(w), fake, C.byref(out_bad), None, None) == G.ERR_ALIGNMENT
    out_bad = G.FFCompact(fake, fake, fake, None, None, 37, 48)
    assert c(C.byref(desc), C.byref(w), fake, C.byref(out_bad), None, None) == G.ERR_INVALID_ARG
    # decode
    dcd = lib.griffin_ff_decode
    sets = (G.FFCompact * 2)(out, out)
    assert dcd(C.byref(desc), 0, sets, None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_INVALID_ARG
    assert dcd(C.byref(desc), 33, sets, None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_UNSUPPORTED
    assert dcd(C.byref(desc), 2, sets, None, fake, fake, fake, 1 << 30, 16, None) == G.ERR_INVALID_ARG   # an unknown flag
    assert dcd(C.byref(desc), 2, sets, None, fake, fake, fake, 1 << 30, G.DECODE_RING | G.DECODE_STREAM, None) == G.ERR_INVALID_ARG
    assert dcd(C.byref(desc), 2, sets, None, fake, fake, fake, 100, 0, None) == G.ERR_WORKSPACE
    assert dcd(C.byref(desc), 2, sets, None, odd, fake, fake, 1 << 30, 0, None) == G.ERR_ALIGNMENT
    mixed = (G.FFCompact * 2)(out, G.FFCompact(fake, fake, fake, None, None, 336, 336))
    assert dcd(C.byref(desc), 2, mixed, None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_INVALID_ARG
    wide = G.make_desc(8200, 688, "swiglu", "f32")
    assert dcd(C.byref(wide), 1, sets, None, fake, fake, fake, 1 << 30, 0, None) == G.ERR_UNSUPPORTED
    # decode through the index list
    dix = lib.griffin_ff_decode_indexed
    bdesc = G.make_desc(256, 688, "swiglu", "bf16")
    wn = G.FFWeightsNM(fake, fake, fake, None, None, None)
    big = 1 << 30
    assert dix(C.byref(bdesc), 1, None, fake, 344, fake, fake, fake, big, 0, None) == G.ERR_INVALID_ARG
    assert dix(C.byref(bdesc), 1, C.byref(wn), None, 344, fake, fake, fake, big, 0, None) == G.ERR_INVALID_ARG
    assert dix(C.byref(bdesc), 1, C.byref(wn), fake, 0, fake, fake, fake, big, 0, None) == G.ERR_INVALID_ARG
    assert dix(C.byref(bdesc), 1, C.byref(wn), fake, 689, fake, fake, fake, big, 0, None) == G.ERR_INVALID_ARG
    assert dix(C.byref(bdesc), 1, C.byref(wn), fake, 344, fake, fake, fake, big, 2, None) == G.ERR_INVALID_ARG
    assert dix(C.byref(desc), 1, C.byref(wn), fake, 344, fake, fake, fake, big, 0, None) == G.ERR_UNSUPPORTED  # fp32
    assert dix(C.byref(bdesc), 33, C.byref(wn), fake, 344, fake, fake, fake, big, 0, None) == G.ERR_UNSUPPORTED
    assert dix(C.byref(bdesc), 1, C.byref(wn), fake, 344, odd, fake, fake, big, 0, None) == G.ERR_ALIGNMENT
    assert dix(C.byref(bdesc), 1, C.byref(wn), fake, 344, fake, fake, None, 0, 0, None) == G.ERR_WORKSPACE
    assert dix(C.byref(bdesc), 2, C.byref(wn), fake, 344, fake, fake, fake,
               G.griffin_workspace_bytes(bdesc, 0, 1), 0, None) == G.ERR_WORKSPACE   # sized for one sequence
    no_down = G.FFWeightsNM(fake, fake, None, None, None, None)
    assert dix(C.byref(bdesc), 1, C.byref(no_down), fake, 344, fake, fake, fake, big, 0, None) == G.ERR_INVALID_ARG
    # combine
    cmb = lib.griffin_combine_scores
    lens = (C.c_int32 * 2)(4, 0)
    assert cmb(fake, lens, 2, 688, fake, None) == G.ERR_INVALID_ARG
    assert cmb(fake, lens, 300, 688, fake, None) == G.ERR_UNSUPPORTED
    # workspace
    assert lib.griffin_workspace_init(None, 4096, None) == G.ERR_WORKSPACE
    assert lib.griffin_check_device_status(None, None) == G.ERR_WORKSPACE


def test_binding_fails_loudly_without_library(tmp_path, monkeypatch):
    monkeypatch.setattr(G, "_lib", None)
    with pytest.raises(RuntimeError, match="missing"):
        G.load(str(tmp_path / "nope.so"))


def test_slicing_from_neuron_major_weights_validates_like_the_row_major_call(lib):
    desc = G.make_desc(256, 688, "swiglu", "bf16")
    fake, odd = C.c_void_p(0x10000), C.c_void_p(0x10004)
    wn = G.FFWeightsNM(fake, fake, fake, None, None, None)
    out = G.FFCompact(fake, fake, fake, None, None, 344, 344)
    f = lib.griffin_compact_experts_nm
    assert f(None, C.byref(wn), fake, C.byref(out), None, None) == G.ERR_INVALID_ARG
    assert f(C.byref(desc), None, fake, C.byref(out), None, None) == G.ERR_INVALID_ARG
    assert f(C.byref(desc), C.byref(wn), None, C.byref(out), None, None) == G.ERR_INVALID_ARG
    no_down = G.FFWeightsNM(fake, fake, None, None, None, None)
    assert f(C.byref(desc), C.byref(no_down), fake, C.byref(out), None, None) == G.ERR_INVALID_ARG
    no_gate = G.FFWeightsNM(None, fake, fake, None, None, None)          # a gated block needs W_g
    assert f(C.byref(desc), C.byref(no_gate), fake, C.byref(out), None, None) == G.ERR_INVALID_ARG
    misaligned = G.FFWeightsNM(fake, fake, odd, None, None, None)
    assert f(C.byref(desc), C.byref(misaligned), fake, C.byref(out), None, None) == G.ERR_ALIGNMENT
    bad_ldk = G.FFCompact(fake, fake, fake, None, None, 344, 352)        # ldk must be k rounded up to 8
    assert f(C.byref(desc), C.byref(wn), fake, C.byref(bad_ldk), None, None) == G.ERR_INVALID_ARG
    too_many = G.FFCompact(fake, fake, fake, None, None, 696, 696)       # k beyond d_ff
    assert f(C.byref(desc), C.byref(wn), fake, C.byref(too_many), None, None) == G.ERR_INVALID_ARG
    relu = G.make_desc(256, 688, "relu", "bf16")                         # without a gate, naming W_g is an error
    assert f(C.byref(relu), C.byref(wn), fake, C.byref(out), None, None) == G.ERR_INVALID_ARG


def test_launch_counter_starts_at_zero_and_refused_calls_do_not_count(lib):
    before = G.griffin_kernel_launches()
    desc = G.make_desc(256, 688, "swiglu", "bf16")
    assert lib.griffin_select_topk(None, 1, 688, 344, None, None) == G.ERR_INVALID_ARG
    assert lib.griffin_workspace_init(None, 0, None) == G.ERR_WORKSPACE
    assert G.griffin_kernel_launches() == before
    assert isinstance(before, int) and before >= 0
