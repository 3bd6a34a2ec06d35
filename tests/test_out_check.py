"""The output acceptance test itself, on the CPU: it must notice what the relative L2 error alone lets
through -- one wrong element of a wide decode output, a short wrong segment of a prompt output -- and must
accept the rounding the storage type implies.  The mistakes are planted in copies of the oracle's output."""
import numpy as np
import pytest
import torch

from oracle import griffin_oracle as O
from out_check import STATED_L2, assert_output, output_error


def _decode_output(d=4096, k=512, seed=3):
    g = np.random.default_rng(seed)
    c = {"w_gate": g.standard_normal((k, d)) / np.sqrt(d), "w_up": g.standard_normal((k, d)) / np.sqrt(d),
         "w_down": g.standard_normal((d, k)) / np.sqrt(k)}
    x = g.standard_normal(d)
    e = np.arange(k)
    cs = O.compact_experts(e, c["w_gate"], c["w_up"], c["w_down"])
    return O.ff_pruned(x, cs, "swiglu")


def _as_bf16(a):
    return torch.from_numpy(a).to(torch.bfloat16).double().numpy()


def test_rounding_of_the_storage_type_is_accepted():
    y = _decode_output()
    assert_output(_as_bf16(y), y, "bf16")
    assert_output(y.astype(np.float32).astype(np.float64), y, "f32")


def test_one_wrong_element_of_a_wide_vector_is_caught_although_the_l2_error_is_inside_the_stated_bound():
    y = _decode_output()
    bad = _as_bf16(y)
    i = int(np.argmin(np.abs(y)))            # the least conspicuous place: an element near zero ...
    bad[i] = np.sqrt(np.mean(y ** 2))        # ... that comes out as a typical element's size
    l2, mx = output_error(bad, y)
    assert l2 < STATED_L2["bf16"]        # 1/64: the stated metric alone would pass it
    with pytest.raises(AssertionError):
        assert_output(bad, y, "bf16")


def test_a_wrong_32_column_segment_of_a_prompt_output_is_caught():
    g = np.random.default_rng(0)
    y = g.standard_normal((256, 4096))
    bad = _as_bf16(y)
    bad[100, 64:96] = 0.0                    # a dropped store of one 64-byte piece
    l2, _ = output_error(bad, y)
    assert l2 < STATED_L2["bf16"]
    with pytest.raises(AssertionError):
        assert_output(bad, y, "bf16")


def test_a_small_uniform_error_beyond_the_measured_level_is_caught_for_fp32():
    y = _decode_output(d=1024, k=128)
    with pytest.raises(AssertionError):
        assert_output(y * (1 + 2e-5), y, "f32")          # inside 1e-4, far above fp32 accumulation noise
    with pytest.raises(AssertionError):
        assert_output(y + 1.0, y, "f32")
    with pytest.raises(AssertionError):
        assert_output(np.where(np.arange(y.size) == 5, np.nan, y), y, "f32")
