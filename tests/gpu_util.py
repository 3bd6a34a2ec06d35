"""Helpers shared by the GPU parity tests (CUDA path through the C ABI vs. the CPU oracle)."""
import numpy as np
import torch

from oracle import griffin_oracle as O
from paper_2404_01365_b200 import binding as G

from out_check import assert_output  # noqa: F401  (the output acceptance test: relative L2 and largest element error)

TIE_WINDOW = 1e-3                           # expert sets may differ only this close to the k-th score


def score_tol(dtype):
    """Relative tolerance on each s_j.  The statistic is computed from fp32 activations in both
    storage types; what is left is fp32 accumulation noise over d (dot products), d_ff (row
    norm) and S (column sum) terms."""
    return 1e-5 if dtype == "f32" else 2e-5


def dev():
    return torch.device("cuda:0")


def np64(t):
    return t.detach().to("cpu", torch.float64).numpy()


def rel_l2(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def rand(shape, dtype, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(dtype)


def check_expert_set(e_gpu, s_ref, k):
    """|E| = k, ascending, no duplicates; differs from the oracle's set only at scores within
    TIE_WINDOW (relative) of the oracle's k-th largest score."""
    e_gpu = np.asarray(e_gpu)
    assert e_gpu.shape == (k,)
    assert np.all(np.diff(e_gpu) > 0), "indices must be strictly ascending"
    assert e_gpu.min() >= 0 and e_gpu.max() < len(s_ref)
    e_ref = O.select_topk(s_ref, k)
    tau = np.sort(s_ref)[-k]
    diff = np.setxor1d(e_gpu, e_ref)
    assert np.all(np.abs(s_ref[diff] - tau) <= TIE_WINDOW * tau), (len(diff), s_ref[diff], tau)
    return len(diff)


class GpuLayer:
    """One FF block on the GPU: device copies of the weights plus a workspace."""

    def __init__(self, d, d_ff, act, dtype, wg, wu, wd, bg=None, bu=None, bd=None, S_max=0, n_seq=1):
        self.desc = G.make_desc(d, d_ff, act, dtype)
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        up = lambda t: None if t is None else t.to(dev()).contiguous()
        self.t = dict(wg=up(wg), wu=up(wu), wd=up(wd), bg=up(bg), bu=up(bu), bd=up(bd))
        self.weights = G.make_weights(self.t["wg"], self.t["wu"], self.t["wd"], self.t["bg"], self.t["bu"], self.t["bd"])
        self.ws = G.alloc_workspace(self.desc, S_max, n_seq, dev())
        self.d, self.d_ff = d, d_ff

    def prefill(self, x, want_y=True):
        x = x.to(dev()).contiguous()
        y = torch.empty((x.shape[0], self.d), device=dev(), dtype=self.tdtype) if want_y else None
        s = torch.empty((self.d_ff,), device=dev(), dtype=torch.float32)
        G.griffin_ff_prefill_score(self.desc, self.weights, x, y, s, self.ws)
        return y, s

    def select(self, s, k):
        n_seq = 1 if s.dim() == 1 else s.shape[0]
        e = torch.empty((n_seq, k), device=dev(), dtype=torch.int32)
        G.griffin_select_topk(s, k, e)
        return e[0] if s.dim() == 1 else e

    def compact(self, e):
        k = e.numel()
        cs = G.alloc_compact(self.desc, k, dev(), self.tdtype, with_bias=self.t["bu"] is not None)
        G.griffin_compact_experts(self.desc, self.weights, e, cs, self.ws)
        return cs

    def compact_nm(self, e):
        """The same compact set from neuron-major weights (W_2 transposed once, as at model load)."""
        self._neuron_major()
        k = e.numel()
        cs = G.alloc_compact(self.desc, k, dev(), self.tdtype, with_bias=self.t["bu"] is not None)
        G.griffin_compact_experts_nm(self.desc, self.weights_nm, e, cs, self.ws)
        return cs

    def _neuron_major(self):
        if not hasattr(self, "weights_nm"):
            self.t["wd_t"] = self.t["wd"].t().contiguous()
            self.weights_nm = G.make_weights_nm(self.t["wg"], self.t["wu"], self.t["wd_t"], self.t["bg"], self.t["bu"],
                                                self.t["bd"])

    def dense_set(self):
        """The full weights viewed as a compact set with E = all neurons."""
        return G.make_compact(self.t["wg"], self.t["wu"], self.t["wd"], self.d_ff, self.d_ff, self.t["bg"], self.t["bu"])

    def decode(self, sets, x, flags=0):
        x = x.to(dev()).contiguous()
        y = torch.empty_like(x)
        G.griffin_ff_decode(self.desc, sets, self.t["bd"], x, y, self.ws, flags)
        return y

    def decode_indexed(self, idx, x, flags=0):
        """Pruned FF straight from the full weights (W_2 transposed once, as at model load)."""
        self._neuron_major()
        x = x.to(dev()).contiguous()
        y = torch.empty_like(x)
        G.griffin_ff_decode_indexed(self.desc, self.weights_nm, idx, x, y, self.ws, flags)
        return y

    def status(self):
        return G.griffin_check_device_status(self.ws)
