"""Seeded synthetic inputs for the GRIFFIN feed-forward path.

This module only draws random tensors; it holds none of the method's
arithmetic.  Both the CPU oracle's tests and the CUDA path consume exactly the
tensors produced here, so the two sides see the same numbers.

The workloads stand in for the models the paper measures (Llama 2 7B / 13B,
Gemma 7B, Mistral 7B): only the FF shapes are taken from them.  Weights are
random, hidden states are Gaussian noise plus one direction shared by every
token of a sequence, which gives the activations a per-sequence structure in
the spirit of the "flocking" the paper describes (Section 4.1).

Every tensor is drawn on its own counter-derived seed
    seed = mix(base_seed, config index, layer, sequence, tensor id)
so any single (layer, sequence) can be regenerated without the others.
Tensors are rounded once to the workload's storage dtype; the oracle widens
those rounded values to float64.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

F32 = "f32"
BF16 = "bf16"
SWIGLU = "swiglu"
GEGLU_TANH = "geglu_tanh"
RELU = "relu"                      # a block without a gate (Eq. 2 of the paper, as in OPT)
NON_GATED = ("relu", "gelu_tanh", "gelu_erf", "silu")

_T_W_GATE, _T_W_UP, _T_W_DOWN, _T_DIR, _T_NORM, _T_PROMPT, _T_DECODE = range(7)


@dataclass(frozen=True)
class Workload:
    name: str
    index: int           # position in the list of workloads (enters the seed)
    d: int
    d_ff: int
    S: int               # prompt tokens
    T: int               # decode steps
    B: int               # sequences decoded together, each with its own experts
    keeps: tuple         # keep ratios (1 - FF sparsity)
    dtype: str           # storage dtype of X, weights, Y
    act: str
    L: int               # independent FF blocks ("layers")
    mean_norm: tuple     # (lo, hi) of the shared direction's norm; lo == hi -> fixed
    base_seed: int = 0

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == F32 else torch.bfloat16

    @property
    def elem_bytes(self):
        return 4 if self.dtype == F32 else 2


WORKLOADS = {
    w.name: w
    for w in (
        Workload("tiny_swiglu_f32", 0, 256, 688, 64, 16, 1, (0.5,), F32, SWIGLU, 1, (2.0, 2.0)),
        Workload("llama2_7b", 1, 4096, 11008, 512, 128, 1, (0.5,), BF16, SWIGLU, 32, (4.0, 4.0)),
        Workload("gemma_7b", 2, 3072, 24576, 1024, 256, 1, (0.5,), BF16, GEGLU_TANH, 28, (4.0, 4.0)),
        Workload("llama2_13b", 3, 5120, 13824, 2048, 256, 8, (0.5,), BF16, SWIGLU, 40, (4.0, 4.0)),
        Workload("mistral_7b", 4, 4096, 14336, 4096, 512, 4, (0.25, 0.5, 0.75, 1.0), BF16, SWIGLU, 32,
                 (1.0, 8.0)),
        # not one of the five measured workloads: the FF shape of OPT-6.7B, a ReLU block without a gate
        Workload("opt_6p7b", 5, 4096, 16384, 512, 128, 1, (0.5,), BF16, RELU, 32, (4.0, 4.0)),
    )
}


def scaled(w: Workload, **changes) -> Workload:
    """A copy of a workload with some fields replaced (smaller test cases)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(changes)
    return Workload(**d)


_MASK = (1 << 64) - 1


def _mix(*words) -> int:
    """splitmix64-style hash of a tuple of small integers -> 63-bit seed."""
    h = 0x9E3779B97F4A7C15
    for w in words:
        h = (h + (int(w) & _MASK) + 0x9E3779B97F4A7C15) & _MASK
        h ^= h >> 30
        h = (h * 0xBF58476D1CE4E5B9) & _MASK
        h ^= h >> 27
        h = (h * 0x94D049BB133111EB) & _MASK
        h ^= h >> 31
    return h & ((1 << 63) - 1)


def _gen(w: Workload, layer, seq, tensor_id, device):
    g = torch.Generator(device=device)
    g.manual_seed(_mix(w.base_seed, w.index, layer, seq, tensor_id))
    return g


def _randn(shape, g, device, std=1.0):
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t


def make_weights(w: Workload, layer: int, device="cpu"):
    """(w_gate [d_ff, d], w_up [d_ff, d], w_down [d, d_ff]) for one FF block.

    Entries are i.i.d. N(0, 1/d) for the gate and up projections and
    N(0, 1/d_ff) for the down projection, rounded to the storage dtype.
    w_gate is None for a block without a gate.
    """
    dt = w.torch_dtype
    wg = None
    if w.act not in NON_GATED:
        wg = _randn((w.d_ff, w.d), _gen(w, layer, 0, _T_W_GATE, device), device, w.d ** -0.5).to(dt)
    wu = _randn((w.d_ff, w.d), _gen(w, layer, 0, _T_W_UP, device), device, w.d ** -0.5).to(dt)
    wd = _randn((w.d, w.d_ff), _gen(w, layer, 0, _T_W_DOWN, device), device, w.d_ff ** -0.5).to(dt)
    return wg, wu, wd


def _shared_mean(w: Workload, layer: int, seq: int, device):
    u = _randn((w.d,), _gen(w, layer, seq, _T_DIR, device), device)
    u = u / u.norm()
    lo, hi = w.mean_norm
    if hi > lo:
        r = torch.rand((), generator=_gen(w, layer, seq, _T_NORM, device), device=device)
        m = lo + (hi - lo) * float(r)
    else:
        m = lo
    return u * m


def make_prompt(w: Workload, layer: int, seq: int, device="cpu", S=None):
    """Prompt hidden states X [S, d]: N(0, I) per token plus the sequence's
    shared mean direction."""
    S = w.S if S is None else S
    x = _randn((S, w.d), _gen(w, layer, seq, _T_PROMPT, device), device)
    x += _shared_mean(w, layer, seq, device)
    return x.to(w.torch_dtype)


def make_decode_inputs(w: Workload, layer: int, seq: int, device="cpu", T=None):
    """Decode-step hidden states [T, d] for one sequence: same law as the
    prompt (fresh noise, same shared direction)."""
    T = w.T if T is None else T
    x = _randn((T, w.d), _gen(w, layer, seq, _T_DECODE, device), device)
    x += _shared_mean(w, layer, seq, device)
    return x.to(w.torch_dtype)


def shard_units(n_units: int, rank: int, world: int):
    """Contiguous block of unit indices owned by `rank` when `n_units`
    independent problems are split over `world` processes."""
    base, rem = divmod(n_units, world)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))
