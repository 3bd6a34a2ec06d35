"""CPU oracle for the GRIFFIN gated feed-forward path.  TEST INFRASTRUCTURE ONLY.

This module is a plain, slow, fp64 restatement of what the GRIFFIN paper
(arXiv 2404.01365) defines for one feed-forward (FF) block.  It exists so that
the CUDA path can be checked against something written independently of it.
It shares no code with the CUDA path and must never be imported by it: only
the tests, the smoke check and the benchmark's CPU-baseline leg call it.

Everything is numpy float64.  A matmul is used as a library step where the
paper writes a matrix product; nothing is blocked, fused or reordered.

Notation (paper Section 3): D -> d, D_FF -> d_ff, W_g -> w_gate [d_ff, d],
W_1 -> w_up [d_ff, d], W_2 -> w_down [d, d_ff], b_g / b_1 / b_2 optional
biases, X [S, d] the prompt's hidden states, Z = FF_1(X) [S, d_ff] the "FF
activations", s [d_ff] the selection statistic, E the expert set, k = |E|.

Pinning status (see tests/test_oracle_pins.py):
  * ff1_activations, ff_dense     pinned (brute force, identity weights,
                                  closed-form sigma values; the blocks
                                  without a gate: brute force, identity
                                  weights, the gated form with a constant
                                  second branch)
  * flock_score                   pinned (sum_j s_j^2 = S, S = 1, rank one,
                                  row-rescale invariance, permutation
                                  equivariance, brute force)
  * select_topk                   pinned (brute force, constructed ties)
  * compact_experts               pinned (indexing identity, the paper's
                                  active-parameter counts)
  * ff_pruned                     pinned (keep = 1 equals the dense FF, mask
                                  form)
  * combine_scores                pinned (single sample reduces to s/sqrt(S);
                                  brute force)
  * How well FF_hat approximates FF on real models: parity unpinned (it needs
    trained weights; nothing here tests it).
"""
from __future__ import annotations

import math

import numpy as np

SWIGLU = "swiglu"
GEGLU_TANH = "geglu_tanh"
REGLU = "reglu"
GEGLU_ERF = "geglu_erf"
ACTIVATIONS = (SWIGLU, GEGLU_TANH, REGLU, GEGLU_ERF)
# FF blocks without a gate (Eq. 2, e.g. OPT): the name of the block -> the sigma it uses
RELU = "relu"
GELU_TANH = "gelu_tanh"
GELU_ERF = "gelu_erf"
SILU = "silu"
NON_GATED = {RELU: REGLU, GELU_TANH: GEGLU_TANH, GELU_ERF: GEGLU_ERF, SILU: SWIGLU}

_erf = np.vectorize(math.erf, otypes=[np.float64])


def _f64(a):
    return None if a is None else np.asarray(a, dtype=np.float64)


def sigma(t, act):
    """Gate non-linearity sigma of Eq. 3.

    The paper names the GLU variants (SwiGLU, GEGLU, ReGLU) without writing
    sigma out; the readings taken here are
      swiglu      sigma(t) = t / (1 + exp(-t))                       (SiLU)
      geglu_tanh  sigma(t) = t/2 * (1 + tanh(sqrt(2/pi) (t + 0.044715 t^3)))
      reglu       sigma(t) = max(t, 0)
      geglu_erf   sigma(t) = t/2 * (1 + erf(t / sqrt(2)))            (exact GELU)
    """
    t = _f64(t)
    if act == SWIGLU:
        with np.errstate(over="ignore"):
            return t / (1.0 + np.exp(-t))
    if act == GEGLU_TANH:
        return 0.5 * t * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (t + 0.044715 * t ** 3)))
    if act == REGLU:
        return np.maximum(t, 0.0)
    if act == GEGLU_ERF:
        return 0.5 * t * (1.0 + _erf(t / math.sqrt(2.0)))
    raise ValueError(f"unknown activation {act!r}")


def ff1_activations(x, w_gate, w_up, act, b_gate=None, b_up=None):
    """Z = FF_1(X) = sigma(X W_g^T + b_g) * (X W_1^T + b_1)   (Eq. 3).

    x is [S, d] (or [d] for one token); the result is [S, d_ff] (or [d_ff]).
    sigma acts on the gate branch only.

    For a block without a gate (act in NON_GATED; Eq. 2) there is no W_g:
    Z = sigma(X W_1^T + b_1); w_gate and b_gate must be None.
    """
    x, w_up = _f64(x), _f64(w_up)
    u = x @ w_up.T
    if b_up is not None:
        u = u + _f64(b_up)
    if act in NON_GATED:
        if w_gate is not None or b_gate is not None:
            raise ValueError("a block without a gate has no W_g, b_g")
        return sigma(u, NON_GATED[act])
    g = x @ _f64(w_gate).T
    if b_gate is not None:
        g = g + _f64(b_gate)
    return sigma(g, act) * u


def ff_dense(x, w_gate, w_up, w_down, act, b_gate=None, b_up=None, b_down=None):
    """FF(X) = FF_2(FF_1(X)), FF_2(Z) = Z W_2^T + b_2   (Eq. 1 with Eq. 3).

    Returns (Y [S, d], Z [S, d_ff]).  This is the full, unpruned block: the
    prompt phase always uses it, whatever k is (Section 4.2).
    """
    z = ff1_activations(x, w_gate, w_up, act, b_gate, b_up)
    y = z @ _f64(w_down).T
    if b_down is not None:
        y = y + _f64(b_down)
    return y, z


def flock_score(z):
    """Selection statistic s of Eq. 6 from the FF activations Z [S, d_ff].

    Step 1 (Section 4.1): each row of Z is scaled to a unit vector,
        Zbar_i = Z_i / ||Z_i||_2.
    Step 2 (Eq. 6): s_j is the l2 norm of column j of Zbar over the S tokens.
    Reading for a row whose norm is zero (the paper does not say): that token
    contributes nothing to any s_j.  The printed equation runs its column
    index to D; s has d_ff entries, so the columns run to d_ff.
    """
    z = _f64(z)
    if z.ndim != 2:
        raise ValueError("Z must be [S, d_ff]")
    r = np.sqrt(np.sum(z * z, axis=1))
    zbar = np.zeros_like(z)
    nz = r > 0.0
    zbar[nz] = z[nz] / r[nz, None]
    return np.sqrt(np.sum(zbar * zbar, axis=0))


def k_from_keep_ratio(d_ff, keep):
    """Number of experts for a keep ratio (1 - the paper's "FF sparsity").

    The paper does not state a rounding rule; round-half-up, clamped to
    [1, d_ff], is the reading taken.
    """
    k = int(math.floor(keep * d_ff + 0.5))
    return max(1, min(int(d_ff), k))


def select_topk(s, k):
    """E = indices of the k largest entries of s (Section 4.2).

    Readings: equal scores are broken towards the lower index, and E is
    returned in ascending index order (the paper treats E as a set).
    """
    s = _f64(s)
    if s.ndim != 1:
        raise ValueError("s must be a vector")
    n = s.shape[0]
    if not (1 <= k <= n):
        raise ValueError("k out of range")
    if not np.all(np.isfinite(s)):
        raise ValueError("non-finite score")
    order = np.argsort(-s, kind="stable")  # descending score, ties by index
    return np.sort(order[:k]).astype(np.int32)


def compact_experts(e, w_gate, w_up, w_down, b_gate=None, b_up=None):
    """W_g_hat = W_g[E, :], W_1_hat = W_1[E, :], W_2_hat = W_2[:, E], and the
    matching entries of b_g, b_1 (Section 4.2).  b_2 is not pruned (Eq. 5).

    Returns a dict with w_gate [k, d], w_up [k, d], w_down [d, k] and the two
    bias slices (None where no bias was given).
    """
    e = np.asarray(e, dtype=np.int64)
    return {
        "w_gate": None if w_gate is None else np.asarray(w_gate)[e, :],
        "w_up": np.asarray(w_up)[e, :],
        "w_down": np.asarray(w_down)[:, e],
        "b_gate": None if b_gate is None else np.asarray(b_gate)[e],
        "b_up": None if b_up is None else np.asarray(b_up)[e],
    }


def ff_pruned(x, compact, act, b_down=None):
    """Generation-phase FF with the expert neurons only (Eqs. 4 and 5):
        z_hat = sigma(W_g_hat x + b_g_hat) * (W_1_hat x + b_1_hat)
        y_hat = W_2_hat z_hat + b_2.
    x is [B, d] or [d]; `compact` is what compact_experts returned.
    """
    z = ff1_activations(x, compact["w_gate"], compact["w_up"], act,
                        compact["b_gate"], compact["b_up"])
    y = z @ _f64(compact["w_down"]).T
    if b_down is not None:
        y = y + _f64(b_down)
    return y


def combine_scores(scores, prompt_lengths):
    """Batch statistic s_bar = sum_i s_i / sqrt(S_i)   (Eq. 7), used to pick
    one expert set for several samples."""
    acc = np.zeros_like(_f64(scores[0]))
    for s_i, S_i in zip(scores, prompt_lengths):
        acc = acc + _f64(s_i) / math.sqrt(float(S_i))
    return acc


def removed_parameters(n_layers, d, d_ff, k):
    """Parameters that leave the active set when every FF block of a gated
    model keeps k of d_ff neurons: three matrices lose (d_ff - k) rows or
    columns of length d each (Section 3, compressed FF shapes)."""
    return int(n_layers) * 3 * (int(d_ff) - int(k)) * int(d)


def griffin_layer(x_prompt, x_decode, w_gate, w_up, w_down, act, k,
                  b_gate=None, b_up=None, b_down=None):
    """One FF block through both phases, in the paper's order: prompt-phase
    dense FF, statistic, top-k, slicing, then the pruned FF on the decode
    tokens.  Returns a dict of every intermediate."""
    y, z = ff_dense(x_prompt, w_gate, w_up, w_down, act, b_gate, b_up, b_down)
    s = flock_score(z)
    e = select_topk(s, k)
    c = compact_experts(e, w_gate, w_up, w_down, b_gate, b_up)
    y_hat = ff_pruned(x_decode, c, act, b_down)
    return {"y": y, "z": z, "s": s, "e": e, "compact": c, "y_hat": y_hat}
