"""A stack of independent FF blocks driven through the C ABI, phase by phase.

This is call sequencing and buffer ownership only: every step of the path runs in the
library's CUDA kernels (binding.py).  One FFStack holds, for one process / one GPU:
  * L blocks of full weights (w_gate, w_up, w_down) on the device,
  * one workspace shared by all calls (they are ordered on one stream),
  * per block and per sequence: the statistic s, the expert indices E and the compact
    weight set, all allocated once.
The phases mirror the GRIFFIN algorithm (Section 4.2 of the paper): prompt phase with the
full FF and the statistic, top-k selection, slicing of the weights, then the generation
phase on the compact weights.  With indexed=True the slicing is left out: the generation phase
reads the expert rows in place from neuron-major full weights (W_2 is transposed once, when a
block is added), and no compact sets are allocated.
"""
from __future__ import annotations

import torch

from . import binding as G


class FFStack:
    def __init__(self, d, d_ff, act, dtype, L, n_seq, S_max, k, device, indexed=False):
        self.d, self.d_ff, self.L, self.n_seq, self.S_max, self.k = d, d_ff, L, n_seq, S_max, k
        self.device = device
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        self.desc = G.make_desc(d, d_ff, act, dtype)
        self.n_mats = 3 if G.act_is_gated(act) else 2   # a block without a gate has no W_g (w_gate is None)
        self.ldk = G.griffin_compact_ldk(k)
        self.ws = G.alloc_workspace(self.desc, S_max, n_seq, device)
        self.indexed = indexed
        self.decode_flags = 0  # GRIFFIN_DECODE_RING / _STREAM / _TCGEN05 to add to every decode call (0: the library's own choice)
        self.weights = []      # per block: binding.FFWeights
        self.weights_nm = []   # per block (indexed only): binding.FFWeightsNM
        self.score = torch.empty((L, n_seq, d_ff), device=device, dtype=torch.float32)
        self.idx = torch.empty((L, n_seq, k), device=device, dtype=torch.int32)
        self.sets = []         # per block: list of n_seq compact sets
        self.set_arrays = []   # per block: C array of the n_seq sets, ready for decode
        for _ in range(0 if indexed else L):
            sets = [G.alloc_compact(self.desc, k, device, self.tdtype) for _ in range(n_seq)]
            self.sets.append(sets)
            self.set_arrays.append(G.compact_array(sets))

    def add_block(self, w_gate, w_up, w_down):
        self.weights.append(G.make_weights(w_gate, w_up, w_down))
        if self.indexed:  # a layout step at model-load time, not a step of the path
            self.weights_nm.append(G.make_weights_nm(w_gate, w_up, w_down.t().contiguous()))

    # ---- prompt phase -------------------------------------------------------------------
    def prefill_score(self, layer, seq, x, y):
        """Full FF over one sequence's prompt: y = FF(x); the statistic goes to score[layer, seq]."""
        G.griffin_ff_prefill_score(self.desc, self.weights[layer], x, y, self.score[layer, seq], self.ws)

    def select_all(self):
        """Top-k for every (block, sequence) in one launch."""
        G.griffin_select_topk(self.score.view(self.L * self.n_seq, self.d_ff), self.k,
                              self.idx.view(self.L * self.n_seq, self.k))

    def compact(self, layer, seq):
        G.griffin_compact_experts(self.desc, self.weights[layer], self.idx[layer, seq], self.sets[layer][seq], self.ws)

    # ---- generation phase ---------------------------------------------------------------
    def decode(self, layer, x, y, overlap):
        """Pruned FF for one token of each of the n_seq sequences: x, y are [n_seq, d]."""
        G.griffin_ff_decode(self.desc, self.set_arrays[layer], None, x, y, self.ws,
                            (G.DECODE_OVERLAP_WEIGHT_PREFETCH if overlap else G.DECODE_DEFAULT) | self.decode_flags)

    def decode_indexed(self, layer, x, y, overlap):
        """The same without compact sets: the rows idx[layer] are read from the full weights."""
        G.griffin_ff_decode_indexed(self.desc, self.weights_nm[layer], self.idx[layer], x, y, self.ws,
                                    G.DECODE_OVERLAP_WEIGHT_PREFETCH if overlap else G.DECODE_DEFAULT)

    def status(self):
        return G.griffin_check_device_status(self.ws)

    # ---- accounting (bytes and flops the algorithm needs, not what was moved) -----------
    def decode_bytes_per_call(self):
        b = 4 if self.tdtype == torch.float32 else 2
        return self.n_seq * (self.n_mats * self.k * self.d * b + 2 * self.d * b)

    def prefill_flops(self, S):
        return 2 * self.n_mats * S * self.d * self.d_ff

    def compact_bytes(self):
        b = 4 if self.tdtype == torch.float32 else 2
        return 2 * self.n_mats * self.k * self.d * b
