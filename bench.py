#!/usr/bin/env python
"""Benchmark of the GRIFFIN feed-forward hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input, for a stack of L
independent FF blocks shaped like the named model:
    prompt phase (full FF + statistic) for every block and sequence  ->  top-k for all of them
    ->  expert compaction for every block and sequence  ->  T decode steps, each through all L blocks.
The weights of all blocks stay resident in HBM (they are the model); the hidden states are the
step's input.  All L blocks are visited in turn, so every weight byte comes from HBM, not L2.

The headline workload is the largest one: the Llama-2-13B shape with 8 sequences that each select
their own experts (about 100 GB resident).  The same JSON line carries, under "workloads", the
other bf16 shapes (Llama-2-7B, Gemma-7B, Llama-2-13B at batch 1, Mistral-7B over its keep sweep),
each measured by the same code on a few steps, with the buffers of one freed before the next.

Prints ONE JSON line (rank 0).  `value` = generated tokens per second per block for the whole
step (B*T*L / step time, summed over ranks: every rank runs its own sequences, there is no
exchange between ranks).  `--impl reference` times the CPU oracle on a bounded sample instead.
`--gpus N` with N > 1, when not already launched by torch.distributed.run, starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import gc
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pruned-FF decode tokens/s/layer (whole GRIFFIN FF path: prefill+score, top-k, compaction, decode)"
UNIT = "tokens/s/layer"
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "llama2_13b"
SHAPE_NOTE = {
    "llama2_7b": "Llama-2-7B-shaped SwiGLU FF",
    "gemma_7b": "Gemma-7B-shaped GeGLU FF (tanh-GELU gate)",
    "llama2_13b": "Llama-2-13B-shaped SwiGLU FF, every sequence with its own expert set",
    "mistral_7b": "Mistral-7B-shaped SwiGLU FF, every sequence with its own expert set",
    "opt_6p7b": "OPT-6.7B-shaped ReLU FF without a gate",
    "tiny_swiglu_f32": "tiny fp32 SwiGLU FF (L2-resident)",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--keep", type=float, default=None)
    ap.add_argument("--batch", type=int, default=None, help="override the number of sequences decoded together")
    ap.add_argument("--layers", type=int, default=None, help="override the number of blocks (smaller footprint)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every decode call from the host instead of replaying a CUDA graph")
    ap.add_argument("--decode", default="compact", choices=["compact", "indexed"],
                    help="indexed: no compaction step, the decode calls read the expert rows in place from the full weights")
    ap.add_argument("--decode-kernel", default="auto", choices=["auto", "ring", "stream"],
                    help="bf16, sequences with their own sets: force one of the two warp-level decode kernels "
                         "(auto: the library picks by the size of the call)")
    ap.add_argument("--shared-set", action="store_true",
                    help="the batch statistic of Eq. 7 in place of per-sequence sets: every sequence of a decode call uses the "
                         "first sequence's expert set, so the weights are streamed once per call")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="leave out the section with the other shapes")
    ap.add_argument("--section-steps", type=int, default=3, help="timed steps of each entry of the workloads section")
    return ap.parse_args()


def measured_peaks():
    """(hbm GB/s, bf16 burst TFLOP/s, bf16 sustained TFLOP/s, where they come from)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, 1590.0, 1400.0, "fallback (6.65 TB/s, 1.59 / 1.40 PFLOP/s: earlier measurements on this pool)"


def decode_kernel_name(w, B, k, forced="auto"):
    """Which of the two warp-level kernels griffin_ff_decode picks for sequences with their own sets (bf16): the
    register stream from about 150 MB of compact weights per call, the shared-memory ring below (the rule stated
    with GRIFFIN_DECODE_RING / GRIFFIN_DECODE_STREAM in include/griffin_ff.h)."""
    if w.dtype != "bf16":
        return "decode_gate_up_kernel + decode_down_kernel"
    if forced != "auto":
        return {"ring": "decode_fused_kernel", "stream": "decode_stream_kernel"}[forced]
    return "decode_stream_kernel" if B * 3 * k * w.d * 2 >= 150e6 else "decode_fused_kernel"


def recorded_traffic(key, kernel):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary of this workload, if it is the
    kernel that ran and its sources are unchanged since that capture; otherwise None."""
    p = os.path.join(ROOT, "profiles", "decode_traffic.json")
    try:
        rec = json.load(open(p))[key]
        h = hashlib.sha1()
        for name in rec["sources"]:
            h.update(open(os.path.join(ROOT, name), "rb").read())
        if h.hexdigest() == rec["sha1"] and rec.get("kernel") == kernel:
            return rec["dram_bytes_per_decode_call"]
    except Exception:
        pass
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.gpu_id, self.proc, self.lines = gpu_id, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_id), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [v.strip() for v in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


# --------------------------------------------------------------------------------------------
# CPU oracle: the reference arm, and the cpu_baseline leg of the GPU arm
# --------------------------------------------------------------------------------------------
_oracle_inputs = {}


def oracle_phases(w, keep, layer, S_sample, T_sample):
    """The oracle, as it stands, on one block and one sequence of the workload: prompt phase over the first
    S_sample prompt tokens, statistic, top-k, slicing and T_sample decode steps.  Returns the seconds of each
    phase.  (The inputs of a block are drawn once and kept: drawing them is not part of the path.)"""
    from oracle import griffin_oracle as O
    from paper_2404_01365_b200 import synth
    key = (w.name, layer)
    if key not in _oracle_inputs:
        if len(_oracle_inputs) >= 2:
            _oracle_inputs.pop(next(iter(_oracle_inputs)))
        wg, wu, wd = (None if t is None else t.double().numpy() for t in synth.make_weights(w, layer))
        _oracle_inputs[key] = (wg, wu, wd, synth.make_prompt(w, layer, 0).double().numpy(),
                               synth.make_decode_inputs(w, layer, 0, T=min(w.T, 64)).double().numpy())
    wg, wu, wd, x, xd = _oracle_inputs[key]
    x, xd = x[:S_sample], xd[:T_sample]
    k = O.k_from_keep_ratio(w.d_ff, keep)
    t0 = time.perf_counter()
    y, z = O.ff_dense(x, wg, wu, wd, w.act)
    s = O.flock_score(z)
    t1 = time.perf_counter()
    e = O.select_topk(s, k)
    t2 = time.perf_counter()
    c = O.compact_experts(e, wg, wu, wd)
    t3 = time.perf_counter()
    for t in range(len(xd)):
        O.ff_pruned(xd[t], c, w.act)
    t4 = time.perf_counter()
    return {"prefill": t1 - t0, "select": t2 - t1, "compact": t3 - t2, "decode": t4 - t3, "S": len(x), "T": len(xd)}


def compose_tokens_per_s(w, ph):
    """tokens/s/layer of the whole path for one sequence from the phase times of a sample: the prompt phase
    scales with the prompt tokens, the decode phase with the decode steps (both are sums over tokens)."""
    t = ph["prefill"] * w.S / ph["S"] + ph["select"] + ph["compact"] + ph["decode"] * w.T / ph["T"]
    return w.T / t


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def cpu_baseline(w, keep):
    """The oracle on all host cores (whole prompt, 16 decode steps) and on one core (a quarter of that)."""
    import numpy  # noqa: F401  (loads the BLAS that blas_threads() asks about)
    from threadpoolctl import threadpool_limits
    S1, T1 = min(w.S, 2048), min(w.T, 16)
    ph = oracle_phases(w, keep, 0, S1, T1)
    out = {"value": compose_tokens_per_s(w, ph), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
           "sample": f"one block, one sequence: prompt phase on {ph['S']} of {w.S} tokens, top-k, slicing, {ph['T']} of {w.T} "
                     f"decode steps ({sum(ph[p] for p in ('prefill', 'select', 'compact', 'decode')):.1f} s), phases scaled to the "
                     f"whole prompt and all decode steps; numpy fp64"}
    S2, T2 = min(w.S, 256), min(w.T, 4)
    with threadpool_limits(limits=1):
        ph1 = oracle_phases(w, keep, 0, S2, T2)
    out["one_core"] = {"value": compose_tokens_per_s(w, ph1), "unit": UNIT, "cores": 1,
                       "sample": f"the same block with BLAS held to one thread: {ph1['S']} prompt tokens, {ph1['T']} decode steps "
                                 f"({sum(ph1[p] for p in ('prefill', 'select', 'compact', 'decode')):.1f} s), scaled the same way"}
    return out


def run_reference(args, w, keep):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    S_sample, T_sample = min(w.S, 1024), min(w.T, 16)
    times, phases = [], []
    for i in range(args.warmup + args.steps):
        ph = oracle_phases(w, keep, i % 2, S_sample, T_sample)
        if i >= args.warmup:
            times.append(sum(ph[p] for p in ("prefill", "select", "compact", "decode")))
            phases.append(ph)
    med = {p: statistics.median(ph[p] for ph in phases) for p in ("prefill", "select", "compact", "decode")}
    med["S"], med["T"] = S_sample, T_sample
    value = compose_tokens_per_s(w, med)
    ms = 1e3 * sum(times) / len(times)
    sample = (f"each step: one block, one sequence of the workload -- prompt phase on {S_sample} of {w.S} tokens, top-k, slicing, "
              f"{T_sample} of {w.T} decode steps; value = T / (whole-prompt + top-k + slicing + T decode steps) from the median phase "
              f"times; every sequence of a batch costs the same; numpy fp64")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, w.L, w.B if args.batch is None else args.batch, keep, 1, args.decode == "indexed", None),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, L, B, keep, world, indexed, graphed, shared=False):
    k = max(1, min(w.d_ff, int(keep * w.d_ff + 0.5)))
    n_mats = 2 if w.act in ("relu", "gelu_tanh", "gelu_erf", "silu") else 3
    cfg = {"workload": f"{w.name} ({SHAPE_NOTE.get(w.name, w.name)})", "d": w.d, "d_ff": w.d_ff, "L": L, "S": w.S,
           "T": w.T, "B": B, "keep": keep, "k": k, "act": w.act,
           "parallelism": f"{world} independent replica(s), no collective",
           "l2": f"inputs larger than L2: {L} blocks of weights ({L * n_mats * w.d * w.d_ff * w.elem_bytes / 1e9:.1f} GB dense, "
                 f"{L * B * n_mats * k * w.d * w.elem_bytes / 1e9:.1f} GB compact) are visited in turn",
           "decode": ("index-direct: no compaction step, expert rows read in place from neuron-major full weights"
                      if indexed else "compact expert sets, one per sequence")}
    if shared:
        cfg["decode"] = "one compact expert set for the whole batch (Eq. 7): the first sequence's"
    if graphed is not None:
        cfg["decode_launch"] = ("the T x L decode calls of a step, captured once from the public API calls, are replayed as a CUDA graph"
                                if graphed else "one host launch per decode call")
    return cfg


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
class Job:
    """One workload resident on one GPU: the stack of blocks, its inputs and outputs, and the step."""

    def __init__(self, w, B, keep, L, dev, rank, indexed, use_graph, shared_set=False):
        import torch
        from paper_2404_01365_b200 import binding as G, synth
        from paper_2404_01365_b200.runner import FFStack
        self.torch, self.G = torch, G
        self.w, self.B, self.keep, self.L, self.dev, self.indexed = w, B, keep, L, dev, indexed
        self.T, self.S = w.T, w.S
        self.k = G.griffin_k_from_keep_ratio(w.d_ff, keep)
        self.stack = FFStack(w.d, w.d_ff, w.act, w.dtype, L, B, w.S, self.k, dev, indexed=indexed)
        for l in range(L):
            self.stack.add_block(*synth.make_weights(w, l, device=dev))
        seq0 = rank * B  # every rank has its own sequences
        self.X = torch.empty((L, B, w.S, w.d), device=dev, dtype=w.torch_dtype)
        self.XD = torch.empty((w.T, L, B, w.d), device=dev, dtype=w.torch_dtype)
        for l in range(L):
            for q in range(B):
                self.X[l, q] = synth.make_prompt(w, l, seq0 + q, device=dev)
                self.XD[:, l, q] = synth.make_decode_inputs(w, l, seq0 + q, device=dev)
        self.Y = torch.empty_like(self.X)
        self.YD = torch.empty_like(self.XD)
        self.shared_set = shared_set and not indexed and B > 1
        if self.shared_set:   # one compact set named for every sequence; its bytes are read once per call
            st = self.stack
            st.set_arrays = [G.compact_array([st.sets[l][0]] * B) for l in range(L)]
            per_seq = st.decode_bytes_per_call() // B
            shared_bytes = per_seq + (B - 1) * 2 * w.d * w.elem_bytes
            st.decode_bytes_per_call = lambda: shared_bytes
        self.stream = torch.cuda.current_stream()
        self.use_graph = use_graph
        self.graph = None
        self.launches_per_step = None

    def decode_loop(self):
        st = self.stack
        for t in range(self.T):
            for l in range(self.L):
                # the very first decode calls follow the kernels that write what they read (the compact
                # sets, or the index lists): launch them fully ordered
                if self.indexed:
                    st.decode_indexed(l, self.XD[t, l], self.YD[t, l], overlap=t > 0)
                else:
                    st.decode(l, self.XD[t, l], self.YD[t, l], overlap=t > 0)

    def capture(self, body):
        """Captures body() -- public API calls only -- into a CUDA graph; None if capture is unavailable."""
        torch = self.torch
        try:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(self.stream)
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    body()
            self.stream.wait_stream(side)
            torch.cuda.synchronize()
            return g
        except Exception as e:  # plain stream launches are always available
            sys.stderr.write(f"bench.py: graph capture failed ({e}); using stream launches\n")
            return None

    def step(self, ev=None, after_prompt=None, before_decode=None):
        st, stream = self.stack, self.stream
        if ev: ev[0].record(stream)
        for l in range(self.L):
            for q in range(self.B):
                st.prefill_score(l, q, self.X[l, q], self.Y[l, q])
        if ev: ev[1].record(stream)
        if after_prompt is not None: after_prompt()
        st.select_all()
        if ev: ev[2].record(stream)
        for l in range(0 if self.indexed else self.L):
            for q in range(self.B):
                st.compact(l, q)
        if ev: ev[3].record(stream)
        if before_decode is not None: before_decode()
        if self.graph is not None:
            self.graph.replay()
        else:
            self.decode_loop()
        if ev: ev[4].record(stream)

    def warm_up(self, n):
        """n untimed steps.  The first one runs eagerly and is the one whose kernel launches the library counts;
        after it the T x L decode calls of a step, which always touch the same buffers, are captured once into a
        CUDA graph that the later steps replay (the launches keep their programmatic-dependent-launch edges)."""
        G, torch = self.G, self.torch
        for i in range(max(1, n)):
            if i == 0:
                torch.cuda.synchronize()
                c0 = G.griffin_kernel_launches()
                self.step()
                self.launches_per_step = G.griffin_kernel_launches() - c0
                torch.cuda.synchronize()
                if self.use_graph:
                    self.graph = self.capture(self.decode_loop)
            else:
                self.step()
        torch.cuda.synchronize()
        if self.stack.status() != G.OK:
            raise RuntimeError("device status word raised during warm-up")

    def time_decode_only(self, set_arrays, B, reps):
        """Median microseconds per decode call of T x L calls that use the given per-block compact sets for the
        first B sequences' inputs (graph replay when available): the dense block, or batch 1 of a larger batch."""
        torch, G, st = self.torch, self.G, self.stack

        def loop():
            for t in range(self.T):
                for l in range(self.L):
                    G.griffin_ff_decode(st.desc, set_arrays[l], None, self.XD[t, l, :B], self.YD[t, l, :B], st.ws,
                                        G.DECODE_OVERLAP_WEIGHT_PREFETCH if t > 0 else G.DECODE_DEFAULT)
        loop()
        torch.cuda.synchronize()
        g = self.capture(loop) if self.use_graph else None
        us = []
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            g.replay() if g is not None else loop()
            e1.record(self.stream)
            torch.cuda.synchronize()
            us.append(e0.elapsed_time(e1) * 1e3 / (self.T * self.L))
        return statistics.median(us[1:])

    def dense_sets(self):
        """Per block, the full weights seen as a compact set with E = all neurons (one sequence)."""
        G, w = self.G, self.w
        out = []
        for fw in self.stack.weights:
            wg, wu, wd = fw._keep[0], fw._keep[1], fw._keep[2]
            out.append(G.compact_array([G.make_compact(wg, wu, wd, w.d_ff, w.d_ff)]))
        return out

    def time_compact_neuron_major(self, reps=2):
        """Median microseconds per (block, sequence) of the slicing step when the source of W_2_hat is the
        neuron-major W_2^T (transposed here once per block, as at model load): the same compact sets, bit for bit,
        from half the bytes of W_2."""
        torch, G, st = self.torch, self.G, self.stack
        nm = []
        for fw in st.weights:
            wg, wu, wd = fw._keep[0], fw._keep[1], fw._keep[2]
            nm.append(G.make_weights_nm(wg, wu, wd.t().contiguous()))
        us = []
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for l in range(self.L):
                for q in range(self.B):
                    G.griffin_compact_experts_nm(st.desc, nm[l], st.idx[l, q], st.sets[l][q], st.ws)
            e1.record(self.stream)
            torch.cuda.synchronize()
            us.append(e0.elapsed_time(e1) * 1e3 / (self.L * self.B))
        return statistics.median(us[1:])

    def first_sequence_sets(self):
        return [self.G.compact_array(self.stack.sets[l][:1]) for l in range(self.L)]


def phase_report(job, ph_ms, peaks):
    """Per-phase figures from the median per-step phase times (ms): prompt, top-k, compaction, decode."""
    hbm, burst, sust, _ = peaks
    st, w, L, B, T = job.stack, job.w, job.L, job.B, job.T
    pf_ms = ph_ms[0] / (L * B)
    tf = st.prefill_flops(w.S) / (pf_ms * 1e-3) / 1e12
    dec_us = ph_ms[3] / (T * L) * 1e3
    dec_gbs = st.decode_bytes_per_call() / (dec_us * 1e-6) / 1e9
    rep = {
        "prefill_score": {"us_per_block_and_sequence": pf_ms * 1e3, "tflops": tf, "frac_of_bf16_burst": tf / burst,
                          "frac_of_bf16_sustained": tf / sust},
        "select_topk": {"us_all_blocks": ph_ms[1] * 1e3, "problems": L * B},
        "compact": None,
        "decode": {"us_per_call": dec_us, "tokens_per_s_per_layer": B / (dec_us * 1e-6), "gbs": dec_gbs,
                   "frac_of_hbm": dec_gbs / hbm, "algorithmic_bytes_per_call": st.decode_bytes_per_call()},
    }
    if not job.indexed:
        c_us = ph_ms[2] / (L * B) * 1e3
        rep["compact"] = {"us_per_block_and_sequence": c_us, "gbs": st.compact_bytes() / (c_us * 1e-6) / 1e9,
                          "frac_of_hbm": st.compact_bytes() / (c_us * 1e-6) / 1e9 / hbm}
    return rep


def add_compact_nm(job, rep, peaks):
    if rep.get("compact") is not None:
        us = job.time_compact_neuron_major()
        gbs = job.stack.compact_bytes() / (us * 1e-6) / 1e9
        rep["compact"]["from_neuron_major_w_down"] = {"us_per_block_and_sequence": us, "gbs": gbs, "frac_of_hbm": gbs / peaks[0]}


def timed_steps(job, steps, barrier):
    """Times exactly `steps` steps between two barriers with events on the launching stream.  Returns the total
    milliseconds and the per-step phase times."""
    torch = job.torch
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e_begin.record(job.stream)
    t_host = time.perf_counter()
    for it in range(steps):
        job.step(evs[it])
    e_end.record(job.stream)
    host_s = time.perf_counter() - t_host
    barrier()
    per_step = [[evs[it][i].elapsed_time(evs[it][i + 1]) for i in range(4)] for it in range(steps)]
    return e_begin.elapsed_time(e_end), per_step, host_s


def median_phases(per_step):
    return [statistics.median(s[i] for s in per_step) for i in range(4)]


def release():
    """Returns freed device memory to the driver (call after dropping the last reference to a Job)."""
    import torch
    gc.collect()
    torch.cuda.empty_cache()


def section_entry(w, B, keep, dev, args, peaks, with_dense):
    """One entry of the workloads section: a few steps of the whole path on another shape."""
    import torch
    job = Job(w, B, keep, w.L, dev, 0, False, not args.no_graph)
    job.warm_up(1)
    total_ms, per_step, _ = timed_steps(job, args.section_steps, torch.cuda.synchronize)
    if job.stack.status() != job.G.OK:
        raise RuntimeError("device status word raised")
    rep = phase_report(job, median_phases(per_step), peaks)
    add_compact_nm(job, rep, peaks)
    entry = {"workload": w.name, "B": B, "keep": keep, "k": job.k, "L": w.L, "S": w.S, "T": w.T, "steps": args.section_steps,
             "ms_per_step": total_ms / args.section_steps,
             "tokens_per_s_per_layer": B * w.T * w.L / (total_ms / args.section_steps / 1e3), "phases": rep}
    if with_dense:
        dense_us = job.time_decode_only(job.dense_sets(), 1, 2)
        b1_us = rep["decode"]["us_per_call"] if B == 1 else job.time_decode_only(job.first_sequence_sets(), 1, 2)
        dbytes = job.stack.n_mats * w.d_ff * w.d * w.elem_bytes + 2 * w.d * w.elem_bytes
        entry["decode_dense"] = {"what": "keep 1.0 (E = all neurons) through the same decode kernel, batch 1",
                                 "us_per_call": dense_us, "gbs": dbytes / (dense_us * 1e-6) / 1e9,
                                 "frac_of_hbm": dbytes / (dense_us * 1e-6) / 1e9 / peaks[0]}
        entry["speedup_vs_dense"] = dense_us / b1_us
    job = None
    release()
    return entry


def shared_set_entry(w, keep, dev, args, peaks):
    """Decode with ONE expert set for the whole batch (the batch statistic of Eq. 7): the compact weights are
    streamed once per call whatever the batch, so the algorithmic bytes are those of one sequence plus the
    vectors.  Timed on the decode calls alone, T x L of them per repetition, for batches of 2, 4 and 8."""
    import torch
    job = Job(w, 8, keep, w.L, dev, 0, False, not args.no_graph)
    job.warm_up(1)                                   # fills the expert sets; the first sequence's is the one shared
    st, out = job.stack, {}
    for Bs in (2, 4, 8):
        arrays = [job.G.compact_array([st.sets[l][0]] * Bs) for l in range(w.L)]
        us = job.time_decode_only(arrays, Bs, 2)
        nbytes = st.n_mats * job.k * w.d * w.elem_bytes + Bs * 2 * w.d * w.elem_bytes
        out[f"B{Bs}"] = {"us_per_call": us, "tokens_per_s_per_layer": Bs / (us * 1e-6), "gbs": nbytes / (us * 1e-6) / 1e9,
                         "frac_of_hbm": nbytes / (us * 1e-6) / 1e9 / peaks[0], "algorithmic_bytes_per_call": nbytes}
    if job.stack.status() != job.G.OK:
        raise RuntimeError("device status word raised")
    job = None
    release()
    return {"workload": w.name, "keep": keep, "k": out and int(max(1, min(w.d_ff, int(keep * w.d_ff + 0.5)))), "L": w.L, "T": w.T,
            "what": "decode calls whose sequences all name one compact expert set", "decode": out}


def run_ours(args, w, keep):
    import torch
    import torch.distributed as dist
    from paper_2404_01365_b200 import binding as G, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    use_dist = "RANK" in os.environ and "MASTER_ADDR" in os.environ   # launched by torch.distributed.run
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)
    G.load()
    peaks = measured_peaks()

    def barrier():
        torch.cuda.synchronize()
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    L = args.layers or w.L
    B = args.batch or w.B
    indexed = args.decode == "indexed"
    job = Job(w, B, keep, L, dev, rank, indexed, not args.no_graph, shared_set=args.shared_set)
    job.stack.decode_flags = {"auto": 0, "ring": 4, "stream": 8}[args.decode_kernel]   # GRIFFIN_DECODE_RING / _STREAM
    T, S = job.T, job.S
    job.warm_up(args.warmup)
    barrier()

    sampler = ClockSampler(local)
    sampler.start()
    total_ms, per_step, host_s = timed_steps(job, args.steps, barrier)
    clocks = sampler.stop()
    if job.stack.status() != G.OK:
        raise RuntimeError("device status word raised during the timed region")
    ph_ms = median_phases(per_step)

    # ---- end to end: inputs start in pinned host memory, outputs end there ------------------
    e2e = None
    if not args.no_e2e:
        stream = job.stream
        pinned = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        Xh, XDh, Yh, YDh = pinned(job.X), pinned(job.XD), pinned(job.Y), pinned(job.YD)
        Xh.copy_(job.X)
        XDh.copy_(job.XD)
        # Every copy of a step is inside the timed region; the two that the phase running at the time does not
        # depend on go over copy streams of their own (the decode inputs come in under the prompt phase, the
        # prompt outputs leave under the decode phase), and the step ends when all of them have.
        copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()

        def prompt_outputs_leave():
            copy_out.wait_stream(stream)            # the prompt phase has written Y
            with torch.cuda.stream(copy_out):
                Yh.copy_(job.Y, non_blocking=True)

        def step_e2e():
            job.X.copy_(Xh, non_blocking=True)
            copy_in.wait_stream(stream)             # the previous step's decode has read XD
            with torch.cuda.stream(copy_in):
                job.XD.copy_(XDh, non_blocking=True)
            job.step(after_prompt=prompt_outputs_leave, before_decode=lambda: stream.wait_stream(copy_in))
            YDh.copy_(job.YD, non_blocking=True)
            stream.wait_stream(copy_out)
        n_e2e = min(args.steps, 5)
        step_e2e()
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record(stream)
        for _ in range(n_e2e):
            step_e2e()
        b1.record(stream)
        barrier()
        nbytes = lambda t: t.numel() * t.element_size()
        e2e = [b0.elapsed_time(b1) / n_e2e, nbytes(Xh) + nbytes(XDh), nbytes(Yh) + nbytes(YDh), n_e2e]
        Xh = XDh = Yh = YDh = None

    # ---- max over ranks ----------------------------------------------------------------------
    vals = torch.tensor([total_ms] + ph_ms + ([e2e[0]] if e2e else [0.0]), device=dev, dtype=torch.float64)
    if use_dist:
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
    total_ms, ph_ms, e2e_ms = float(vals[0]), [float(v) for v in vals[1:5]], float(vals[5])

    line = None
    if rank == 0:
        K = args.steps
        ms_per_step = total_ms / K
        tokens = world * B * T * L
        rep = phase_report(job, ph_ms, peaks)
        if world == 1:
            add_compact_nm(job, rep, peaks)
        dec = rep["decode"]
        traffic_key = f"{w.name}_B{B}_keep{keep}"
        line = {
            "metric": METRIC, "value": tokens / (ms_per_step / 1e3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": workload_config(w, L, B, keep, world, indexed, job.graph is not None, job.shared_set),
            "phases": dict(rep, note="medians over the timed steps of per-phase CUDA-event times"),
            "roofline": {"bound": "hbm", "kernel": ("decode_indexed_kernel" if indexed else
                                                    "decode_shared_kernel" if job.shared_set else
                                                    decode_kernel_name(w, B, job.k, args.decode_kernel)) +
                         " (one launch per decode call; the decode phase is "
                         f"{100.0 * ph_ms[3] / sum(ph_ms):.0f} % of the step)", "achieved": dec["gbs"],
                         "peak": peaks[0], "unit": "GB/s", "frac": dec["frac_of_hbm"], "peak_source": peaks[3],
                         "algorithmic_bytes_per_launch": dec["algorithmic_bytes_per_call"],
                         "traffic": None if indexed or job.shared_set else
                         recorded_traffic(traffic_key, decode_kernel_name(w, B, job.k, args.decode_kernel))},
            "clocks": clocks,
            "gpu_launches": job.launches_per_step * K,
            "gpu_launches_per_step": job.launches_per_step,
            "host_issue_s": host_s,
        }
        if e2e:
            line["e2e"] = {"value": tokens / (e2e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": e2e[1],
                           "d2h_bytes_per_step": e2e[2], "steps": e2e[3]}
    if rank == 0 and world == 1 and not indexed and w.dtype == "bf16" and not job.shared_set:
        # decode of the unpruned block (keep 1.0) through the same kernel, and of one pruned sequence: the
        # speed-up that pruning half of the neurons buys at batch 1 (the byte ratio is 2)
        dense_us = job.time_decode_only(job.dense_sets(), 1, 3)
        b1_us = rep["decode"]["us_per_call"] if B == 1 else job.time_decode_only(job.first_sequence_sets(), 1, 3)
        dbytes = job.stack.n_mats * w.d_ff * w.d * w.elem_bytes + 2 * w.d * w.elem_bytes
        b1_bytes = job.stack.decode_bytes_per_call() // B
        line["decode_dense"] = {"what": "keep 1.0 (E = all neurons) through the same decode kernel, batch 1",
                                "us_per_call": dense_us, "gbs": dbytes / (dense_us * 1e-6) / 1e9,
                                "frac_of_hbm": dbytes / (dense_us * 1e-6) / 1e9 / peaks[0]}
        line["decode_batch1"] = {"what": f"keep {keep}, one sequence's expert set, batch 1", "us_per_call": b1_us,
                                 "gbs": b1_bytes / (b1_us * 1e-6) / 1e9, "frac_of_hbm": b1_bytes / (b1_us * 1e-6) / 1e9 / peaks[0]}
        line["speedup_vs_dense"] = dense_us / b1_us
    job = None
    release()

    if rank == 0 and world == 1 and not args.no_workloads and not indexed and not args.shared_set:
        sect = []
        W = synth.WORKLOADS
        for name, with_dense in (("llama2_7b", True), ("gemma_7b", True), ("llama2_13b", True)):
            sect.append(section_entry(W[name], 1, 0.5, dev, args, peaks, with_dense))
        for kp in W["mistral_7b"].keeps:
            sect.append(section_entry(W["mistral_7b"], W["mistral_7b"].B, kp, dev, args, peaks, False))
        line["workloads"] = sect
        line["shared_expert_set"] = shared_set_entry(W["llama2_7b"], 0.5, dev, args, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, keep)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def start_ranks(args):
    """`--gpus N` outside torch.distributed.run: start the N ranks on this node, one per GPU."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(start_ranks(args))
    from paper_2404_01365_b200 import synth
    w = synth.WORKLOADS[args.workload]
    keep = args.keep if args.keep is not None else 0.5
    if args.impl == "reference":
        run_reference(args, w, keep)
    else:
        run_ours(args, w, keep)


if __name__ == "__main__":
    main()
