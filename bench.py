#!/usr/bin/env python
"""Benchmark of the GRIFFIN feed-forward hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input, for a stack of L
independent FF blocks shaped like the named model:
    prompt phase (full FF + statistic) for every block  ->  top-k for every block
    ->  expert compaction for every block  ->  T decode steps, each through all L blocks.
The weights of all blocks stay resident in HBM (they are the model); the hidden states are the
step's input.  All L blocks are visited in turn, so every weight byte comes from HBM, not L2.

Prints ONE JSON line (rank 0).  `value` = generated tokens per second per block for the whole
step (B*T*L / step time, summed over ranks: every rank runs its own sequences, there is no
exchange between ranks).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b")
    ap.add_argument("--keep", type=float, default=None)
    ap.add_argument("--layers", type=int, default=None, help="override the number of blocks (smaller footprint)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every decode call from the host instead of replaying a CUDA graph")
    ap.add_argument("--decode", default="compact", choices=["compact", "indexed"],
                    help="indexed: no compaction step, the decode calls read the expert rows in place from the full weights")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def measured_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s from MEASURED_PEAKS.json, else the machine's fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(p))
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"])
    except Exception:
        return 1590.0, 1400.0


def down_projection_splits(S, d, d_ff):
    """How many K splits the library's down projection takes for this shape (its own rule, restated here
    only to count the launches of a step: with a split there is one more kernel per prompt)."""
    bn = 256 if d % 256 == 0 else 128
    tiles = ((S + 127) // 128) * (d // bn)
    tile_us = 2.0 * 128 * bn * d_ff / 10e12 * 1e6
    cost1 = best_cost = None
    best = 1
    for sp in range(1, 5):
        rounds = (tiles * sp + 147) // 148
        cost = rounds * tile_us / sp
        if sp > 1:
            cost += 2.0 * sp * S * d * 4.0 / 4e12 * 1e6 + 3.0
        if sp == 1:
            cost1 = best_cost = cost
        elif cost < 0.9 * cost1 and cost < best_cost:
            best_cost, best = cost, sp
    return best


def down_projection_tail_cut(S, d, d_ff):
    """Whether the library cuts the last round of the down projection's tiles along K (one more kernel per
    prompt); its rule, restated to count launches."""
    if d % 256 != 0 or down_projection_splits(S, d, d_ff) != 1:
        return False
    tiles = ((S + 127) // 128) * (d // 256)
    rem = tiles % 148
    return tiles > 148 and 0 < rem and 2 * rem <= 148 and d_ff // 64 >= 16


def recorded_traffic():
    """DRAM bytes per decode call from the committed ncu summary, if the kernel source is
    unchanged since that capture; otherwise None."""
    p = os.path.join(ROOT, "profiles", "decode_traffic.json")
    try:
        rec = json.load(open(p))
        h = hashlib.sha1()
        for name in rec["sources"]:
            h.update(open(os.path.join(ROOT, name), "rb").read())
        if h.hexdigest() == rec["sha1"]:
            return rec
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
# CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# --------------------------------------------------------------------------------------------
def oracle_sample(w, keep, layer, T_sample):
    """The oracle, as it stands, on one block of the workload: prompt phase, statistic, top-k,
    slicing and T_sample decode steps.  Returns (seconds, tokens)."""
    import numpy as np
    from oracle import griffin_oracle as O
    from paper_2404_01365_b200 import synth
    wg, wu, wd = (None if t is None else t.double().numpy() for t in synth.make_weights(w, layer))
    x = synth.make_prompt(w, layer, 0).double().numpy()
    xd = synth.make_decode_inputs(w, layer, 0, T=T_sample).double().numpy()
    k = O.k_from_keep_ratio(w.d_ff, keep)
    t0 = time.perf_counter()
    y, z = O.ff_dense(x, wg, wu, wd, w.act)
    s = O.flock_score(z)
    e = O.select_topk(s, k)
    c = O.compact_experts(e, wg, wu, wd)
    for t in range(T_sample):
        O.ff_pruned(xd[t], c, w.act)
    return time.perf_counter() - t0, T_sample


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, w, keep):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    T_sample = min(w.T, 128)
    times = []
    for i in range(args.warmup + args.steps):
        sec, tok = oracle_sample(w, keep, i % w.L, T_sample)
        if i >= args.warmup:
            times.append(sec)
    ms = 1e3 * sum(times) / len(times)
    value = T_sample / (ms / 1e3)  # tokens per second per block, one block per step
    sample = f"one block per step (prompt S={w.S}, top-k, slicing, {T_sample} of {w.T} decode steps, batch 1), numpy fp64"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "d": w.d, "d_ff": w.d_ff, "S": w.S, "T": w.T, "B": 1, "L": w.L, "keep": keep,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def run_ours(args, w, keep):
    import torch
    import torch.distributed as dist
    from paper_2404_01365_b200 import binding as G, synth
    from paper_2404_01365_b200.runner import FFStack

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

    L = args.layers or w.L
    B, T, S = w.B, w.T, w.S
    k = G.griffin_k_from_keep_ratio(w.d_ff, keep)
    indexed = args.decode == "indexed"
    stack = FFStack(w.d, w.d_ff, w.act, w.dtype, L, B, S, k, dev, indexed=indexed)
    for l in range(L):
        stack.add_block(*synth.make_weights(w, l, device=dev))
    seq0 = rank * B  # every rank has its own sequences
    X = torch.stack([torch.stack([synth.make_prompt(w, l, seq0 + q, device=dev) for q in range(B)]) for l in range(L)])
    XD = torch.stack([torch.stack([synth.make_decode_inputs(w, l, seq0 + q, device=dev) for q in range(B)], 1)
                      for l in range(L)], 1).contiguous()          # [T, L, B, d]
    Y = torch.empty_like(X)                                          # [L, B, S, d]
    YD = torch.empty_like(XD)
    stream = torch.cuda.current_stream()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(max(1, args.steps))]

    def step(ev=None, after_prompt=None, before_decode=None):
        record = ev is not None
        if record: ev[0].record(stream)
        for l in range(L):
            for q in range(B):
                stack.prefill_score(l, q, X[l, q], Y[l, q])
        if record: ev[1].record(stream)
        if after_prompt is not None: after_prompt()
        stack.select_all()
        if record: ev[2].record(stream)
        for l in range(0 if indexed else L):
            for q in range(B):
                stack.compact(l, q)
        if record: ev[3].record(stream)
        if before_decode is not None: before_decode()
        if dec_graph[0] is not None:
            dec_graph[0].replay()
        else:
            decode_loop()
        if record: ev[4].record(stream)

    def decode_loop():
        for t in range(T):
            for l in range(L):
                # the very first decode calls follow the kernels that write what they read (the compact
                # sets, or the index lists): launch them fully ordered
                if indexed:
                    stack.decode_indexed(l, XD[t, l], YD[t, l], overlap=t > 0)
                else:
                    stack.decode(l, XD[t, l], YD[t, l], overlap=t > 0)

    # The T x L decode calls of a step always touch the same buffers: after the first warm-up step
    # they are captured once, through the same public API calls, into a CUDA graph that the
    # later steps replay (the launches keep their programmatic-dependent-launch edges).
    dec_graph = [None]

    def capture_decode():
        try:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    decode_loop()
            stream.wait_stream(side)
            torch.cuda.synchronize()
            dec_graph[0] = g
        except Exception as e:  # plain stream launches are always available
            sys.stderr.write(f"bench.py: decode graph capture failed ({e}); using stream launches\n")
            dec_graph[0] = None

    def barrier():
        torch.cuda.synchronize()
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step()
        if i == 0 and not args.no_graph:
            torch.cuda.synchronize()
            capture_decode()
    barrier()
    if stack.status() != G.OK:
        raise RuntimeError("device status word raised during warm-up")

    sampler = ClockSampler(local)
    sampler.start()
    phase_ms = [0.0] * 4
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e_begin.record(stream)
    t_host = time.perf_counter()
    for it in range(args.steps):
        step(evs[it])
    e_end.record(stream)
    host_s = time.perf_counter() - t_host
    barrier()
    for it in range(args.steps):
        for i in range(4):
            phase_ms[i] += evs[it][i].elapsed_time(evs[it][i + 1])
    clocks = sampler.stop()
    total_ms = e_begin.elapsed_time(e_end)
    if stack.status() != G.OK:
        raise RuntimeError("device status word raised during the timed region")

    # ---- end to end: inputs start in pinned host memory, outputs end there ------------------
    e2e = None
    if not args.no_e2e:
        Xh, XDh = X.cpu().pin_memory(), XD.cpu().pin_memory()
        Yh, YDh = torch.empty_like(Xh).pin_memory(), torch.empty_like(XDh).pin_memory()
        # Every copy of a step is inside the timed region; the two that the phase running at the time does not
        # depend on go over copy streams of their own (the decode inputs come in under the prompt phase, the
        # prompt outputs leave under the decode phase), and the step ends when all of them have.
        copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()

        def prompt_outputs_leave():
            copy_out.wait_stream(stream)            # the prompt phase has written Y
            with torch.cuda.stream(copy_out):
                Yh.copy_(Y, non_blocking=True)

        def step_e2e():
            X.copy_(Xh, non_blocking=True)
            copy_in.wait_stream(stream)             # the previous step's decode has read XD
            with torch.cuda.stream(copy_in):
                XD.copy_(XDh, non_blocking=True)
            step(after_prompt=prompt_outputs_leave, before_decode=lambda: stream.wait_stream(copy_in))
            YDh.copy_(YD, non_blocking=True)
            stream.wait_stream(copy_out)
        step_e2e()
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record(stream)
        for _ in range(args.steps):
            step_e2e()
        b1.record(stream)
        barrier()
        e2e_ms = b0.elapsed_time(b1)
        e2e = [e2e_ms, Xh.numel() * Xh.element_size() + XDh.numel() * XDh.element_size(),
               Yh.numel() * Yh.element_size() + YDh.numel() * YDh.element_size()]

    # ---- max over ranks ----------------------------------------------------------------------
    vals = torch.tensor([total_ms] + phase_ms + ([e2e[0]] if e2e else [0.0]), device=dev, dtype=torch.float64)
    if use_dist:
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
    total_ms, phase_ms, e2e_ms = float(vals[0]), [float(v) for v in vals[1:5]], float(vals[5])

    if rank == 0:
        K = args.steps
        ms_per_step = total_ms / K
        tokens = world * B * T * L
        value = tokens / (ms_per_step / 1e3)
        peak, peak_src = measured_peak()
        tensor_peaks = measured_tensor_peaks()
        dec_ms_per_call = phase_ms[3] / K / (T * L)
        dec_bytes = stack.decode_bytes_per_call()
        achieved = dec_bytes / (dec_ms_per_call * 1e-3) / 1e9
        traffic = recorded_traffic()
        pf_ms = phase_ms[0] / K / (L * B)
        # kernels launched per step: prompt phase = 2 GEMM kernels (+1 when the down projection is
        # K-split, i.e. when its 128x256 tiles number at most half the SMs) + 3 statistic kernels;
        # one top-k launch for all blocks; 1 compaction kernel; one fused kernel per decode call
        # (two for fp32 storage)
        m_tiles = (S + 127) // 128
        split = w.dtype == "bf16" and down_projection_splits(S, w.d, w.d_ff) > 1
        # ... and the finishing kernel of the first GEMM when its last round of tiles is cut along K
        gated = G.act_is_gated(w.act)
        g1_tiles = m_tiles * (w.d_ff // 128 if gated else w.d_ff // 256)
        cut = (w.dtype == "bf16" and w.d % 128 == 0 and w.d_ff % (128 if gated else 256) == 0 and 148 < g1_tiles <= 4 * 148
               and 0 < g1_tiles % 148 <= 74 and w.d // 64 >= 16)
        cut2 = w.dtype == "bf16" and w.d % 128 == 0 and w.d_ff % (128 if gated else 256) == 0 and down_projection_tail_cut(S, w.d, w.d_ff)
        launches = (L * B * (5 + (1 if split else 0) + (1 if cut else 0) + (1 if cut2 else 0)) + 1 + (0 if indexed else L * B) +
                    T * L * (1 if w.dtype == "bf16" else 2))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": f"{w.name} (Llama-2-7B-shaped SwiGLU FF)" if w.name == "llama2_7b" else w.name,
                       "d": w.d, "d_ff": w.d_ff, "L": L, "S": S, "T": T, "B": B, "keep": keep, "k": k,
                       "parallelism": f"{world} independent replica(s), no collective",
                       "l2": f"inputs larger than L2: {L} blocks of weights ({L * 3 * w.d * w.d_ff * w.elem_bytes / 1e9:.1f} GB dense, "
                             f"{L * B * 3 * k * w.d * w.elem_bytes / 1e9:.1f} GB compact) are visited in turn",
                       "decode": ("index-direct: no compaction step, expert rows read in place from neuron-major full weights"
                                  if indexed else "compact expert sets"),
                       "decode_launch": ("the T x L decode calls of a step, captured once from the public API calls, are replayed as a CUDA graph"
                                         if dec_graph[0] is not None else "one host launch per decode call")},
            "phases": {
                "prefill_score": {"ms_per_block": pf_ms, "tflops": stack.prefill_flops(S) / (pf_ms * 1e-3) / 1e12,
                                  "frac_of_bf16_burst": stack.prefill_flops(S) / (pf_ms * 1e-3) / 1e12 / tensor_peaks[0],
                                  "frac_of_bf16_sustained": stack.prefill_flops(S) / (pf_ms * 1e-3) / 1e12 / tensor_peaks[1]},
                "select_topk": {"ms_all_blocks": phase_ms[1] / K},
                "compact": (None if indexed else
                            {"ms_per_block": phase_ms[2] / K / (L * B),
                             "gbs": stack.compact_bytes() / (phase_ms[2] / K / (L * B) * 1e-3) / 1e9}),
                "decode": {"us_per_call": dec_ms_per_call * 1e3, "tokens_per_s_per_layer": B / (dec_ms_per_call * 1e-3),
                           "gbs": achieved},
            },
            "roofline": {"bound": "hbm", "kernel": ("decode_indexed_kernel" if indexed else "decode_fused_kernel") +
                         " (one launch per decode call)", "achieved": achieved,
                         "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": dec_bytes,
                         "traffic": traffic["dram_bytes_per_decode_call"] if traffic and not indexed else None},
            "clocks": clocks,
            "gpu_launches": launches,
            "host_issue_s": host_s,
        }
        if e2e:
            line["e2e"] = {"value": tokens / (e2e_ms / K / 1e3), "unit": UNIT, "h2d_bytes_per_step": e2e[1],
                           "d2h_bytes_per_step": e2e[2]}
        if world == 1 and not args.no_cpu_baseline:
            T_sample, sec, tok, blocks = min(T, 128), 0.0, 0, 0
            while blocks < min(L, 24) and sec < 15.0:   # a bounded sample: 10-30 s of CPU work
                s1, t1 = oracle_sample(w, keep, blocks, T_sample)
                sec, tok, blocks = sec + s1, tok + t1, blocks + 1
            line["cpu_baseline"] = {
                "value": tok / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                "sample": f"{blocks} of {L} blocks, each: prompt S={S}, top-k, slicing, {T_sample} of {T} decode steps, "
                          f"batch 1; numpy fp64; {sec:.1f} s"}
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2404_01365_b200 import synth
    w = synth.WORKLOADS[args.workload]
    keep = args.keep if args.keep is not None else 0.5
    if args.impl == "reference":
        run_reference(args, w, keep)
    else:
        run_ours(args, w, keep)


if __name__ == "__main__":
    main()
