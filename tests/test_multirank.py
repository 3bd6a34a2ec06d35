"""The N > 1 path on CPU: two gloo ranks shard the independent (block, sequence) units, each
computes its own sequences with no exchange, and the job-level figures are the max of the
times and the sum of the tokens, exactly as bench.py combines them."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2404_01365_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.scaled(synth.WORKLOADS["llama2_13b"], d=64, d_ff=96, S=8, T=4, L=3)
    B = w.B
    seqs = list(range(rank * B, (rank + 1) * B))                 # bench.py: sequence offset = rank * B
    units = list(synth.shard_units(w.L * world * B, rank, world))  # the same split through shard_units
    x = torch.stack([synth.make_prompt(w, 0, q) for q in seqs])
    fake_ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)
    tokens = torch.tensor([float(B * w.T * w.L)], dtype=torch.float64)
    dist.barrier()
    dist.all_reduce(fake_ms, op=dist.ReduceOp.MAX)
    dist.all_reduce(tokens, op=dist.ReduceOp.SUM)
    gathered = [None] * world
    dist.all_gather_object(gathered, (seqs, units, float(x.double().sum())))
    if rank == 0:
        out.put((float(fake_ms), float(tokens), gathered))
    dist.destroy_process_group()


def test_two_ranks_take_disjoint_sequences_and_combine_like_the_bench():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    ms, tokens, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0                                   # max over ranks
    assert tokens == 2 * 8 * 4 * 3                      # sum over ranks
    seq_sets = [set(g[0]) for g in gathered]
    assert seq_sets[0].isdisjoint(seq_sets[1]) and len(seq_sets[0] | seq_sets[1]) == 16
    all_units = sorted(u for g in gathered for u in g[1])
    assert all_units == list(range(3 * 2 * 8))          # every unit owned exactly once
    assert gathered[0][2] != gathered[1][2]             # different sequences, different inputs
