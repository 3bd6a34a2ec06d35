"""Host-side check of the index arithmetic of the register-streaming decode kernel (csrc/decode_stream.cu).

The kernel deals the B * P pairs of a half to the CTAs as contiguous ranges and a CTA's range, counted in steps, to
its 16 warps as contiguous ranges.  The formulas are restated here in integers and checked for what the kernel
relies on: every step of every pair is taken exactly once, a CTA's range spans at most two sequences, the pieces
of a cut pair follow each other in the order of the partial-sum entries (2 * warp + slot), and no address computed
from (pair, step, lane) leaves its row."""
import itertools

import pytest

ST_WARPS, ST_H = 16, 4
STEP_UNITS = 32 * ST_H
GATE_UP, DOWN, UP = 0, 1, 2


def geom(mode, d, k, ldk):
    rows = d if mode == DOWN else k
    P = rows if mode == GATE_UP else (rows + 1) // 2
    row_units = (ldk if mode == DOWN else d) // 8
    S = (row_units + STEP_UNITS - 1) // STEP_UNITS
    return rows, P, row_units, S


def cta_range(B, P, cta, grid):
    T = B * P
    return T * cta // grid, T * (cta + 1) // grid


def warp_steps(lo, hi, S, warp):
    n = (hi - lo) * S
    return n * warp // ST_WARPS, n * (warp + 1) // ST_WARPS


SHAPES = [  # d, k, ldk, B
    (4096, 5504, 5504, 1), (5120, 6912, 6912, 8), (3072, 12288, 12288, 2), (4096, 7168, 7168, 4),
    (64, 37, 40, 3), (128, 1, 8, 2), (136, 9, 16, 5), (256, 344, 344, 32), (8192, 512, 512, 1), (1000, 751, 752, 2),
]


@pytest.mark.parametrize("d,k,ldk,B", SHAPES)
@pytest.mark.parametrize("mode", [GATE_UP, DOWN, UP])
@pytest.mark.parametrize("grid", [148, 132, 7])
def test_every_step_is_taken_once_and_ranges_span_two_sequences_at_most(d, k, ldk, B, mode, grid):
    if B > grid:
        pytest.skip("the launcher hands such a call to the ring kernel (a range could span three sequences)")
    rows, P, row_units, S = geom(mode, d, k, ldk)
    taken = {}
    for cta in range(grid):
        lo, hi = cta_range(B, P, cta, grid)
        assert 0 <= lo <= hi <= B * P
        if hi > lo:
            assert (hi - 1) // P - lo // P <= 1          # two vectors are staged: sequences b0 and b0 + 1
        entries = []                                       # (entry index, pair) of the partial sums, in entry order
        for warp in range(ST_WARPS):
            s0, s1 = warp_steps(lo, hi, S, warp)
            mid = s0 % S != 0
            for s in range(s0, s1):
                f, sp = lo + s // S, s % S
                assert lo <= f < hi
                taken[(f, sp)] = taken.get((f, sp), 0) + 1
                last_of_pair, last_of_warp = sp == S - 1, s == s1 - 1
                if last_of_pair or last_of_warp:
                    if not (last_of_pair and not mid):
                        entries.append((2 * warp + (0 if mid else 1), f))
                    mid = False
        # the pieces of one pair are consecutive among the entries, which are in increasing entry order
        assert [e for e, _ in entries] == sorted(e for e, _ in entries)
        assert len(set(e for e, _ in entries)) == len(entries)
        pairs_seen = [f for f, _ in itertools.groupby(f for _, f in entries)]
        assert len(pairs_seen) == len(set(pairs_seen))
    assert len(taken) == B * P * S and all(v == 1 for v in taken.values())
    # addresses: unit (sp * STEP_UNITS + i * 32 + lane) is loaded only when it is inside the row
    for sp, i, lane in itertools.product(range(S), range(ST_H), (0, 31)):
        u = sp * STEP_UNITS + i * 32 + lane
        full_step = (sp + 1) * STEP_UNITS <= row_units
        assert not full_step or u < row_units


def pool_chunks(B, k, gated, grid, d=4096, pct=8, min_pairs_per_warp=16):
    """The launcher's rule for the pool of the first half (pairs handed out at run time, 16 at a time)."""
    per_seq = k if gated else (k + 1) // 2
    pairs = B * per_seq
    if pairs // (grid * ST_WARPS) < min_pairs_per_warp or d // 8 <= 3 * STEP_UNITS:
        return 0
    return min(per_seq, pairs * pct // 100) // ST_WARPS


@pytest.mark.parametrize("B,k,gated", [(8, 6912, True), (8, 6912, False), (32, 5504, True), (4, 7168, True), (16, 24576, True)])
def test_the_pool_lies_in_the_last_sequence_and_the_rest_is_dealt_out_as_before(B, k, gated):
    grid = 148
    per_seq = k if gated else (k + 1) // 2
    T = B * per_seq
    n = pool_chunks(B, k, gated, grid)
    if T // (grid * ST_WARPS) < 16:                      # e.g. the Mistral shape with 4 sets: 12 pairs per warp
        assert n == 0
        return
    assert n > 0
    pool_base = T - n * ST_WARPS
    assert pool_base // per_seq == B - 1 and (T - 1) // per_seq == B - 1      # one vector (the third slot) serves the pool
    covered = 0
    for cta in range(grid):
        lo, hi = (T - n * ST_WARPS) * cta // grid, (T - n * ST_WARPS) * (cta + 1) // grid
        covered += hi - lo
        if hi > lo:
            assert (hi - 1) // per_seq - lo // per_seq <= 1
    assert covered == pool_base and covered + n * ST_WARPS == T
    # the claims of one call take the counter round: n successful ones and one failing per CTA
    counter, limit = 0, n + grid - 1
    for _ in range(n + grid):
        counter = 0 if counter >= limit else counter + 1
    assert counter == 0


def test_the_size_rule_of_the_bench_names_the_kernel_the_library_picks():
    import bench
    from paper_2404_01365_b200 import synth
    w7, w13 = synth.WORKLOADS["llama2_7b"], synth.WORKLOADS["llama2_13b"]
    assert bench.decode_kernel_name(w7, 1, 5504) == "decode_fused_kernel"       # 135 MB: the ring
    assert bench.decode_kernel_name(w7, 2, 5504) == "decode_stream_kernel"      # 271 MB
    assert bench.decode_kernel_name(w13, 8, 6912) == "decode_stream_kernel"
    assert bench.decode_kernel_name(synth.WORKLOADS["tiny_swiglu_f32"], 1, 344).startswith("decode_gate_up_kernel")
