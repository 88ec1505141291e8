"""CPU: the work distribution of the chunked kernel (host arithmetic shared with the kernel).  Every (unit, chunk)
must be processed exactly once; a tile split between two runs must have its head processed before its tail is
reached, so that no block ever waits for another; and the layout chosen for the benchmark shapes is the expected one."""
import random

import pytest

from paper_2609_39034_b200 import binding, workloads as wl


def _runs(units, nch, per):
    nruns = (units * nch + per - 1) // per
    return [binding.chunk_run_pieces(units, nch, per, r) for r in range(nruns)]


def _check_runs(units, nch, per):
    runs = _runs(units, nch, per)
    assert binding.chunk_run_pieces(units, nch, per, len(runs)) == []  # nothing past the end
    seen = {}
    head_done, tail_start = {}, {}
    for r, pieces in enumerate(runs):
        assert pieces, r
        t = 0
        for i, (u, cb, ce) in enumerate(pieces):
            assert 0 <= u < units and 0 <= cb < ce <= nch
            for c in range(cb, ce):
                assert (u, c) not in seen, (u, c)
                seen[(u, c)] = r
            if cb > 0:  # a tail: reaches the end of its unit, comes last, needs another run's head
                assert ce == nch and i == len(pieces) - 1
                tail_start[u] = (r, t)
            if ce < nch:  # a head: starts the unit, comes first, leaves its state to another run
                assert cb == 0 and i == 0
                head_done[u] = (r, t + ce - cb)
            t += ce - cb
        assert t <= per
    assert len(seen) == units * nch
    for u, (r_tail, t_tail) in tail_start.items():
        assert u in head_done, u
        r_head, t_head = head_done[u]
        assert r_head == r_tail - 1          # the dependency chain is one link long: no cycles
        # in step with each other the tail never waits -- except in a last, shortened run that holds nothing but
        # the tail, which then still ends within the length of a full run
        last_short = r_tail == len(runs) - 1 and len(runs[r_tail]) == 1
        assert t_head <= t_tail or (last_short and t_head + (nch - runs[r_tail][0][1]) <= per)
    assert set(head_done) == set(tail_start)


@pytest.mark.parametrize("cfg", [1, 2])
def test_benchmark_shapes_on_148_sms(cfg):
    w = wl.CONFIGS[cfg]
    pl = binding.chunk_plan(w.B, w.H, w.T, w.Dv, w.J, 148, True)
    nslice = w.Dv // (128 // w.J)
    assert pl["nch"] == w.T // 32
    if cfg == 2:  # 64 (batch, head) units on 37 gangs of 4 blocks: 443 chunks per run instead of 2 x 256
        assert pl == {"split": 1, "gang": 4, "nch": 256, "per": 443, "units": 64, "grid": 148}
    if pl["split"]:
        assert pl["gang"] == nslice and pl["grid"] <= 148 and pl["per"] >= pl["nch"]
        _check_runs(pl["units"], pl["nch"], pl["per"])
    # without a state output a split tile would have nowhere to leave its state
    plain = binding.chunk_plan(w.B, w.H, w.T, w.Dv, w.J, 148, False)
    assert plain["split"] == 0 and plain["grid"] == w.B * w.H * nslice and plain["per"] == plain["nch"]


def test_no_split_when_it_does_not_pay():
    # fewer tiles than SMs, a whole number of waves, short sequences
    assert binding.chunk_plan(1, 8, 4096, 128, 4, 148)["split"] == 0
    assert binding.chunk_plan(37, 2, 4096, 128, 4, 148)["split"] == 0   # 296 tiles = exactly two waves
    assert binding.chunk_plan(4, 16, 256, 128, 4, 148)["split"] == 0    # 8 chunks per tile


def test_random_layouts_cover_everything_once_and_never_wait():
    rng = random.Random(1234)
    for _ in range(300):
        nch = rng.randint(1, 40)
        units = rng.randint(1, 60)
        per = rng.randint(nch, 3 * nch + 5)  # the plan only ever uses per >= nch
        _check_runs(units, nch, per)


def test_one_tile_per_block_layout():
    for units, nch in ((5, 7), (1, 1), (13, 256)):
        runs = _runs(units, nch, nch)
        assert runs == [[(u, 0, nch)] for u in range(units)]


def test_probe_rejects_bad_arguments():
    with pytest.raises(Exception):
        binding.chunk_plan(4, 16, 8192, 128, 2, 148)      # J = 2 has no chunked kernel
    with pytest.raises(Exception):
        binding.chunk_run_pieces(0, 4, 4, 0)
