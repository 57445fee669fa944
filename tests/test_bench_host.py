"""Host-side logic of bench.py: unit sharding, the max-over-ranks reduction on a 2-rank gloo
group (the multi-GPU path of the benchmark runs independent replicas, so this is all the
cross-rank traffic there is), the algorithmic work formulas and the clock-sample parser."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
import esa_synth as syn  # noqa: E402


def test_shard_units_partitions_everything_once():
    for total in (0, 1, 7, 32, 257):
        for world in (1, 2, 3, 8):
            spans = [bench.shard_units(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = bench.shard_units(32, rank, world)              # layers of the stack, one share per rank
        mine = 10.0 + 5.0 * rank                                  # this rank's time for its replica
        worst = bench.max_over_ranks(mine)
        t = torch.tensor([float(hi - lo)])
        dist.all_reduce(t)
        out.put((rank, worst, float(t[0])))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_on_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]        # every rank sees the slowest rank's time
    assert [r[2] for r in res] == [32.0, 32.0]        # the shares cover the 32 layers


def test_max_over_ranks_without_a_group_is_identity():
    assert bench.max_over_ranks(3.5) == 3.5


def test_work_formulas_match_the_papers_counts():
    cfg = syn.get_config("c5")
    t, l_C = 255 * 512, 512
    n_att = 128 + 4096 + 2048 + 512
    # Appendix A: QK^T and PV of the sparse attention, 4 d_H flops per (query, key) pair
    assert bench.attend_flops(cfg, t, l_C) == 4.0 * cfg.d_H * l_C * (n_att - l_C / 2.0)
    l_M = t - 2048 - 128
    assert bench.score_flops(cfg, t, l_C) == (2.0 * 128 + 1.0) * l_C * l_M          # 2 l_M l_C d' + l_M l_C
    assert bench.score_flops(cfg, 2048 + 128 + 100, l_C) == 0.0                      # k covers all of M: no scoring
    c3 = syn.get_config("c3")
    t3 = c3.S
    assert bench.decode_bytes(c3, t3) == 2.0 * (t3 - 2048 - 128) * 128 + 4.0 * (128 + 4096 + 2048 + 1) * c3.d_G


def test_clock_sample_parser():
    s = bench.ClockSampler(0)
    s.proc = type("P", (), {"terminate": lambda self: None, "wait": lambda self, timeout=None: 0, "kill": lambda self: None})()
    s.lines = ["0, 1350, 1965, 950.1, 0x4, Not Active, Not Active, Not Active, Active",
               "0, 1410, 1965, 990.0, 0x4, Not Active, Not Active, Not Active, Active",
               "0, 1380, 1965, 970.0, 0x0, Not Active, Not Active, Not Active, Not Active", "garbage"]
    out = s.stop()
    assert out["sm_mhz"] == 1380.0 and out["sm_max_mhz"] == 1965.0 and out["reasons"] == ["sw_power_cap"]
