"""Host-side logic of bench.py: the variant table, the aggregation, and the multi-replica path
(max over ranks) exercised with two gloo processes on the CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_variant_table_shape_and_bytes():
    specs = bench.variant_specs()
    assert len(specs) == 120
    fam = {}
    for sp in specs:
        fam[sp["family"]] = fam.get(sp["family"], 0) + 1
        assert sp["touched"] >= sp["useful"] > 0
        # every variant is sized to a working set of about 256 MiB of touched memory
        per_pass = sp["touched"] / {"axpy": 1.5, "swap": 2, "rot": 2, "ger": 2, "scal": 2}.get(sp["routine"], 1)
        assert 0.9 * 256 * bench.MIB <= per_pass <= 1.1 * 256 * bench.MIB, sp["name"]
    assert fam == {"l1_map": 20, "l1_reduce": 16, "l2_tile": 48, "ger": 4, "trsv": 32}
    small = bench.variant_specs(16)
    assert len(small) == 120 and small[0]["n"] * 16 == specs[0]["n"]


def test_aggregate_and_geomean():
    specs = bench.variant_specs()[:3]
    rows, value = bench.aggregate(specs, [1.0, 2.0, 4.0], world=2, peak=1000.0)
    rates = [sp["touched"] / (t * 1e-3) / 1e9 for sp, t in zip(specs, [1.0, 2.0, 4.0])]
    assert rows[1]["gbs"] == pytest.approx(rates[1]) and rows[1]["frac"] == pytest.approx(rates[1] / 1000.0)
    assert value == pytest.approx(2 * (rates[0] * rates[1] * rates[2]) ** (1 / 3))
    assert bench.max_over_ranks([3.0, 1.0]) == [3.0, 1.0]  # no process group: identity


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 5.0 - rank, 2.0]
    got = bench.max_over_ranks(mine)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, got))


def test_max_over_ranks_two_gloo_processes():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [2.0, 5.0, 2.0]
