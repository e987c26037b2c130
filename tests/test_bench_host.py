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


def test_final_line_is_short_and_keeps_the_summary_keys():
    """The last stdout line must survive a reader that keeps only the end of the output: summary
    keys only, no per-variant rows, well under 4 KB even with all 120 variants aggregated."""
    import json
    specs = bench.variant_specs()
    rows, value = bench.aggregate(specs, [0.05 + 0.001 * k for k in range(len(specs))], world=1, peak=6547.2)
    fams = sorted({sp["family"] for sp in specs})
    by_kernel = {k: {"achieved": 5269.388006569296, "frac": 0.8048307683543034, "share_of_time": 0.2382904333518465,
                     "variants": 48} for k in fams}
    out = {
        "metric": "achieved HBM GB/s per BLAS-1/2 variant, geomean over variants", "value": value, "unit": "GB/s",
        "n_gpus": 1, "steps": 20, "warmup": 3, "ms_per_step": 16.193397521972656, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32+f64", "data": "synthetic",
        "config": {"workload": "w" * 120, "variants": 120, "l2": "x" * 220, "bytes": "touched sectors (span bytes)",
                   "parallelism": "single GPU"},
        "geomean_frac_of_peak": 0.6152370341687622, "geomean_frac_of_peak_without_trsv": 0.8522784166663647,
        "geomean_frac_by_family": {k: 0.9382842251889021 for k in fams}, "min_variant": "trsv_unn_f64_inc1",
        "gpu_launches": 7040, "clocks": {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": [], "samples": 2},
        "roofline": {"bound": "hbm", "kernel": "trsv", "achieved": 1640.9586225995336, "peak": 6547.2, "unit": "GB/s",
                     "frac": 0.2506351757391761, "traffic": 274000000.0,
                     "peak_source": "measured (MEASURED_PEAKS.json hbm_gbs)", "by_kernel": by_kernel},
        "e2e": {"value": 36.17699841312217, "unit": "GB/s (geomean over variants, host buffers in and out)",
                "h2d_bytes_per_step": 50775709228, "d2h_bytes_per_step": 5369180156, "steps": 2},
        "cpu_baseline": {"value": 1.313513313524947, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": "s" * 100},
        "variants": rows, "next_rows": {"variants": rows},
    }
    line = bench.final_line(out)
    assert "\n" not in line and len(line) < 4096
    back = json.loads(line)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "roofline", "cpu_baseline",
                "e2e", "clocks", "gpu_launches", "config"):
        assert key in back, key
    assert "variants" not in back and "next_rows" not in back
    assert back["value"] == pytest.approx(value, rel=1e-4)
    assert back["e2e"]["h2d_bytes_per_step"] == 50775709228  # integers are kept whole
    assert set(back["roofline"]["by_kernel"]) == set(fams)


def test_clock_summary_windows():
    """Samples inside the timed region are used when there are at least three; a shorter region
    falls back to everything from the warm-up on, and slowdown reasons are collected."""
    mk = lambda t, mhz, flags="Not Active, Not Active, Not Active, Not Active": (t, f"{mhz}, 1965, {flags}")
    lines = [mk(0.0, 300), mk(1.0, 1900), mk(1.1, 1950), mk(2.0, 1965), mk(2.05, 1965), mk(2.1, 1960),
             mk(2.15, 1965, "Not Active, Not Active, Not Active, Active")]
    out = bench.ClockSampler.summarise(lines, t_load=0.9, t0=1.95, t1=2.2)
    assert out["samples"] == 4 and out["sm_mhz"] == 1965 and out["sm_max_mhz"] == 1965
    assert out["reasons"] == ["sw_power_cap"] and out["window"] == "timed region"
    out = bench.ClockSampler.summarise(lines, t_load=0.9, t0=2.12, t1=2.2)  # one sample inside: widen
    assert out["samples"] == 6 and out["window"].startswith("warm-up") and out["sm_mhz"] == 1965
    assert bench.ClockSampler.summarise([], None, None, None)["sm_mhz"] is None
