"""Host-side logic of bench.py that needs no GPU: the rank launcher, the workload overrides,
the tie between tracked ncu counters and the kernel sources, and the sharded batches."""
import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2603_06619_b200 import sharding  # noqa: E402
from paper_2603_06619_b200 import workloads as wl  # noqa: E402


def test_launcher_starts_one_process_per_gpu_on_the_loopback_address():
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "2"], 29511)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
    assert 1024 < bench.free_port() < 65536


def test_workload_overrides():
    ns = argparse.Namespace(workload="long_cot", prompts=0, selection="urs:1.0")
    w = bench.pick_workload(ns)
    assert (w.sel_mode, w.p, w.P) == ("urs", 1.0, 4)
    ns = argparse.Namespace(workload="qwen3_8b", prompts=1, selection="det:0.5")
    w = bench.pick_workload(ns)
    assert (w.sel_mode, w.beta, w.P, w.d) == ("det", 0.5, 1, 4096)
    assert "C=100" in bench.selection_label(wl.WORKLOADS["qwen3_8b"])


def test_tracked_traffic_is_tied_to_the_kernel_sources(tmp_path, monkeypatch):
    h = bench.kernel_source_hash()
    assert len(h) == 16 and h == bench.kernel_source_hash()
    f = tmp_path / "traffic.json"
    entry = {"kernel": "e", "d": 4096, "V": 151936, "chunk_rows": 8192,
             "dram_bytes_per_launch": 9.5e9, "summary": "x.md"}
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    assert bench.dram_traffic("e", 4096, 151936, 8192)[0] is None           # no file
    f.write_text(json.dumps({"source_hash": h, "captures": [entry]}))
    assert bench.dram_traffic("e", 4096, 151936, 8192) == (9.5e9, "x.md")
    assert bench.dram_traffic("dw", 4096, 151936, 8192)[0] is None          # kernel not covered
    assert bench.dram_traffic("e", 1024, 151936, 8192)[0] is None           # shape not covered
    f.write_text(json.dumps({"source_hash": "0" * 16, "captures": [entry]}))
    got, why = bench.dram_traffic("e", 4096, 151936, 8192)
    assert got is None and "changed" in why                                  # stale counters


def test_sharded_batches_partition_the_global_batch_and_share_W():
    w = wl.variant(wl.WORKLOADS["tiny"], P=3)
    T_all = wl.make_lengths(w, 0)
    world, shards = 2, []
    for rank in range(world):
        lo, hi = sharding.response_range(w.P, w.G, rank, world)
        wloc = wl.variant(w, P=(hi - lo) // w.G)
        b = wl.make_batch(wloc, seed=1000 * (rank + 1), lengths=T_all[lo:hi], W_seed=0)
        assert b["n_tot"] == int(T_all[lo:hi].sum()) and b["rewards"].numel() == hi - lo
        shards.append(b)
    assert torch.equal(shards[0]["W"], shards[1]["W"])                      # replicated head
    assert not torch.equal(shards[0]["hidden"][:8], shards[1]["hidden"][:8])
    assert sum(b["n_tot"] for b in shards) == int(T_all.sum())


def test_a_bad_clock_record_is_measured_again():
    ok = {"sm_mhz": 1300.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"], "samples": 40}
    assert not bench.clocks_rejected(ok)                                     # power cap: kept
    assert bench.clocks_rejected(dict(ok, reasons=["hw_thermal_slowdown", "sw_power_cap"]))
    assert bench.clocks_rejected(dict(ok, reasons=["sw_thermal_slowdown"]))
    assert bench.clocks_rejected(dict(ok, reasons=["hw_slowdown"]))
    assert bench.clocks_rejected(dict(ok, sm_mhz=900.0, reasons=[]))         # a leftover lock
    assert not bench.clocks_rejected(dict(ok, sm_mhz=1900.0, reasons=[]))
    assert not bench.clocks_rejected(dict(ok, sm_mhz=900.0, reasons=[], samples=1))  # too short
    assert not bench.clocks_rejected(None)
    assert not bench.clocks_rejected({"sm_mhz": None, "reasons": ["nvidia-smi unavailable"]})
