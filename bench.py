"""Benchmark of the partial-token GRPO policy-gradient step (NAT) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over one synthetic batch: advantages,
selection, compaction, policy-loss forward and backward (by default through the
single-pass call nat_policy_loss_fwd_bwd; --route two times the separate calls).  Rank 0 prints ONE
JSON line.  `value` is selected tokens per second with inputs resident in HBM;
`e2e` is the same with the step's inputs copied from pinned host memory and the
loss read back inside the timed region.  `--impl reference` times the fp64 CPU
oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "selected tokens/sec, fused policy-loss fwd+bwd (Qwen3-8B head); % bf16 TC peak"
UNIT = "selected tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count()


# ---------------------------------------------------------------- CPU oracle
def oracle_sample_rate(w, seed, rows, repeats=1):
    """Selected tokens/s of the fp64 oracle (loss forward + backward) on `rows`
    selected tokens of the workload's head (same d, V, dtype and value recipe)."""
    import numpy as np
    import oracle
    from paper_2603_06619_b200 import workloads as wl

    # a short batch with the workload's head: enough tokens that `rows` are selected
    T = np.full(w.B, max(4, (2 * rows + w.B - 1) // w.B), dtype=np.int32)
    batch = wl.to_numpy(wl.make_batch(w, seed=seed, lengths=T))
    adv = oracle.grpo_adv(batch["rewards"], w.P, w.G, 1e-6)
    mask, pi, _ = oracle.select(oracle.SEL_URS, batch["cu_seqlens"], p=1.0)
    si, sr, _, _ = oracle.compact(mask, batch["cu_seqlens"])
    si, sr = si[:rows], sr[:rows]
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.policy_loss_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"],
                               adv, pi, batch["cu_seqlens"], si, sr)
        times.append(time.perf_counter() - t0)
    return len(si) / min(times), min(times), len(si), times


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = args.ref_rows
    for _ in range(args.warmup):
        pass  # the oracle has no warm state worth building; keep the run short
    rate, _, n, times = oracle_sample_rate(w, seed=0, rows=rows, repeats=max(1, args.steps))
    ms = 1e3 * statistics.mean(times)
    cores = host_cores()
    sample = f"{n} selected rows of the {w.name} head per step (fp64 loss fwd+bwd, all of V)"
    line = {
        "impl": "reference", "metric": METRIC, "value": n / (ms / 1e3), "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "d": w.d, "V": w.V, "sample": sample},
        "cpu_baseline": {"value": n / (ms / 1e3), "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": n / (ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------- ours
def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2603_06619_b200 import build as _build
    from paper_2603_06619_b200 import sharding
    from paper_2603_06619_b200 import workloads as wl
    from paper_2603_06619_b200.step import NatStep

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()

    # Responses are independent, so ranks take disjoint batches (weak scaling):
    # no collective sits on the data path.
    seed = sharding.rank_seed(args.seed, rank)
    batch = wl.make_batch(w, seed=seed, device=dev)
    n_tot = batch["n_tot"]
    dtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    st = NatStep(w.P, w.G, w.d, w.V, dtype, n_tot, device=dev)
    cu = batch["cu_seqlens"]
    sel = dict(mode=w.sel_mode, p=w.p, min_cut=w.min_cut, beta=w.beta, seed=seed)

    def exchange():
        if args.allreduce_dw and world > 1:
            sharding.allreduce_grads(st.loss, st.dW)

    def step(b, offset):
        st.grpo_adv(b["rewards"])
        st.select(cu, offset=offset, **sel)
        st.compact(cu)
        st.loss_fwd_bwd(b["hidden"], b["W"], b["targets"], b["old_logp"], cu)
        exchange()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def step_two_pass(b, offset):
        st.grpo_adv(b["rewards"])
        st.select(cu, offset=offset, **sel)
        st.compact(cu)
        st.loss_fwd(b["hidden"], b["W"], b["targets"], b["old_logp"], cu)
        st.loss_bwd(b["hidden"], b["W"], b["targets"], b["old_logp"], cu)
        exchange()

    main_step = step if args.route == "single" else step_two_pass
    for i in range(args.warmup):
        main_step(batch, i)
    sync_all()
    if st.status() & ~4:
        raise RuntimeError(f"device status {st.status()} after warm-up")

    # ---- device-resident timing of the whole step; the loss call bracketed by events
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sync_all()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(args.steps):
        off = args.warmup + i
        st.grpo_adv(batch["rewards"])
        st.select(cu, offset=off, **sel)
        st.compact(cu)
        ev[i][0].record()
        if args.route == "single":
            st.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
            ev[i][1].record()
        else:
            st.loss_fwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
            ev[i][1].record()
            st.loss_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
        ev[i][2].record()
        exchange()
    t_end.record()
    sync_all()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = t_begin.elapsed_time(t_end)
    loss_call_ms = statistics.mean(e[0].elapsed_time(e[2]) for e in ev)
    first_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    status = st.status()
    loss_val = float(st.loss.item())
    # selected tokens per step: selection with offsets warmup..warmup+K-1 (replayed, untimed)
    n_sel_total = 0
    for i in range(args.steps):
        st.select(cu, offset=args.warmup + i, **sel)
        st.compact(cu)
        n_sel_total += int(st.n_sel.item())

    # ---- per-kernel durations: the same K steps again with event pairs around every
    # tensor-core launch (kept out of the timed region above)
    from paper_2603_06619_b200 import nat as _nat
    trace = None
    if w.dtype == "bf16":
        _nat.nat_trace_begin()
        for i in range(args.steps):
            main_step(batch, args.warmup + i)
        trace = _nat.nat_trace_end()
        sync_all()

    # ---- the other route, for the record (same batch, same offsets, 1 warm-up)
    other = step_two_pass if args.route == "single" else step
    other_ms = float("nan")
    if not args.skip_other_route:
        other(batch, 0)
        sync_all()
        o_begin = torch.cuda.Event(enable_timing=True)
        o_end = torch.cuda.Event(enable_timing=True)
        o_begin.record()
        for i in range(args.steps):
            other(batch, args.warmup + i)
        o_end.record()
        sync_all()
        other_ms = o_begin.elapsed_time(o_end)

    # ---- end to end: every step's inputs come from pinned host memory and its loss goes
    # back to the host.  As a trainer's input pipeline would, the copy of step i+1's inputs
    # runs on a second stream into the other of two device buffer sets while step i computes;
    # the first step's copy has nothing to hide behind.  All copies are inside the timed region.
    host = {k: batch[k].cpu().pin_memory() for k in ("hidden", "targets", "old_logp", "rewards")}
    dev_in = [{k: torch.empty_like(batch[k]) for k in host} for _ in range(2)]
    loss_host = torch.zeros(1, dtype=torch.float32).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    main_stream = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream()
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def issue_copy(slot):
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[slot])   # the step that last read this set is done
            for k in host:
                dev_in[slot][k].copy_(host[k], non_blocking=True)
            copied[slot].record(copy_stream)

    def e2e_steps(n, first_offset):
        start = torch.cuda.Event(enable_timing=True)
        start.record()
        copy_stream.wait_event(start)                # no copy starts before the clock does
        issue_copy(0)
        for i in range(n):
            slot = i % 2
            if i + 1 < n:
                issue_copy(1 - slot)
            main_stream.wait_event(copied[slot])
            main_step(dict(dev_in[slot], W=batch["W"]), first_offset + i)
            consumed[slot].record(main_stream)
            loss_host.copy_(st.loss, non_blocking=True)
        end = torch.cuda.Event(enable_timing=True)
        end.record()
        return start, end

    e2e_steps(1, 0)
    sync_all()
    e_begin, e_end = e2e_steps(args.steps, args.warmup)
    sync_all()
    e2e_ms = e_begin.elapsed_time(e_end)

    # ---- max over ranks, totals over ranks
    (elapsed_ms, e2e_ms, loss_call_ms, first_ms, other_ms), n_all = sharding.aggregate_timing(
        [elapsed_ms, e2e_ms, loss_call_ms, first_ms, other_ms], n_sel_total, device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    n_step = n_sel_total / args.steps              # this rank's selected tokens per step
    dV = float(w.d) * float(w.V)
    # The step runs for most of a second under the power cap, so the sustained tensor
    # peak is the roofline's denominator; the burst figure is reported beside it.
    peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    step_ms = elapsed_ms / args.steps
    counted = 6.0 * n_step * dV
    executed = counted if args.route == "single" else 8.0 * n_step * dV
    call_tflops = counted / (loss_call_ms * 1e-3) / 1e12
    step_tflops = counted / (step_ms * 1e-3) / 1e12
    cap_pad = (n_tot + 255) // 256 * 256
    n_chunks = (cap_pad + min(cap_pad, 8192) - 1) // min(cap_pad, 8192)
    sel_launches = 1 + (1 if w.sel_mode == "urs" else 2) + 3
    if w.dtype == "f32":
        launches = sel_launches + 2 + 3
    elif args.route == "single":
        launches = sel_launches + 2 + 9 * n_chunks + 3      # gather, references; per chunk 9; tail 3
    else:
        launches = sel_launches + 4 + (3 + 3 * n_chunks)
    kernel = ("nat_tc_kernel<kE|kDh|kDw> (the launches inside nat_policy_loss_fwd_bwd)"
              if args.route == "single" else
              "nat_tc_kernel<kFwd|kDz|kDh|kDw> (nat_policy_loss_fwd + nat_policy_loss_bwd)")
    roof_ms, roof_flops, per_kernel, traffic = loss_call_ms, counted, None, None
    if trace:
        # counted FLOPs of one step per kernel kind: the forward's 2NdV belongs to kFwd or kE,
        # dH and dW have 2NdV each, the recompute (kDz) and the one-tile reference pass have none
        unit = 2.0 * n_step * dV
        credit = {"e": unit, "dh": unit, "dw": unit, "dz": 0.0,
                  "fwd": unit if args.route == "two" else 0.0}
        active = -(-int(n_step) // 8192)
        per_kernel = {}
        for kind, (ms, n_launch) in trace.items():
            if n_launch == 0:
                continue
            ms_step = ms / args.steps
            per_kernel[kind] = {
                "ms_per_step": ms_step, "launches_per_step": n_launch / args.steps,
                "ms_per_active_launch": ms_step / active if kind != "fwd" or args.route == "two"
                else None,
                "tflops_counted": credit[kind] / (ms_step * 1e-3) / 1e12 if ms_step > 0 else None}
        top = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_step"])
        kernel = "nat_tc_kernel<%s>" % {"e": "kE", "dh": "kDh", "dw": "kDw", "dz": "kDz",
                                         "fwd": "kFwd"}[top]
        roof_ms, roof_flops = per_kernel[top]["ms_per_step"], credit[top]
        # DRAM bytes per launch (one 8192-row chunk of this head) from the ncu capture
        # summarised in profiles/nat_tc_kernel_qwen3_8b_chunk.md; null for other shapes
        if w.name == "qwen3_8b":
            traffic = {"e": 9.51e9, "dh": 16.79e9, "dw": 21.37e9}.get(top)
    call_tflops = roof_flops / (roof_ms * 1e-3) / 1e12

    line = {
        "metric": METRIC, "value": n_all / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": w.name, "P": w.P, "G": w.G, "d": w.d, "V": w.V,
                   "selection": w.sel_mode, "p": w.p, "min_cut": w.min_cut,
                   "route": ("single pass (nat_policy_loss_fwd_bwd)" if args.route == "single"
                             else "two pass (nat_policy_loss_fwd, nat_policy_loss_bwd)"),
                   "n_tot_per_gpu": n_tot, "n_sel_per_step_per_gpu": n_step,
                   "l2": "inputs larger than L2 (hidden and W_lm are GBs); no flush needed",
                   "parallelism": (f"dp{world} (independent batches, loss and dW all-reduced "
                                   "every step)" if args.allreduce_dw and world > 1 else
                                   f"dp{world} (independent batches, no collective)")},
        "tflops_counted": step_tflops,
        "tflops_executed": executed / (step_ms * 1e-3) / 1e12,
        "frac_of_peak_counted": {
            "burst": step_tflops / float(peaks["bf16_tflops"]),
            "sustained": step_tflops / peak,
            "datasheet_2250": step_tflops / 2250.0},
        "loss_call_ms": loss_call_ms, "loss": loss_val, "device_status": status,
        "other_route": None if args.skip_other_route else {
            "route": "two pass" if args.route == "single" else "single pass",
            "ms_per_step": other_ms / args.steps,
            "tflops_counted": counted / (other_ms / args.steps * 1e-3) / 1e12},
        "roofline": {
            "kernel": kernel, "bound": "tensor", "achieved": call_tflops, "peak": peak,
            "unit": "TFLOP/s", "frac": call_tflops / peak,
            "peak_source": f"{peak_kind} bf16_tflops_sustained (of measured)"
            if peak_kind == "measured" else "fallback (of fallback)",
            "flops": ("counted 2*N_sel*d*V per step for this kernel, divided by its event-timed "
                      "duration summed over the step's launches (nat_trace_begin/end)") if trace
            else "counted 6*N_sel*d*V per step divided by the event-timed loss call(s)",
            "traffic": traffic, "traffic_unit": "DRAM bytes per launch (8192-row chunk)"},
        "per_kernel": per_kernel,
        "e2e": {"value": n_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": 4, "ms_per_step": e2e_ms / args.steps,
                "pipeline": "step i+1's inputs are copied on a second stream (two device buffer "
                            "sets) while step i computes; all copies inside the timed region"},
        "gpu_launches": launches * args.steps,
        "clocks": clocks,
    }
    if args.route == "two":
        line["fwd_ms"], line["bwd_ms"] = first_ms, loss_call_ms - first_ms
    if not args.no_cpu_baseline and world == 1:
        rate, secs, n, _ = oracle_sample_rate(w, seed=0, rows=args.ref_rows)
        line["cpu_baseline"] = {
            "value": rate, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": f"{n} selected rows of the {w.name} head (fp64 loss fwd+bwd over all of V) "
                      f"in {secs:.1f} s"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3_8b")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--ref-rows", type=int, default=384,
                    help="selected rows the fp64 oracle evaluates per timed sample (about 15 s on 16 cores)")
    ap.add_argument("--allreduce-dw", action="store_true",
                    help="N > 1: sum loss and dW over the ranks inside every step (the exchange of "
                         "a data-parallel trainer); off by default: ranks then run independent "
                         "batches with no collective")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-other-route", action="store_true",
                    help="do not also time the route that was not selected")
    ap.add_argument("--route", default="single", choices=["single", "two"],
                    help="single: nat_policy_loss_fwd_bwd; two: forward then backward calls")
    args = ap.parse_args()
    from paper_2603_06619_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
