"""Benchmark of the partial-token GRPO policy-gradient step (NAT) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over one synthetic batch: advantages,
selection, compaction, policy-loss forward and backward (by default through the
single-pass call nat_policy_loss_fwd_bwd; --route two times the separate calls).  Rank 0
prints ONE JSON line.  `value` is selected tokens per second with inputs resident in HBM;
`e2e` is the same with the step's inputs copied from pinned host memory and the
loss read back inside the timed region.  `--impl reference` times the fp64 CPU
oracle on a bounded sample of the same workload.

With --gpus N > 1 and no torchrun environment the script starts the N ranks itself (one
process per GPU).  By default the ranks run independent batches (weak scaling, no
collective on the data path); --sharded makes them split ONE batch by prompt groups and
sum loss and dW with an all-reduce every step (the exchange of a data-parallel trainer).

Other measurements (markdown tables on stdout instead of the JSON line):
    --mode sweep     time against the selected-token fraction (URS p, RPC, truncation)
    --mode stress    selection / compaction / packing GB/s on a 2^28-token stream
    --mode ceiling   the loss kernels against the library's plain GEMMs on the same operands
    --mode source-hash   hash of the tensor-core kernel sources (ties ncu counters to a build)
"""
import argparse
import glob
import hashlib
import json
import os
import re
import socket
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
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "nat_tc_kernel_dram_traffic.json")
KERNEL_SOURCES = ("nat_loss_bf16.cu", "nat_tc.cuh")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def kernel_source_hash():
    """sha256 over the code of the tensor-core loss kernels (comments and blank lines
    left out): the ncu counters kept under profiles/ carry the hash of the code they
    were taken from."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2603_06619_b200", "csrc", name)) as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for line in text.splitlines():
            line = re.sub(r"//.*", "", line).strip()
            if line:
                h.update(line.encode() + b"\n")
    return h.hexdigest()[:16]


def dram_traffic(kind, d, V, chunk_rows):
    """DRAM bytes per launch of one loss kernel from the tracked ncu capture, or (None, why)
    when no capture covers this shape or the kernels changed after it was taken."""
    if not os.path.exists(TRAFFIC_FILE):
        return None, "no capture on file"
    with open(TRAFFIC_FILE) as f:
        t = json.load(f)
    if t.get("source_hash") != kernel_source_hash():
        return None, "kernel sources changed since the counters were taken"
    for c in t.get("captures", []):
        if (c["kernel"], c["d"], c["V"], c["chunk_rows"]) == (kind, d, V, chunk_rows):
            return c["dram_bytes_per_launch"], c.get("summary", "")
    return None, "shape not covered by the capture"


def dh_k_parts(chunk_rows, d, V, slots=74):
    """K parts the library uses for the dHidden contraction of one row chunk on a whole B200
    (74 CTA pairs): the smallest count up to 8 that fills the pairs' rounds to 95 %.  Only
    used to count this script's own kernel launches."""
    tiles = (chunk_rows // 512) * ((d + 255) // 256)
    kb = (V + 63) // 64
    best, best_eff = 1, 0.0
    for parts in range(1, 9):
        if parts > 1 and kb // parts < 64:
            break
        units = tiles * parts
        eff = units / (-(-units // slots) * slots) if units else 0.0
        if eff > best_eff + 1e-9:
            best, best_eff = parts, eff
        if eff >= 0.95:
            return parts
    return best


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
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def board_gemm_rate(seconds=3.0, n=8192):
    """Sustained bf16 rate of the library's plain GEMM (torch.matmul, n^3) on THIS board, now:
    looped for `seconds` under the power cap, second half timed.  The boards of a pool settle
    at different clocks under the same cap, so this puts a same-board figure beside the
    pool-wide measured peak.  The library is called for this denominator only."""
    import torch
    a = torch.randn(n, n, device="cuda").to(torch.bfloat16)
    b = torch.randn(n, n, device="cuda").to(torch.bfloat16)
    c = torch.empty(n, n, device="cuda", dtype=torch.bfloat16)
    ms = _time(lambda: torch.matmul(a, b, out=c), 4, warmup=2)
    reps = max(8, int(seconds * 1e3 / ms))
    for _ in range(reps // 2):
        torch.matmul(a, b, out=c)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    ms = _time(lambda: torch.matmul(a, b, out=c), reps - reps // 2, warmup=0)
    clk = sampler.stop()
    return {"tflops": 2.0 * n ** 3 / (ms * 1e-3) / 1e12, "sm_mhz": clk.get("sm_mhz"),
            "power_w": clk.get("power_w"),
            "how": f"torch.matmul {n}^3 bf16 looped for about {seconds:.0f} s after the timed "
                   "region, second half timed"}


def clocks_rejected(c):
    """True for a clock record that invalidates a timing: a hardware or thermal slowdown seen,
    or SM clocks well below the maximum with no throttle reason active."""
    if not c or c.get("sm_mhz") is None or c.get("samples", 0) < 3:
        return False
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(c["reasons"])
    stuck = not c["reasons"] and c.get("sm_max_mhz") and c["sm_mhz"] < 0.75 * c["sm_max_mhz"]
    return bool(bad) or bool(stuck)


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count()


def pick_workload(args):
    """The named workload with the command line's overrides (selection, prompt count)."""
    from paper_2603_06619_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    if args.prompts:
        w = wl.variant(w, P=args.prompts)
    if args.selection:
        mode, _, val = args.selection.partition(":")
        if mode == "urs":
            w = wl.variant(w, sel_mode="urs", p=float(val or 0.5))
        elif mode == "rpc":
            w = wl.variant(w, sel_mode="rpc", min_cut=int(val or 100))
        elif mode == "det":
            w = wl.variant(w, sel_mode="det", beta=float(val or 0.5))
        else:
            raise SystemExit("--selection takes urs:P, rpc:C or det:BETA")
    return w


def selection_label(w):
    return {"urs": f"URS p={w.p:g}", "rpc": f"RPC C={w.min_cut}",
            "det": f"deterministic truncation beta={w.beta:g}"}[w.sel_mode]


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
    # W warm-up passes and K timed ones over the same bounded sample (its size is kept: the
    # oracle's per-call setup, widening W_lm to fp64, would weigh more on a smaller one);
    # about 8 s per pass on 16 cores at the default sample, so K = 20 ends within a few minutes
    passes = max(1, args.steps) + max(0, args.warmup)
    rows = args.ref_rows
    rate, _, n, times = oracle_sample_rate(w, seed=0, rows=rows, repeats=passes)
    times = times[max(0, args.warmup):]
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


# ------------------------------------------------------------------ launcher
def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launcher_command(n, argv, port):
    """The command that starts `n` ranks of this script on one node (one process per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node",
            str(n), "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.abspath(__file__)] + list(argv)


def launch_ranks(args, argv):
    """--gpus N given to a plain `python bench.py`: start the N ranks and pass rank 0's JSON
    line through.  NCCL's communicator log goes to a file per rank so that stdout stays one
    line; rank 0 reads the rank count back from it into the line."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", f"/tmp/nat_bench_nccl_{os.getpid()}.%h.%p.log")
    cmd = launcher_command(args.gpus, argv, free_port())
    return subprocess.call(cmd, env=env)


def nccl_log_summary():
    """Rank count and NVLS use as NCCL's own log states them (None when no log was kept)."""
    pattern = os.environ.get("NCCL_DEBUG_FILE")
    if not pattern:
        return None
    path = pattern.replace("%h", socket.gethostname()).replace("%p", str(os.getpid()))
    files = [path] if os.path.exists(path) else glob.glob(re.sub(r"%[hp]", "*", pattern))
    nranks, nvls = None, False
    for fpath in files[:8]:
        try:
            text = open(fpath, errors="replace").read()
        except OSError:
            continue
        m = re.findall(r"nranks (\d+)", text)
        if m:
            nranks = max(int(x) for x in m)
        nvls = nvls or ("NVLS" in text and "NVLS multicast support is available" in text)
    return {"nranks": nranks, "nvls": nvls, "log": pattern}


# --------------------------------------------------------------------- ours
def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2603_06619_b200 import build as _build
    from paper_2603_06619_b200 import nat as _nat
    from paper_2603_06619_b200 import sharding
    from paper_2603_06619_b200 import workloads as wl
    from paper_2603_06619_b200.step import NatStep

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if local_rank >= torch.cuda.device_count():
        raise SystemExit(f"rank {rank}: no GPU {local_rank} (this node shows "
                         f"{torch.cuda.device_count()}); --gpus must not exceed the GPUs present")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()

    sharded = args.sharded          # with one rank: the same path, the exchange a no-op
    exchange_on = sharded or (args.allreduce_dw and world > 1)
    if sharded:
        # ONE batch, split by prompt groups: this rank holds responses [lo, hi) of it, keeps
        # the batch's size as the divisor of the batch mean and draws its masks with the
        # global response indices; W is the same on every rank.
        seed = args.seed
        T_all = wl.make_lengths(w, seed)
        lo, hi = sharding.response_range(w.P, w.G, rank, world)
        if hi == lo:
            raise SystemExit(f"--sharded needs at least one prompt per rank (P = {w.P}, {world} ranks)")
        w_local = wl.variant(w, P=(hi - lo) // w.G)
        batch = wl.make_batch(w_local, seed=seed + 1000 * (rank + 1), device=dev,
                              lengths=T_all[lo:hi], W_seed=seed)
        step_kw = dict(B_global=w.B, resp_base=lo)
    else:
        # Responses are independent, so ranks take disjoint batches (weak scaling):
        # no collective sits on the data path.
        seed = sharding.rank_seed(args.seed, rank)
        w_local = w
        batch = wl.make_batch(w, seed=seed, device=dev)
        step_kw = {}
    n_tot = batch["n_tot"]
    dtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    st = NatStep(w_local.P, w_local.G, w.d, w.V, dtype, n_tot, device=dev, **step_kw)
    cu = batch["cu_seqlens"]
    sel = dict(mode=w.sel_mode, p=w.p, min_cut=w.min_cut, beta=w.beta, seed=args.seed if sharded else seed)

    def exchange():
        if exchange_on:
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
    def timed_region():
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
        return elapsed_ms, ev, clocks

    # A clock record with a thermal or hardware slowdown, or clocks far below the maximum with
    # no reason active (a leftover clock lock), does not count: the region is measured once more.
    elapsed_ms, ev, clocks = timed_region()
    redo = torch.tensor([1 if rank == 0 and clocks_rejected(clocks) else 0], device=dev)
    if world > 1:
        dist.broadcast(redo, src=0)
    rejected_clocks = None
    if int(redo.item()):
        rejected_clocks = clocks
        elapsed_ms, ev, clocks = timed_region()
        if rank == 0:
            clocks["rejected_first_attempt"] = rejected_clocks
    loss_call_ms = statistics.mean(e[0].elapsed_time(e[2]) for e in ev)
    first_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    prep_ms = (elapsed_ms - sum(e[0].elapsed_time(e[2]) for e in ev)) / args.steps
    status = st.status()
    loss_val = float(st.loss.item())
    if args.only_steps:
        if rank == 0:
            print(json.dumps({"only_steps": True, "workload": w.name, "steps": args.steps,
                              "ms_per_step": elapsed_ms / args.steps, "device_status": status}))
        if world > 1:
            dist.destroy_process_group()
        return
    # selected tokens per step: selection with offsets warmup..warmup+K-1 (replayed, untimed)
    n_sel_total = 0
    for i in range(args.steps):
        st.select(cu, offset=args.warmup + i, **sel)
        st.compact(cu)
        n_sel_total += int(st.n_sel.item())

    # ---- per-kernel durations: the same K steps again with event pairs around every
    # tensor-core launch (kept out of the timed region above)
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
    cap_pad = (n_tot + 511) // 512 * 512
    chunk_rows = min(cap_pad, 8192)
    n_chunks = (cap_pad + chunk_rows - 1) // chunk_rows
    sel_launches = 1 + (1 if w.sel_mode == "urs" else 2) + (3 if w.sel_mode == "urs" else 2)
    k_parts = dh_k_parts(chunk_rows, w.d, w.V)
    if w.dtype == "f32":
        launches = sel_launches + 2 + 3
    elif args.route == "single":
        # gather, row references; per chunk kE, finalize, kDh (+ its finalize when the K range
        # is cut into parts), kDw and the predicated redo (kFwd, finalize, kDz, kDh (+), kDw);
        # tail: fallback note, five kernels of the ordered one-hot pass, loss sum
        launches = sel_launches + 2 + (9 + (2 if k_parts > 1 else 0)) * n_chunks + 7
    else:
        launches = sel_launches + 4 + 2 + (3 + (1 if k_parts > 1 else 0)) * n_chunks + 5
    kernel = ("nat_tc_kernel<kE|kDh|kDw> (the launches inside nat_policy_loss_fwd_bwd)"
              if args.route == "single" else
              "nat_tc_kernel<kFwd|kDz|kDh|kDw> (nat_policy_loss_fwd + nat_policy_loss_bwd)")
    roof_ms, roof_flops, per_kernel, traffic, traffic_note = loss_call_ms, counted, None, None, None
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
        # DRAM bytes per launch (one row chunk of this head) from the tracked ncu capture
        traffic, traffic_note = dram_traffic(top, w.d, w.V, chunk_rows)
    call_tflops = roof_flops / (roof_ms * 1e-3) / 1e12
    sm_mhz = clocks.get("sm_mhz") if clocks else None

    if sharded:
        parallelism = (f"dp{world}: one batch of {w.B} responses split by prompt groups, loss and "
                       "dW all-reduced (NCCL) every step")
    elif exchange_on:
        parallelism = f"dp{world} (independent batches, loss and dW all-reduced every step)"
    else:
        parallelism = f"dp{world} (independent batches, no collective)"
    line = {
        "metric": METRIC, "value": n_all / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
        "higher_is_better": True, "scaling": "strong" if sharded and world > 1 else "weak",
        "vs_baseline": None,
        "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": w.name, "P": w.P, "G": w.G, "d": w.d, "V": w.V,
                   "selection": w.sel_mode, "p": w.p, "min_cut": w.min_cut, "beta": w.beta,
                   "selection_label": selection_label(w),
                   "route": ("single pass (nat_policy_loss_fwd_bwd)" if args.route == "single"
                             else "two pass (nat_policy_loss_fwd, nat_policy_loss_bwd)"),
                   "n_tot_per_gpu": n_tot, "n_sel_per_step_per_gpu": n_step,
                   "l2": "inputs larger than L2 (hidden and W_lm are GBs); no flush needed"
                   if n_tot * w.d * 2 > 2 * 126e6 else
                   "W_lm (hundreds of MB) and the numerator scratch exceed L2; hidden does not",
                   "parallelism": parallelism},
        "tflops_counted": step_tflops,
        "tflops_executed": executed / (step_ms * 1e-3) / 1e12,
        "frac_of_peak_counted": {
            "burst": step_tflops / float(peaks["bf16_tflops"]),
            "sustained": step_tflops / peak,
            "datasheet_2250": step_tflops / 2250.0},
        "loss_call_ms": loss_call_ms, "select_compact_adv_ms": prep_ms, "loss": loss_val,
        "device_status": status,
        "ms_times_sm_mhz": step_ms * sm_mhz if sm_mhz else None,
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
            "traffic": traffic, "traffic_unit": "DRAM bytes per launch (one row chunk)",
            "traffic_source": traffic_note},
        "per_kernel": per_kernel,
        "e2e": {"value": n_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": 4, "ms_per_step": e2e_ms / args.steps,
                "pipeline": "step i+1's inputs are copied on a second stream (two device buffer "
                            "sets) while step i computes; all copies inside the timed region",
                "stays_on_device": "W_lm is resident; of the results only the loss scalar returns "
                                   "to the host: dHidden and dW stay in HBM, where a trainer's "
                                   "backward pass and optimizer consume them"},
        "gpu_launches": launches * args.steps,
        "clocks": clocks,
    }
    if world > 1:
        line["nccl"] = nccl_log_summary()
    if args.route == "two":
        line["fwd_ms"], line["bwd_ms"] = first_ms, loss_call_ms - first_ms
    if not args.no_cpu_baseline and world == 1 and w.dtype == "bf16":
        # the same fraction against what the library's GEMM sustains on this very board
        try:
            lib = board_gemm_rate()
            line["roofline"]["library_gemm_this_board"] = lib
            line["roofline"]["frac_of_this_board"] = call_tflops / lib["tflops"]
        except Exception as e:  # an extra denominator: never at the price of the line itself
            line["roofline"]["library_gemm_this_board"] = {"unavailable": repr(e)[:200]}
    if not args.no_cpu_baseline and world == 1:
        try:
            rate, secs, n, _ = oracle_sample_rate(w, seed=0, rows=args.ref_rows)
            line["cpu_baseline"] = {
                "value": rate, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
                "sample": f"{n} selected rows of the {w.name} head (fp64 loss fwd+bwd over all "
                          f"of V) in {secs:.1f} s"}
        except Exception as e:  # the GPU measurement above stands on its own
            line["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": host_cores(),
                                    "kind": "oracle", "sample": "failed: " + repr(e)[:200]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------- other measurements
def _time(fn, reps, warmup=1):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def fraction_sweep(w, reps=2, seed=0):
    """The single-pass loss on one batch under every selection setting of the sweep (URS
    p = 0.25 .. 1, RPC with the paper's minimum cut of 100, deterministic 50 % truncation)
    and the fit time = a + b * fraction."""
    import numpy as np
    import torch
    from paper_2603_06619_b200 import workloads as wl
    from paper_2603_06619_b200.step import NatStep

    batch = wl.make_batch(w, seed=seed, device="cuda")
    n_tot = batch["n_tot"]
    st = NatStep(w.P, w.G, w.d, w.V, torch.bfloat16, n_tot)
    cu = batch["cu_seqlens"]
    st.grpo_adv(batch["rewards"])
    settings = [("URS p=0.25", dict(mode="urs", p=0.25)), ("URS p=0.5", dict(mode="urs", p=0.5)),
                ("URS p=0.75", dict(mode="urs", p=0.75)),
                ("full tokens (URS p=1)", dict(mode="urs", p=1.0)),
                ("RPC C=100", dict(mode="rpc", min_cut=100)),
                ("Det. trunc. 50%", dict(mode="det", beta=0.5))]
    peaks, kind = load_peaks()
    rows = []
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    for label, kw in settings:
        st.select(cu, seed=seed, **kw)
        st.compact(cu)
        n_sel = int(st.n_sel.item())
        args = (batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
        ms = _time(lambda: st.loss_fwd_bwd(*args), reps)
        assert st.status() & ~4 == 0
        tf = 6.0 * n_sel * w.d * w.V / (ms * 1e-3) / 1e12
        rows.append((label, n_sel, n_sel / n_tot, ms, tf))
    clocks = sampler.stop()
    x = np.array([r[2] for r in rows])
    y = np.array([r[3] for r in rows])
    b, a = np.polyfit(x, y, 1)
    resid = y - (a + b * x)
    out = [f"Workload {w.name}: N_tot = {n_tot}, d = {w.d}, V = {w.V}; single-pass "
           f"nat_policy_loss_fwd_bwd, mean of {reps} calls after 1 warm-up; peaks {kind}; SM clock "
           f"median {clocks['sm_mhz']} MHz, reasons {clocks['reasons']}.", "",
           "| selection | n_sel | fraction | ms | TFLOP/s counted | of burst peak | of sustained peak |",
           "|---|---|---|---|---|---|---|"]
    for label, n_sel, frac, ms, tf in rows:
        out.append(f"| {label} | {n_sel} | {frac:.3f} | {ms:.1f} | {tf:.0f} | "
                   f"{tf / peaks['bf16_tflops']:.3f} | {tf / peaks['bf16_tflops_sustained']:.3f} |")
    out += ["", f"Least-squares fit: time = a + b * fraction with a = {a:.1f} ms, b = {b:.1f} ms "
            f"(a/b = {a / b:.3f}); largest residual {np.abs(resid).max():.1f} ms "
            f"({100 * np.abs(resid / y).max():.1f} % of its point)."]
    return "\n".join(out)


def select_compact_stress(log2_tokens=28, T=8192, reps=5):
    """Selection, compaction and row packing on a stream long enough (2^28 tokens) for HBM
    bandwidth, not launch latency, to be what is measured."""
    import numpy as np
    import torch
    from paper_2603_06619_b200 import nat
    from paper_2603_06619_b200 import workloads as wl
    from paper_2603_06619_b200.step import NatStep

    n_tot = 1 << log2_tokens
    B = n_tot // T
    G = 8
    P = B // G
    cu = torch.arange(0, n_tot + 1, T, dtype=torch.int32, device="cuda")
    st = NatStep(P, G, 64, 512, torch.float32, n_tot, want_grads=False)
    peaks, kind = load_peaks()
    hbm = peaks["hbm_gbs"]
    out = [f"N_tot = 2^{log2_tokens} tokens, B = {B} responses of {T}; mean of {reps} calls; "
           f"HBM peak {hbm:.0f} GB/s ({kind}).", "",
           "| call | selected fraction | ms | algorithmic bytes | GB/s | of HBM peak |",
           "|---|---|---|---|---|---|"]

    def row(label, frac, ms, what, nbytes):
        out.append(f"| {label} | {frac} | {ms:.3f} | {what} | {nbytes / ms / 1e6:.0f} | "
                   f"{nbytes / ms / 1e6 / hbm:.3f} |")

    for label, kw in (("URS p=0.5", dict(mode="urs", p=0.5)), ("RPC C=100", dict(mode="rpc", min_cut=100))):
        ms = _time(lambda: st.select(cu, seed=1, **kw), reps)
        st.compact(cu)
        frac = int(st.n_sel.item()) / n_tot
        row(f"nat_select {label}", f"{frac:.3f}", ms, "5 B/token (mask + pi written)", 5.0 * n_tot)
        msc = _time(lambda: st.compact(cu, from_mask=True), reps)
        row(f"nat_compact after {label}", f"{frac:.3f}", msc,
            "1 B/token read + 8 B per selected token written", (1.0 + 8.0 * frac) * n_tot)
        if kw["mode"] == "rpc":
            msp = _time(lambda: st.compact(cu), reps)
            row(f"nat_compact_prefix after {label}", f"{frac:.3f}", msp,
                "8 B per selected token written (the mask is not read)", 8.0 * frac * n_tot)
    # a cut law given as masses: three reads of q, mask and pi written
    q = torch.rand(n_tot, device="cuda") / T
    ws = nat.alloc_workspace(nat.nat_select_cutlaw_workspace_bytes(B, n_tot), "cuda")
    ms = _time(lambda: nat.nat_select_cutlaw(B, cu, n_tot, q, 1, 0, st.mask, st.pi, st.cut_len, ws),
               reps)
    row("nat_select_cutlaw (random law)", "-", ms,
        "4 B/token read (the law) + 5 B/token written; executed: the law is read twice", 9.0 * n_tot)
    del q
    st.grpo_adv(torch.zeros(B, device="cuda"))
    ms = _time(lambda: st.grpo_adv(torch.zeros(B, device="cuda")), reps)
    out.append(f"| nat_grpo_adv ({P} groups of {G}) | - | {ms:.3f} | launch bound | - | - |")
    del st
    # packing of the selected rows: the Qwen3-8B-shaped batch's hidden states under RPC
    w = wl.WORKLOADS["qwen3_8b"]
    Tl = wl.make_lengths(w, 0)
    cu2 = torch.from_numpy(wl.cu_from_lengths(Tl)).cuda()
    n2 = int(Tl.sum())
    st2 = NatStep(w.P, w.G, 64, 512, torch.float32, n2, want_grads=False)
    st2.select(cu2, "rpc", min_cut=100, seed=0)
    st2.compact(cu2)
    n_sel = int(st2.n_sel.item())
    x = torch.randn(n2, w.d, device="cuda").to(torch.bfloat16)
    packed = torch.empty_like(x)
    full = torch.empty_like(x)
    rowb = w.d * 2
    ms = _time(lambda: nat.nat_gather_rows(x, st2.sel_idx, st2.n_sel, n2, packed), reps)
    row(f"nat_gather_rows ({n_sel} of {n2} rows of {rowb} B)", f"{n_sel / n2:.3f}", ms,
        "row read + row written", 2.0 * n_sel * rowb)
    ms = _time(lambda: nat.nat_scatter_rows(packed, st2.sel_idx, st2.n_sel, n2, n2, full), reps)
    row(f"nat_scatter_rows (same, into {n2} zeroed rows)", f"{n_sel / n2:.3f}", ms,
        "row read + row written + zero fill", 2.0 * n_sel * rowb + 1.0 * n2 * rowb)
    return "\n".join(out)


def ceiling(base, rows=32768, seconds=4.0):
    """Per contraction: TFLOP/s of the loss kernels and of the library GEMM (torch.matmul) on
    the same shapes and operand values, each measured inside a loop that runs for `seconds`
    under the power cap.  The library is called here only, never on the product path."""
    import torch
    from paper_2603_06619_b200 import nat
    from paper_2603_06619_b200 import workloads as wl
    from paper_2603_06619_b200.step import NatStep

    T = rows // base.G
    w = wl.variant(base, P=1, sel_mode="urs", p=1.0, length_law="uniform", len_lo=T, len_hi=T)
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = NatStep(w.P, w.G, w.d, w.V, torch.bfloat16, batch["n_tot"])
    cu = batch["cu_seqlens"]
    st.grpo_adv(batch["rewards"])
    st.select(cu, "urs", p=1.0)
    st.compact(cu)
    n = int(st.n_sel.item())
    args = (batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
    ms_call = _time(lambda: st.loss_fwd_bwd(*args), 2)
    calls = max(2, int(seconds * 1e3 / ms_call))
    sampler = ClockSampler(torch.cuda.current_device())
    for _ in range(calls // 2):
        st.loss_fwd_bwd(*args)
    sampler.start()
    nat.nat_trace_begin()
    for _ in range(calls - calls // 2):
        st.loss_fwd_bwd(*args)
    tr = nat.nat_trace_end()
    torch.cuda.synchronize()
    ours_clk = sampler.stop()
    assert st.status() & ~4 == 0
    traced = calls - calls // 2
    flop = 2.0 * n * w.d * w.V
    ours = {k: flop / (tr[k][0] / traced * 1e-3) / 1e12 for k in ("e", "dh", "dw")}

    # the same three products by the library, chunk by chunk, on the same values
    chunk = 8192
    W = batch["W"]
    Hc = batch["hidden"][:chunk]
    S = (Hc @ W.t()).float()
    E = torch.exp(S - S[:, :256].max(dim=1, keepdim=True).values).to(torch.bfloat16)
    del S
    Hs = (Hc.float() * (-1e-4 / E.float().sum(dim=1, keepdim=True))).to(torch.bfloat16)
    Et = E.t()
    Wt = W.t()
    out_s = torch.empty(chunk, w.V, dtype=torch.bfloat16, device="cuda")
    out_h = torch.empty(chunk, w.d, dtype=torch.bfloat16, device="cuda")
    out_w = torch.empty(w.V, w.d, dtype=torch.bfloat16, device="cuda")
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]

    def lib_chunk(record):
        if record:
            ev[0].record()
        torch.matmul(Hc, Wt, out=out_s)
        if record:
            ev[1].record()
        torch.matmul(E, W, out=out_h)
        if record:
            ev[2].record()
        torch.matmul(Et, Hs, out=out_w)
        if record:
            ev[3].record()

    ms_chunk = _time(lambda: lib_chunk(False), 4)
    reps = max(4, int(seconds * 1e3 / ms_chunk))
    for _ in range(reps // 2):
        lib_chunk(False)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    sums = [0.0, 0.0, 0.0]
    for _ in range(reps - reps // 2):
        lib_chunk(True)
        torch.cuda.synchronize()
        for j in range(3):
            sums[j] += ev[j].elapsed_time(ev[j + 1])
    lib_clk = sampler.stop()
    timed = reps - reps // 2
    cflop = 2.0 * chunk * w.d * w.V
    lib = {k: cflop / (sums[j] / timed * 1e-3) / 1e12 for j, k in enumerate(("e", "dh", "dw"))}
    peaks, kind = load_peaks()
    label = {"e": "S = Hc W^T (kE: + exp, row sums, bf16 store)",
             "dh": "dH = E W (kDh: + row factor, one-hot term)",
             "dw": "dW += E^T Hs (kDw: fp32 accumulation into dW)"}
    out = [f"{n} rows of the {base.name} head (d = {w.d}, V = {w.V}); each side looped for about "
           f"{seconds:.0f} s, second half timed; library = torch.matmul, bf16 output, no "
           f"accumulation; peaks {kind}: sustained {peaks['bf16_tflops_sustained']:.0f} TFLOP/s.", "",
           "| contraction | loss kernel TFLOP/s | library GEMM TFLOP/s | ratio |", "|---|---|---|---|"]
    for k in ("e", "dh", "dw"):
        out.append(f"| {label[k]} | {ours[k]:.0f} | {lib[k]:.0f} | {ours[k] / lib[k]:.3f} |")
    tot_o = 3.0 / sum(1.0 / ours[k] for k in ours)
    tot_l = 3.0 / sum(1.0 / lib[k] for k in lib)
    out.append(f"| all three (harmonic mean) | {tot_o:.0f} | {tot_l:.0f} | {tot_o / tot_l:.3f} |")
    out += ["", f"SM clock / board power while looping (medians): loss kernels "
            f"{ours_clk['sm_mhz']} MHz / {ours_clk['power_w']} W, library {lib_clk['sm_mhz']} MHz / "
            f"{lib_clk['power_w']} W."]
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="step",
                    choices=["step", "sweep", "stress", "ceiling", "source-hash"])
    ap.add_argument("--workload", default="qwen3_8b")
    ap.add_argument("--selection", default=None,
                    help="override the workload's selection: urs:P, rpc:C or det:BETA")
    ap.add_argument("--prompts", type=int, default=0,
                    help="override the workload's number of prompts (a reduced case of the same "
                         "head, e.g. for profiler captures)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--ref-rows", type=int, default=384,
                    help="selected rows the fp64 oracle evaluates per timed sample (about 15 s on 16 cores)")
    ap.add_argument("--sharded", action="store_true",
                    help="N > 1: the ranks split ONE batch by prompt groups (global batch size in "
                         "the weights, global response index in the selection) and all-reduce "
                         "loss and dW every step; strong scaling")
    ap.add_argument("--spawn", action="store_true",
                    help="start the ranks through the launcher even for --gpus 1 (checks the "
                         "launcher itself on a single-GPU machine)")
    ap.add_argument("--allreduce-dw", action="store_true",
                    help="N > 1, independent batches: also sum loss and dW over the ranks inside "
                         "every step (timing of the exchange only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-other-route", action="store_true",
                    help="do not also time the route that was not selected")
    ap.add_argument("--only-steps", action="store_true",
                    help="run the warm-up and the timed steps and nothing else (no per-kernel "
                         "trace, other route, end-to-end or CPU legs): the case to put under a profiler")
    ap.add_argument("--route", default="single", choices=["single", "two"],
                    help="single: nat_policy_loss_fwd_bwd; two: forward then backward calls")
    ap.add_argument("--reps", type=int, default=2, help="calls per point (sweep, stress)")
    ap.add_argument("--log2-tokens", type=int, default=28, help="stream length of --mode stress")
    args = ap.parse_args()
    if args.mode == "source-hash":
        print(kernel_source_hash())
        return
    if (args.impl == "ours" and args.mode == "step" and (args.gpus > 1 or args.spawn) and
            "WORLD_SIZE" not in os.environ):
        sys.exit(launch_ranks(args, [a for a in sys.argv[1:] if a != "--spawn"]))
    w = pick_workload(args)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.mode == "sweep":
        from paper_2603_06619_b200 import build as _build
        _build.build()
        print(fraction_sweep(w, reps=args.reps, seed=args.seed))
    elif args.mode == "stress":
        from paper_2603_06619_b200 import build as _build
        _build.build()
        print(select_compact_stress(log2_tokens=args.log2_tokens, reps=max(args.reps, 5)))
    elif args.mode == "ceiling":
        from paper_2603_06619_b200 import build as _build
        _build.build()
        print(ceiling(w))
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
