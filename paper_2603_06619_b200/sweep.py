"""Measurement helpers beyond the headline benchmark.

    python -m paper_2603_06619_b200.sweep fraction   # time vs selected-token fraction
    python -m paper_2603_06619_b200.sweep stress     # select / compact GB/s at 2^28 tokens
    python -m paper_2603_06619_b200.sweep chunk      # two row chunks of the head (for ncu)
    python -m paper_2603_06619_b200.sweep ceiling    # loss kernels vs library GEMMs, same operands

`fraction` runs the single-pass loss on the Qwen3-8B-shaped batch under every
selection setting of the sweep (URS p = 0.25 .. 1, RPC with the paper's minimum
cut of 100, deterministic 50 % truncation) and fits time = a + b * fraction.
`stress` times selection and compaction on a stream long enough (2^28 tokens)
for HBM bandwidth, not launch latency, to be what is measured.  Both print
markdown tables.  `ceiling` runs the three contractions of the single-pass loss for a few
seconds (so that the power cap, not the burst clock, sets the pace) and then the library's
plain GEMMs (torch.matmul) on the same shapes and the same operand values for as long: what
a tensor-core kernel without the loss epilogues reaches on this data under this cap.
"""
import argparse
import json
import os
import statistics

import numpy as np
import torch

from . import workloads as wl
from .step import NatStep

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def _time(fn, reps, warmup=1):
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


def fraction_sweep(name="qwen3_8b", reps=2, seed=0):
    w = wl.WORKLOADS[name]
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
    peaks, kind = _peaks()
    rows = []
    for label, kw in settings:
        st.select(cu, seed=seed, **kw)
        st.compact(cu)
        n_sel = int(st.n_sel.item())
        args = (batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
        ms = _time(lambda: st.loss_fwd_bwd(*args), reps)
        assert st.status() & ~4 == 0
        tf = 6.0 * n_sel * w.d * w.V / (ms * 1e-3) / 1e12
        rows.append((label, n_sel, n_sel / n_tot, ms, tf))
    x = np.array([r[2] for r in rows])
    y = np.array([r[3] for r in rows])
    b, a = np.polyfit(x, y, 1)
    resid = y - (a + b * x)
    out = [f"Workload {name}: N_tot = {n_tot}, d = {w.d}, V = {w.V}; single-pass "
           f"nat_policy_loss_fwd_bwd, mean of {reps} calls after 1 warm-up; peaks {kind}.", "",
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
    n_tot = 1 << log2_tokens
    B = n_tot // T
    G = 8
    P = B // G
    cu = torch.arange(0, n_tot + 1, T, dtype=torch.int32, device="cuda")
    st = NatStep(P, G, 64, 512, torch.float32, n_tot, want_grads=False)
    peaks, kind = _peaks()
    hbm = peaks["hbm_gbs"]
    out = [f"N_tot = 2^{log2_tokens} tokens, B = {B} responses of {T}; mean of {reps} calls; "
           f"HBM peak {hbm:.0f} GB/s ({kind}).", "",
           "| call | selected fraction | ms | algorithmic bytes | GB/s | of HBM peak |",
           "|---|---|---|---|---|---|"]
    for label, kw in (("URS p=0.5", dict(mode="urs", p=0.5)), ("RPC C=100", dict(mode="rpc", min_cut=100))):
        ms = _time(lambda: st.select(cu, seed=1, **kw), reps)
        nbytes = 5.0 * n_tot
        st.compact(cu)
        frac = int(st.n_sel.item()) / n_tot
        out.append(f"| nat_select {label} | {frac:.3f} | {ms:.3f} | 5 B/token (mask + pi written) | "
                   f"{nbytes / ms / 1e6:.0f} | {nbytes / ms / 1e6 / hbm:.3f} |")
        msc = _time(lambda: st.compact(cu), reps)
        cbytes = (1.0 + 8.0 * frac) * n_tot
        out.append(f"| nat_compact after {label} | {frac:.3f} | {msc:.3f} | 1 B/token read + 8 B per "
                   f"selected token written | {cbytes / msc / 1e6:.0f} | {cbytes / msc / 1e6 / hbm:.3f} |")
    st.grpo_adv(torch.zeros(B, device="cuda"))
    ms = _time(lambda: st.grpo_adv(torch.zeros(B, device="cuda")), reps)
    out.append(f"| nat_grpo_adv ({P} groups of {G}) | - | {ms:.3f} | launch bound | - | - |")
    del st
    # packing of the selected rows: the Qwen3-8B-shaped batch's hidden states under RPC
    from . import nat
    w = wl.WORKLOADS["qwen3_8b"]
    T = wl.make_lengths(w, 0)
    cu2 = torch.from_numpy(wl.cu_from_lengths(T)).cuda()
    n2 = int(T.sum())
    st2 = NatStep(w.P, w.G, 64, 512, torch.float32, n2, want_grads=False)
    st2.select(cu2, "rpc", min_cut=100, seed=0)
    st2.compact(cu2)
    n_sel = int(st2.n_sel.item())
    x = torch.randn(n2, w.d, device="cuda").to(torch.bfloat16)
    packed = torch.empty_like(x)
    full = torch.empty_like(x)
    row = w.d * 2
    ms = _time(lambda: nat.nat_gather_rows(x, st2.sel_idx, st2.n_sel, n2, packed), reps)
    gb = 2.0 * n_sel * row
    out.append(f"| nat_gather_rows ({n_sel} of {n2} rows of {row} B) | {n_sel / n2:.3f} | {ms:.3f} | "
               f"row read + row written | {gb / ms / 1e6:.0f} | {gb / ms / 1e6 / hbm:.3f} |")
    ms = _time(lambda: nat.nat_scatter_rows(packed, st2.sel_idx, st2.n_sel, n2, n2, full), reps)
    sb = 2.0 * n_sel * row + 1.0 * n2 * row
    out.append(f"| nat_scatter_rows (same, into {n2} zeroed rows) | {n_sel / n2:.3f} | {ms:.3f} | "
               f"row read + row written + zero fill | {sb / ms / 1e6:.0f} | {sb / ms / 1e6 / hbm:.3f} |")
    return "\n".join(out)


def one_chunk_sample(name="qwen3_8b", rows=16384, calls=2):
    """The single-pass loss on `rows` tokens of the workload's head (two 8192-row chunks by
    default): a small case for profiler captures whose launches have the benchmark's
    per-launch shape (one chunk of this head per launch)."""
    base = wl.WORKLOADS[name]
    T = rows // base.G
    w = wl.variant(base, P=1, sel_mode="urs", p=1.0, length_law="uniform", len_lo=T, len_hi=T)
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = NatStep(w.P, w.G, w.d, w.V, torch.bfloat16, batch["n_tot"])
    cu = batch["cu_seqlens"]
    st.grpo_adv(batch["rewards"])
    st.select(cu, "urs", p=1.0)
    st.compact(cu)
    for _ in range(calls):
        st.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
        torch.cuda.synchronize()
    assert st.status() & ~4 == 0
    return f"{int(st.n_sel.item())} rows of the {name} head, {calls} single-pass calls"


def _clock_sampler():
    import subprocess
    try:
        return subprocess.Popen(
            ["nvidia-smi", "-i", str(torch.cuda.current_device()), "--query-gpu=clocks.sm,power.draw",
             "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE,
            stderr=subprocess.DEVNULL, text=True)
    except OSError:
        return None


def _clock_median(proc):
    if proc is None:
        return float("nan"), float("nan")
    proc.terminate()
    out, _ = proc.communicate(timeout=10)
    sm, pw = [], []
    for line in out.splitlines():
        parts = [c.strip() for c in line.split(",")]
        try:
            sm.append(float(parts[0]))
            pw.append(float(parts[1]))
        except (ValueError, IndexError):
            continue
    # the upper half of the samples: those taken while the loop was running
    sm.sort()
    pw.sort()
    half = len(sm) // 2
    return (statistics.median(sm[half:]) if sm else float("nan"),
            statistics.median(pw[half:]) if pw else float("nan"))


def ceiling(name="qwen3_8b", rows=32768, seconds=4.0):
    """Per contraction: TFLOP/s of the loss kernels and of the library GEMM on the same
    operands, each measured inside a loop that runs for `seconds` under the power cap."""
    from . import nat
    base = wl.WORKLOADS[name]
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
    proc = _clock_sampler()
    for _ in range(calls // 2):
        st.loss_fwd_bwd(*args)
    nat.nat_trace_begin()
    for _ in range(calls - calls // 2):
        st.loss_fwd_bwd(*args)
    tr = nat.nat_trace_end()
    torch.cuda.synchronize()
    ours_clk = _clock_median(proc)
    assert st.status() & ~4 == 0
    traced = calls - calls // 2
    flop = 2.0 * n * w.d * w.V
    ours = {k: flop / (tr[k][0] / traced * 1e-3) / 1e12 for k in ("e", "dh", "dw")}

    # the same three products by the library, chunk by chunk, on the same values
    chunk = 8192
    H = batch["hidden"][:n]
    W = batch["W"]
    Hc = H[:chunk]
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
    proc = _clock_sampler()
    for _ in range(reps // 2):
        lib_chunk(False)
    sums = [0.0, 0.0, 0.0]
    for _ in range(reps - reps // 2):
        lib_chunk(True)
        torch.cuda.synchronize()
        for j in range(3):
            sums[j] += ev[j].elapsed_time(ev[j + 1])
    lib_clk = _clock_median(proc)
    timed = reps - reps // 2
    cflop = 2.0 * chunk * w.d * w.V
    lib = {k: cflop / (sums[j] / timed * 1e-3) / 1e12 for j, k in enumerate(("e", "dh", "dw"))}
    peaks, kind = _peaks()
    label = {"e": "S = Hc W^T (kE: + exp, row sums, bf16 store)",
             "dh": "dH = E W (kDh: + row factor, one-hot term)",
             "dw": "dW += E^T Hs (kDw: fp32 accumulation into dW)"}
    out = [f"{n} rows of the {name} head (d = {w.d}, V = {w.V}); each side looped for about "
           f"{seconds:.0f} s, second half timed; library = torch.matmul, bf16 output, no "
           f"accumulation; peaks {kind}: sustained {peaks['bf16_tflops_sustained']:.0f} TFLOP/s.", "",
           "| contraction | loss kernel TFLOP/s | library GEMM TFLOP/s | ratio |", "|---|---|---|---|"]
    for k in ("e", "dh", "dw"):
        out.append(f"| {label[k]} | {ours[k]:.0f} | {lib[k]:.0f} | {ours[k] / lib[k]:.3f} |")
    tot_o = 3.0 / sum(1.0 / ours[k] for k in ours)
    tot_l = 3.0 / sum(1.0 / lib[k] for k in lib)
    out.append(f"| all three (harmonic mean) | {tot_o:.0f} | {tot_l:.0f} | {tot_o / tot_l:.3f} |")
    out += ["", f"SM clock / board power while looping (median of the busy samples): loss kernels "
            f"{ours_clk[0]:.0f} MHz / {ours_clk[1]:.0f} W, library {lib_clk[0]:.0f} MHz / "
            f"{lib_clk[1]:.0f} W."]
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["fraction", "stress", "chunk", "ceiling"])
    ap.add_argument("--workload", default="qwen3_8b")
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--log2-tokens", type=int, default=28)
    args = ap.parse_args()
    if args.what == "chunk":
        print(one_chunk_sample(args.workload))
    elif args.what == "ceiling":
        print(ceiling(args.workload))
    elif args.what == "fraction":
        print(fraction_sweep(args.workload, reps=args.reps))
    else:
        print(select_compact_stress(log2_tokens=args.log2_tokens, reps=max(args.reps, 5)))


if __name__ == "__main__":
    main()
