"""Shared helpers of the GPU parity tests: run the CUDA path and the oracle on
the same seeded batch and compare.

Tolerances (from the target statement of the method's numerics):
  masks, pi, cut lengths, compacted indices, advantages   bit-exact
  loss                  1e-3 relative (against a floor tied to sum |w S|, since the
                        loss is a near-cancelling sum on centred advantages)
  logp, lse             2e-4 absolute (fp32 accumulation of bf16 products) for logits of
                        the workloads' size (lse <= 16); the rounding of an fp32 running
                        sum is relative to its magnitude, so for the peaked-softmax variants
                        (logits of standard deviation 10..32) this tolerance and the loss
                        floor grow in proportion, by max(1, max lse / 16)
  dHidden, dW           1e-2 relative Frobenius error
  dense parts           2e-2 relative Frobenius error (gradient minus its
                        one-hot target term: the softmax part alone, which the
                        whole-tensor norm would hide behind the one-hot term)
"""
import numpy as np
import torch

import oracle
from paper_2603_06619_b200 import workloads as wl
from paper_2603_06619_b200.step import NatStep

TOL_LOSS = 1e-3
TOL_LOGP = 2e-4
TOL_GRAD = 1e-2
TOL_DENSE = 2e-2

MODE_ID = {"urs": oracle.SEL_URS, "rpc": oracle.SEL_RPC, "det": oracle.SEL_DET}


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a))


def oracle_selection(w, nb, seed, offset, eps=1e-6):
    adv = oracle.grpo_adv(nb["rewards"], w.P, w.G, eps)
    mask, pi, cut = oracle.select(MODE_ID[w.sel_mode], nb["cu_seqlens"], p=w.p, min_cut=w.min_cut,
                                  beta=w.beta, seed=seed, offset=offset)
    si, sr, so, n = oracle.compact(mask, nb["cu_seqlens"])
    return dict(adv=adv, mask=mask, pi=pi, cut=cut, sel_idx=si, sel_resp=sr, sel_offsets=so,
                n_sel=n)


def gpu_step(w, batch, seed, offset, backward=True, n_sel_cap=None, fused=False, **kw):
    dtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    st = NatStep(w.P, w.G, w.d, w.V, dtype, batch["n_tot"], n_sel_cap=n_sel_cap, **kw)
    st.run(batch, w.sel_mode, p=w.p, min_cut=w.min_cut, beta=w.beta, seed=seed, offset=offset,
           backward=backward, fused=fused)
    torch.cuda.synchronize()
    return st


def check_selection(st, ref, w):
    n = ref["n_sel"]
    assert int(st.n_sel.item()) == n
    assert np.array_equal(st.adv.cpu().numpy().view(np.uint32), ref["adv"].view(np.uint32))
    nt = ref["mask"].shape[0]
    assert np.array_equal(st.mask[:nt].cpu().numpy(), ref["mask"])
    assert np.array_equal(st.pi[:nt].cpu().numpy().view(np.uint32), ref["pi"].view(np.uint32))
    if ref["cut"] is not None:
        assert np.array_equal(st.cut_len[:w.B].cpu().numpy(), ref["cut"])
    assert np.array_equal(st.sel_idx[:n].cpu().numpy(), ref["sel_idx"])
    assert np.array_equal(st.sel_resp[:n].cpu().numpy(), ref["sel_resp"])
    assert np.array_equal(st.sel_offsets.cpu().numpy(), ref["sel_offsets"])


def check_loss(st, ref_sel, nb, w, backward=True, hidden_is_compact=False, clip=(0.2, 0.2),
               hidden_np=None, kl_beta=0.0, ref_logp=None, ref=None, B_global=None):
    """Element-by-element comparison of loss, logp, lse, dHidden, dW with the oracle.

    ``ref``: the oracle's result from an earlier call on the same inputs (the fp64
    evaluation is the expensive part; two routes of the library are checked against one).
    """
    n = ref_sel["n_sel"]
    hidden = nb["hidden"] if hidden_np is None else hidden_np
    if ref is None:
        fn = oracle.policy_loss_bwd if backward else oracle.policy_loss_fwd
        ref = fn(hidden, nb["W"], nb["targets"], nb["old_logp"], ref_sel["adv"], ref_sel["pi"],
                 nb["cu_seqlens"], ref_sel["sel_idx"], ref_sel["sel_resp"], clip_lo=clip[0],
                 clip_hi=clip[1], hidden_is_compact=hidden_is_compact, kl_beta=kl_beta,
                 ref_logp=ref_logp)
    assert st.status() & ~4 == 0      # the informational fallback bit may be set
    got_logp = st.logp[:n].cpu().numpy()
    got_lse = st.lse[:n].cpu().numpy()
    mag = max(1.0, float(np.abs(ref["lse"]).max(initial=0)) / 16.0)
    out = dict(logp_err=float(np.abs(got_logp - ref["logp"]).max(initial=0)),
               lse_err=float(np.abs(got_lse - ref["lse"]).max(initial=0)), logit_mag=mag)
    assert out["logp_err"] <= TOL_LOGP * mag, out
    assert out["lse_err"] <= TOL_LOGP * mag, out
    loss = float(st.loss.item())
    floor = 1e-2 * mag * float(np.sum(ref["w"] * np.abs(ref["L"])))
    assert abs(loss - ref["loss"]) <= TOL_LOSS * max(abs(ref["loss"]), floor), (loss, ref["loss"])
    out.update(loss=loss, ref_loss=ref["loss"])
    if backward:
        dH = st.dH[:n].float().cpu().numpy()
        dW = st.dW.cpu().numpy()
        out["dH_err"] = rel_fro(dH, ref["dH"])
        out["dW_err"] = rel_fro(dW, ref["dW"])
        assert out["dH_err"] <= TOL_GRAD, out
        assert out["dW_err"] <= TOL_GRAD, out
        if np.any(ref["g"] != 0):
            # softmax-only parts: subtract the oracle's one-hot terms from both sides
            oh_H = ref["dH"] - ref["dH_dense"]
            oh_W = ref["dW"] - ref["dW_dense"]
            out["dH_dense_err"] = rel_fro(dH - oh_H, ref["dH_dense"])
            out["dW_dense_err"] = rel_fro(dW - oh_W, ref["dW_dense"])
            if w.dtype == "f32":
                assert out["dH_dense_err"] <= TOL_DENSE, out
            else:
                # dHidden is stored in bf16: its rounding (2^-9 of the one-hot
                # dominated total) bounds what the subtraction can resolve
                resolv = 2.0 ** -9 * np.linalg.norm(ref["dH"]) / np.linalg.norm(ref["dH_dense"])
                assert out["dH_dense_err"] <= TOL_DENSE + resolv, out
            assert out["dW_dense_err"] <= TOL_DENSE, out
    return out, ref


def settle_clip_decisions(batch, nb, ref_sel, clip=(0.2, 0.2), band=2e-3, shift=2e-2):
    """Move tokens off the clip bounds, in the inputs of both sides.

    The derivative of the clipped surrogate (Eq. grpo-surrogate) jumps where the ratio
    crosses 1 - clip_lo or 1 + clip_hi, so a token whose ratio lies within the forward's
    numerical error of a bound has no unique gradient: the kernels' forward (bf16 products,
    fp32 sums) and the fp64 oracle may land on different sides, and both are right.  Tokens
    with |log r - log bound| < band * max(1, max lse / 16) (r from the oracle's logp) get
    their old_logp moved by ten times that, away from the bound.  Returns how many moved."""
    fwd = oracle.policy_loss_fwd(nb["hidden"], nb["W"], nb["targets"], nb["old_logp"],
                                 ref_sel["adv"], ref_sel["pi"], nb["cu_seqlens"],
                                 ref_sel["sel_idx"], ref_sel["sel_resp"], clip_lo=clip[0],
                                 clip_hi=clip[1])
    si = np.asarray(ref_sel["sel_idx"], dtype=np.int64)
    mag = max(1.0, float(np.abs(fwd["lse"]).max(initial=0)) / 16.0)
    old = nb["old_logp"]
    logr = fwd["logp"] - old[si].astype(np.float64)
    moved = 0
    for bound in (np.log1p(clip[1]), np.log1p(-clip[0])):
        near = np.abs(logr - bound) < band * mag
        if near.any():
            # log r = logp - old_logp: lower old_logp to push a ratio further above the bound
            step = np.where(logr[near] >= bound, -1.0, 1.0) * (shift * mag)
            old[si[near]] = (old[si[near]].astype(np.float64) + step).astype(np.float32)
            moved += int(near.sum())
    if moved:
        batch["old_logp"].copy_(torch.from_numpy(old))
    return moved


def run_case(w, seed=0, offset=0, backward=True, device="cuda", fused=False, routes=None,
             **batch_kw):
    """One seeded batch through the library and the oracle.  ``routes`` lists the library
    routes to check against the single oracle evaluation (False: forward then backward
    calls, True: the single-pass call); default: the one ``fused`` names."""
    batch = wl.make_batch(w, seed=seed, device=device, **batch_kw)
    nb = wl.to_numpy(batch)
    ref_sel = oracle_selection(w, nb, seed, offset)
    if backward:
        settle_clip_decisions(batch, nb, ref_sel)
    out, ref = None, None
    for f in ([fused] if routes is None else routes):
        st = gpu_step(w, batch, seed, offset, backward=backward, fused=f)
        check_selection(st, ref_sel, w)
        out, ref = check_loss(st, ref_sel, nb, w, backward=backward, ref=ref)
        out["status"] = st.status()
        del st
    return out, ref
