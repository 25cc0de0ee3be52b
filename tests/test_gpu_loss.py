"""GPU parity: policy-loss forward and backward against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_06619_b200 import nat
from paper_2603_06619_b200 import workloads as wl

import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "tiny_rpc"])
@pytest.mark.parametrize("seed", [0, 1])
def test_tiny_fp32(name, seed):
    out, _ = parity.run_case(wl.WORKLOADS[name], seed=seed)
    assert out["dH_err"] < 1e-4 and out["dW_err"] < 1e-4


def test_tiny_wide_noise_and_full_token():
    # both clip branches fire with sigma = 0.3; p = 1 is full-token GRPO
    w = wl.variant(wl.WORKLOADS["tiny"], old_noise=0.3)
    out, ref = parity.run_case(w, seed=2)
    assert (ref["g"] == 0).any() and (ref["g"] != 0).any()
    parity.run_case(wl.variant(w, p=1.0), seed=2)
    parity.run_case(wl.variant(w, sel_mode="det", beta=0.5), seed=2)


@pytest.mark.parametrize("mode", ["urs", "rpc"])
def test_mid_bf16(mode):
    # 3 row tiles with a ragged tail, 20 vocabulary tiles with a ragged tail, 2 splits
    w = wl.variant(wl.WORKLOADS["mid"], sel_mode=mode, min_cut=5)
    parity.run_case(w, seed=0)


def test_mid_bf16_peaked_softmax():
    # logits with std ~8: exercises the running-max rescaling and makes the
    # softmax part of the gradients as large as the one-hot part
    w = wl.variant(wl.WORKLOADS["mid"], w_scale=0.5, old_noise=0.3)
    out, ref = parity.run_case(w, seed=1)
    assert out["dH_dense_err"] <= parity.TOL_DENSE


def test_mid_bf16_multi_chunk_shapes():
    # d not a multiple of 256 and V not a multiple of 8; more rows than one group of tiles
    w = wl.variant(wl.WORKLOADS["mid"], d=320, V=3001, P=4, G=8, len_lo=60, len_hi=200, p=0.75)
    parity.run_case(w, seed=3)


def test_k_parts_with_ragged_columns_and_vocabulary():
    # V large enough for the dHidden contraction to run in K parts (their partial tiles meet
    # in the float32 scratch), with d not a multiple of the 256-column block and V not a
    # multiple of the 64-entry k-block: the last column block and the last k-block are ragged
    w = wl.variant(wl.WORKLOADS["mid"], d=320, V=20001, P=4, G=8, len_lo=60, len_hi=200, p=0.75,
                   old_noise=0.3)
    parity.run_case(w, seed=3, routes=(False, True))
    parity.run_case(wl.variant(w, d=64, V=9000, w_scale=0.5), seed=4, routes=(False, True))


def test_twin_0p6b():
    parity.run_case(wl.WORKLOADS["twin_0p6b"], seed=0, routes=(False, True))


def test_twin_8b():
    parity.run_case(wl.WORKLOADS["twin_8b"], seed=0, routes=(False, True))


@pytest.mark.parametrize("name,w_scale", [("twin_0p6b", 0.5), ("twin_8b", 0.15), ("twin_8b", 0.5)])
def test_twins_with_peaked_softmax(name, w_scale):
    """The real heads (d = 1024 / 4096, V = 151936) with logits of standard deviation 16,
    ~10 and 32 instead of ~1: the softmax part of the gradients is then as large as the
    one-hot part, so the dense-part comparison of dHidden is not hidden behind bf16
    rounding, and the running-max rescaling of the forward is exercised.  (At standard
    deviation 32 a row's largest logit can exceed the single-pass window above its
    reference; the single-pass call then redoes the chunk with the two-pass kernels.)"""
    w = wl.variant(wl.WORKLOADS[name], w_scale=w_scale, old_noise=0.3)
    out, ref = parity.run_case(w, seed=1, routes=(False, True))
    resolv = 2.0 ** -9 * np.linalg.norm(ref["dH"]) / np.linalg.norm(ref["dH_dense"])
    assert resolv < 5e-3                       # the bf16 slack is small here: the check bites
    assert out["dH_dense_err"] <= parity.TOL_DENSE
    assert out["status"] & ~nat.NAT_DEV_FALLBACK == 0


def test_accumulate_dW_and_dloss():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = parity.gpu_step(w, batch, 0, 0)
    base = st.dW.clone()
    baseH = st.dH.clone()
    dloss = torch.tensor([-2.0], device="cuda")
    st.loss_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"],
                batch["cu_seqlens"], dloss=dloss, accumulate_dW=True)
    torch.cuda.synchronize()
    n = int(st.n_sel.item())
    assert parity.rel_fro(st.dW.cpu().numpy(), -base.cpu().numpy()) < 1e-2
    assert parity.rel_fro(st.dH[:n].float().cpu().numpy(), -2 * baseH[:n].float().cpu().numpy()) < 1e-2


def test_compact_hidden_layout():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=4, device="cuda")
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 4, 0)
    idx = torch.from_numpy(ref_sel["sel_idx"]).long().cuda()
    compact = dict(batch, hidden=batch["hidden"][idx].contiguous())
    st = parity.gpu_step(w, compact, 4, 0, hidden_is_compact=True)
    parity.check_selection(st, ref_sel, w)
    parity.check_loss(st, ref_sel, nb, w)


def test_empty_selection_and_reruns_are_deterministic():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = parity.gpu_step(w, batch, 0, 0)
    loss1, logp1, dW1 = st.loss.clone(), st.logp.clone(), st.dW.clone()
    st.run(batch, w.sel_mode, p=w.p, seed=0)
    torch.cuda.synchronize()
    assert torch.equal(loss1, st.loss) and torch.equal(logp1, st.logp)
    assert torch.equal(dW1, st.dW)
    # nothing selected: loss 0 and zero dW
    st.mask.zero_()
    st.compact(batch["cu_seqlens"])
    st.loss_fwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], batch["cu_seqlens"])
    st.loss_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], batch["cu_seqlens"])
    torch.cuda.synchronize()
    assert int(st.n_sel.item()) == 0 and float(st.loss.item()) == 0.0
    assert float(st.dW.abs().max().item()) == 0.0 and st.status() == 0


def test_capacity_overflow_is_reported():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = parity.gpu_step(w, batch, 0, 0, backward=False, n_sel_cap=128)
    assert int(st.n_sel.item()) > 128
    assert st.status() & nat.NAT_DEV_CAPACITY


def test_unsupported_shapes_are_rejected():
    p = nat.loss_params(100, 512, torch.bfloat16, 8)      # d % 64 != 0
    t = torch.zeros(1024, device="cuda")
    ws = nat.alloc_workspace(1 << 20, "cuda")
    with pytest.raises(nat.NatError):
        nat.nat_policy_loss_fwd(p, t, t, t, t, t, t, t, t, t, t, 4, t, t, t, ws)
    p = nat.loss_params(64, 512, torch.float32, 8)
    tiny_ws = nat.alloc_workspace(256, "cuda")
    with pytest.raises(nat.NatError):
        nat.nat_policy_loss_fwd(p, t, t, t, t, t, t, t, t, t, t, 4096, t, t, t, tiny_ws)


# ---- single-pass route: nat_policy_loss_fwd_bwd ------------------------------------
@pytest.mark.parametrize("name", ["tiny", "mid"])
def test_fused_matches_oracle(name):
    parity.run_case(wl.WORKLOADS[name], seed=0, fused=True)


def test_fused_variants():
    mid = wl.WORKLOADS["mid"]
    parity.run_case(wl.variant(mid, sel_mode="rpc", min_cut=5), seed=0, fused=True)
    out, _ = parity.run_case(wl.variant(mid, w_scale=0.5, old_noise=0.3), seed=1, fused=True)
    assert out["dH_dense_err"] <= parity.TOL_DENSE
    parity.run_case(wl.variant(mid, d=320, V=3001, P=4, G=8, len_lo=60, len_hi=200, p=0.75),
                    seed=3, fused=True)


def _two_chunk_batch(spike):
    """~10k selected rows (two row chunks).  With `spike`, vocabulary row 700 gets a logit
    of 100 * h[0]; h[0] is zero in the first half of the stream, so only the second chunk
    leaves the single-pass window."""
    w = wl.variant(wl.WORKLOADS["mid"], d=64, V=1024, P=8, G=8, len_lo=250, len_hi=380, p=0.5)
    batch = wl.make_batch(w, seed=6, device="cuda")
    if spike:
        half = batch["n_tot"] // 2
        batch["hidden"][:half, 0] = 0
        batch["W"][700, :] = 0
        batch["W"][700, 0] = 100.0
        noise = torch.randn(batch["n_tot"], device="cuda") * 0.05
        batch["old_logp"] = wl.library_logp(batch["hidden"], batch["W"], batch["targets"]) + noise
    return w, batch


@pytest.mark.parametrize("spike", [False, True])
def test_fused_two_chunks_and_window_fallback(spike):
    w, batch = _two_chunk_batch(spike)
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 6, 0)
    assert 8192 < ref_sel["n_sel"] < 16384
    st = parity.gpu_step(w, batch, 6, 0, fused=True)
    parity.check_selection(st, ref_sel, w)
    parity.check_loss(st, ref_sel, nb, w)
    assert bool(st.status() & nat.NAT_DEV_FALLBACK) == spike
    # the two routes agree with each other as well
    st2 = parity.gpu_step(w, batch, 6, 0, fused=False)
    n = ref_sel["n_sel"]
    assert parity.rel_fro(st.dW.cpu().numpy(), st2.dW.cpu().numpy()) < 1e-2
    assert float((st.logp[:n] - st2.logp[:n]).abs().max()) < 2 * parity.TOL_LOGP


def test_fused_accumulate_and_dloss():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = parity.gpu_step(w, batch, 0, 0, fused=True)
    base, baseH, loss = st.dW.clone(), st.dH.clone(), st.loss.clone()
    dloss = torch.tensor([-2.0], device="cuda")
    st.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"],
                    batch["cu_seqlens"], dloss=dloss, accumulate_dW=True)
    torch.cuda.synchronize()
    n = int(st.n_sel.item())
    assert torch.equal(loss, st.loss)
    assert parity.rel_fro(st.dW.cpu().numpy(), -base.cpu().numpy()) < 1e-2
    assert parity.rel_fro(st.dH[:n].float().cpu().numpy(), -2 * baseH[:n].float().cpu().numpy()) < 1e-2


def test_fused_compact_hidden_layout():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=4, device="cuda")
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 4, 0)
    idx = torch.from_numpy(ref_sel["sel_idx"]).long().cuda()
    compact = dict(batch, hidden=batch["hidden"][idx].contiguous())
    st = parity.gpu_step(w, compact, 4, 0, hidden_is_compact=True, fused=True)
    parity.check_selection(st, ref_sel, w)
    parity.check_loss(st, ref_sel, nb, w)


def test_fused_empty_selection_capacity_and_reruns():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    args = (batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], batch["cu_seqlens"])
    st = parity.gpu_step(w, batch, 0, 0, fused=True)
    loss1, logp1, dH1, dW1 = st.loss.clone(), st.logp.clone(), st.dH.clone(), st.dW.clone()
    st.run(batch, w.sel_mode, p=w.p, seed=0, fused=True)
    torch.cuda.synchronize()
    n = int(st.n_sel.item())
    assert torch.equal(loss1, st.loss) and torch.equal(logp1[:n], st.logp[:n])
    assert torch.equal(dH1[:n], st.dH[:n])            # every sum has a fixed order
    assert torch.equal(dW1, st.dW)
    # nothing selected: loss 0 and zero dW
    st.mask.zero_()
    st.compact(batch["cu_seqlens"])
    st.loss_fwd_bwd(*args)
    torch.cuda.synchronize()
    assert int(st.n_sel.item()) == 0 and float(st.loss.item()) == 0.0
    assert float(st.dW.abs().max().item()) == 0.0 and st.status() == 0
    # more tokens selected than the stated capacity: reported, the first rows are still right
    cap = 300                                          # not a multiple of any tile extent
    st2 = parity.gpu_step(w, batch, 0, 0, fused=True, n_sel_cap=cap)
    assert int(st2.n_sel.item()) > cap
    assert st2.status() & nat.NAT_DEV_CAPACITY
    assert float((st2.logp[:cap] - logp1[:cap]).abs().max()) < parity.TOL_LOGP
    assert parity.rel_fro(st2.dH[:cap].float().cpu().numpy(), dH1[:cap].float().cpu().numpy()) < 1e-2


def test_trace_reports_per_kernel_time():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    st = parity.gpu_step(w, batch, 0, 0, fused=True)
    nat.nat_trace_begin()
    st.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"],
                    batch["cu_seqlens"])
    tr = nat.nat_trace_end()
    assert tr["e"][1] == 1 and tr["e"][0] > 0 and tr["dh"][0] > 0 and tr["dw"][0] > 0
    assert tr["dz"][1] == 1            # the predicated redo was launched (and did nothing)
    # tracing is off again: nothing is recorded by later calls
    st.loss_fwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], batch["cu_seqlens"])
    nat.nat_trace_begin()
    assert all(v == (0.0, 0) for v in nat.nat_trace_end().values())


@pytest.mark.parametrize("name,fused", [("tiny", False), ("mid", False), ("mid", True)])
def test_kl_term(name, fused):
    # Eq. grpo-token-loss with kl_beta > 0 (sampled-token KL against a reference policy)
    w = wl.variant(wl.WORKLOADS[name], old_noise=0.3)
    batch = wl.make_batch(w, seed=5, device="cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    ref_logp = batch["old_logp"] + 0.1 * torch.randn(batch["n_tot"], generator=g, device="cuda")
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 5, 0)
    st = parity.gpu_step(w, batch, 5, 0, fused=fused, kl_beta=0.05, ref_logp=ref_logp)
    parity.check_selection(st, ref_sel, w)
    out, ref = parity.check_loss(st, ref_sel, nb, w, kl_beta=0.05,
                                 ref_logp=ref_logp.cpu().numpy())
    base = oracle.policy_loss_fwd(nb["hidden"], nb["W"], nb["targets"], nb["old_logp"],
                                  ref_sel["adv"], ref_sel["pi"], nb["cu_seqlens"],
                                  ref_sel["sel_idx"], ref_sel["sel_resp"])
    assert abs(ref["loss"] - base["loss"]) > 1e-4          # the term is not a no-op here
    # kl_beta != 0 without a reference is refused
    with pytest.raises(nat.NatError):
        parity.gpu_step(w, batch, 5, 0, fused=fused, kl_beta=0.05, ref_logp=None)


def test_dW_is_reproducible_when_many_tokens_share_a_target():
    # 40 distinct targets over ~800 selected tokens: every target row of dW receives some
    # twenty one-hot terms, whose order of summation must not depend on the run
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=7, device="cuda")
    batch["targets"] = (batch["targets"] % 40).to(torch.int32)
    batch["old_logp"] = wl.library_logp(batch["hidden"], batch["W"], batch["targets"]) + \
        0.05 * torch.randn(batch["n_tot"], device="cuda")
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 7, 0)
    ref = None
    for fused in (False, True):
        st = parity.gpu_step(w, batch, 7, 0, fused=fused)
        out, ref = parity.check_loss(st, ref_sel, nb, w, ref=ref)
        dW1 = st.dW.clone()
        for _ in range(3):
            st.run(batch, w.sel_mode, p=w.p, seed=7, fused=fused)
            torch.cuda.synchronize()
            assert torch.equal(dW1, st.dW)


def test_dHidden_is_reproducible_when_the_vocabulary_is_cut_into_many_K_parts():
    # d = 1024 with few row blocks: the dHidden contraction runs in eight K parts, whose
    # partial tiles must be added in the same order on every run
    w = wl.variant(wl.WORKLOADS["twin_0p6b"], P=2, len_lo=200, len_hi=400, p=1.0)
    batch = wl.make_batch(w, seed=5, device="cuda")
    for fused in (False, True):
        st = parity.gpu_step(w, batch, 5, 0, fused=fused)
        dH1, dW1, loss1 = st.dH.clone(), st.dW.clone(), st.loss.clone()
        for _ in range(4):
            st.run(batch, w.sel_mode, p=w.p, seed=5, fused=fused)
            torch.cuda.synchronize()
            assert torch.equal(dH1, st.dH) and torch.equal(dW1, st.dW)
            assert torch.equal(loss1, st.loss)


def test_target_outside_the_vocabulary_is_reported_and_left_out():
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=0, device="cuda")
    nb = wl.to_numpy(batch)
    ref_sel = parity.oracle_selection(w, nb, 0, 0)
    bad = ref_sel["sel_idx"][[3, 200]]
    clean = {}
    for fused in (False, True):
        st = parity.gpu_step(w, batch, 0, 0, fused=fused)
        clean[fused] = (st.dW.clone(), st.dH.clone(), st.logp.clone())
    targets = batch["targets"].clone()
    targets[int(bad[0])] = w.V + 5
    targets[int(bad[1])] = -1
    poisoned = dict(batch, targets=targets)
    for fused in (False, True):
        st = parity.gpu_step(w, poisoned, 0, 0, fused=fused)
        assert st.status() & nat.NAT_DEV_BAD_TARGET
        n = ref_sel["n_sel"]
        logp = st.logp[:n]
        assert torch.isnan(logp[3]) and torch.isnan(logp[200]) and int(torch.isnan(logp).sum()) == 2
        assert torch.all(st.dH[3] == 0) and torch.all(st.dH[200] == 0)
        keep = torch.ones(n, dtype=torch.bool, device="cuda")
        keep[3] = keep[200] = False
        assert torch.equal(st.dH[:n][keep], clean[fused][1][:n][keep])
        assert torch.isfinite(st.dW).all() and torch.isfinite(st.loss).all()
    # a clean batch leaves the bit clear
    assert parity.gpu_step(w, batch, 0, 0, fused=True).status() & nat.NAT_DEV_BAD_TARGET == 0
