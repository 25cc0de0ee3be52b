"""Pins for the oracle's policy loss and gradients (CPU only).

Each test ties the oracle to something it does not compute itself: a library
routine, a closed form, an independently written double loop, finite
differences, or the exhaustive expectation over masks / cuts (Proposition 1).
"""
import itertools
import math

import numpy as np
import pytest
from scipy.special import log_softmax

from oracle import (SEL_DET, SEL_RPC, SEL_URS, compact, grad_coeff, grpo_adv, policy_loss_bwd,
                    policy_loss_dW_rows, policy_loss_fwd, select, select_cutlaw)
from paper_2603_06619_b200 import workloads as wl


def _tiny(seed=0, lengths=None, mode="urs", old_noise=None, rewards=None):
    w = wl.WORKLOADS["tiny"]
    if old_noise is not None:
        w = wl.variant(w, old_noise=old_noise)
    b = wl.to_numpy(wl.make_batch(w, seed=seed, lengths=lengths))
    if rewards is not None:
        b["rewards"] = np.asarray(rewards, dtype=np.float32)
    b["adv"] = grpo_adv(b["rewards"], w.P, w.G, 1e-6)
    return w, b


def _full_token_grpo(b, B, clip=0.2):
    """Full-token GRPO written out as plain loops over responses and tokens
    (sequence mean, then batch mean; Eq. grpo-obj with beta = 0), negated."""
    cu = b["cu_seqlens"]
    H = b["hidden"].astype(np.float64)
    W = b["W"].astype(np.float64)
    total = 0.0
    for i in range(B):
        T = cu[i + 1] - cu[i]
        acc = 0.0
        for n in range(cu[i], cu[i + 1]):
            z = W @ H[n]
            lp = log_softmax(z)[b["targets"][n]]
            r = math.exp(lp - float(b["old_logp"][n]))
            A = float(b["adv"][i])
            acc += min(r * A, min(max(r, 1 - clip), 1 + clip) * A)
        total += acc / T
    return -total / B


def _run(b, mask, pi, **kw):
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    return policy_loss_bwd(b["hidden"], b["W"], b["targets"], b["old_logp"], b["adv"], pi,
                           b["cu_seqlens"], si, sr, **kw)


def test_softmax_rows_sum_to_one_and_match_library():
    w, b = _tiny()
    mask, pi, _ = select(SEL_URS, b["cu_seqlens"], p=0.5, seed=0)
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    out = policy_loss_fwd(b["hidden"], b["W"], b["targets"], b["old_logp"], b["adv"], pi,
                          b["cu_seqlens"], si, sr)
    z = b["hidden"][si].astype(np.float64) @ b["W"].astype(np.float64).T
    np.testing.assert_allclose(np.exp(z - out["lse"][:, None]).sum(1), 1.0, rtol=1e-13)
    lib = log_softmax(z, axis=1)[np.arange(n), b["targets"][si]]
    np.testing.assert_allclose(out["logp"], lib, rtol=1e-12, atol=1e-12)
    # compact layout gives the same numbers as gathering from [N_tot, d]
    out2 = policy_loss_fwd(b["hidden"][si], b["W"], b["targets"], b["old_logp"], b["adv"], pi,
                           b["cu_seqlens"], si, sr, hidden_is_compact=True)
    assert out2["loss"] == out["loss"]


def test_p_equal_one_is_full_token_grpo():
    w, b = _tiny(old_noise=0.3)
    for mode, kw in ((SEL_URS, dict(p=1.0)), (SEL_DET, dict(beta=1.0))):
        mask, pi, _ = select(mode, b["cu_seqlens"], seed=1, **kw)
        assert mask.all()
        out = _run(b, mask, pi, want_dW=False)
        want = _full_token_grpo(b, w.B)
        assert abs(out["loss"] - want) <= 1e-12 * max(1.0, abs(want))
    # RPC realised at L_i = T_i with pi forced to 1 is the same thing
    out = _run(b, np.ones_like(mask), np.ones_like(pi), want_dW=False)
    assert abs(out["loss"] - want) <= 1e-12


def test_old_logp_equal_logp_closed_form():
    # r = 1 => S = A, so loss = - sum_n w_n A_resp(n): a function of the mask alone
    w, b = _tiny()
    mask, pi, cut = select(SEL_RPC, b["cu_seqlens"], min_cut=1, seed=5)
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    ref = policy_loss_fwd(b["hidden"], b["W"], b["targets"], b["old_logp"], b["adv"], pi,
                          b["cu_seqlens"], si, sr)
    old = b["old_logp"].astype(np.float64).copy()
    old[si] = ref["logp"]
    out = policy_loss_fwd(b["hidden"], b["W"], b["targets"], old, b["adv"], pi,
                          b["cu_seqlens"], si, sr)
    cu = b["cu_seqlens"]
    want = 0.0
    for i in range(w.B):
        T = cu[i + 1] - cu[i]
        for t in range(1, cut[i] + 1):
            want -= float(b["adv"][i]) / (float(pi[cu[i] + t - 1]) * T * w.B)
    assert abs(out["loss"] - want) < 1e-12
    np.testing.assert_allclose(out["ratio"], 1.0, rtol=1e-12)
    # and at p = 1 it is -(1/B) sum_i A_i, which is ~0 because groups are centred
    ones = np.ones_like(mask)
    si, sr, so, n = compact(ones, cu)
    ref = policy_loss_fwd(b["hidden"], b["W"], b["targets"], b["old_logp"], b["adv"],
                          np.ones_like(pi), cu, si, sr)
    out = policy_loss_fwd(b["hidden"], b["W"], b["targets"], ref["logp"], b["adv"],
                          np.ones_like(pi), cu, si, sr)
    assert abs(out["loss"] + float(b["adv"].astype(np.float64).sum()) / w.B) < 1e-12


def test_gradient_matches_finite_differences():
    w, b = _tiny(old_noise=0.3, lengths=[5, 9, 4, 7, 6, 8, 3, 10],
                 rewards=[1, 0, 0, 1, 0, 1, 0, 0])
    mask, pi, _ = select(SEL_URS, b["cu_seqlens"], p=0.5, seed=2)
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    out = _run(b, mask, pi)
    assert (out["g"] != 0).sum() > 5 and (out["g"] == 0).sum() > 0   # both branches present

    def loss_at(H, W):
        return policy_loss_fwd(H, W, b["targets"], b["old_logp"], b["adv"], pi,
                               b["cu_seqlens"], si, sr)["loss"]

    rng = np.random.default_rng(0)
    H0 = b["hidden"].astype(np.float64)
    W0 = b["W"].astype(np.float64)
    step = 1e-6
    scale_h = np.abs(out["dH"]).max()
    scale_w = np.abs(out["dW"]).max()
    for _ in range(12):
        k = rng.integers(n)
        j = rng.integers(w.d)
        Hp, Hm = H0.copy(), H0.copy()
        Hp[si[k], j] += step
        Hm[si[k], j] -= step
        fd = (loss_at(Hp, W0) - loss_at(Hm, W0)) / (2 * step)
        assert abs(fd - out["dH"][k, j]) < 1e-6 * scale_h + 1e-9
    rows = list(rng.integers(w.V, size=6)) + [int(b["targets"][si[0]]), int(b["targets"][si[-1]])]
    for v in rows:
        j = rng.integers(w.d)
        Wp, Wm = W0.copy(), W0.copy()
        Wp[v, j] += step
        Wm[v, j] -= step
        fd = (loss_at(H0, Wp) - loss_at(H0, Wm)) / (2 * step)
        assert abs(fd - out["dW"][v, j]) < 1e-6 * scale_w + 1e-9
    # a token that is not selected receives no gradient: dH only has selected rows,
    # and a dloss scale passes straight through
    out2 = _run(b, mask, pi, dloss=-2.5)
    np.testing.assert_allclose(out2["dH"], -2.5 * out["dH"], rtol=1e-12, atol=1e-14 * scale_h)
    np.testing.assert_allclose(out2["dW"], -2.5 * out["dW"], rtol=1e-12, atol=1e-14 * scale_w)


def test_gradient_structure():
    w, b = _tiny(old_noise=0.3)
    mask, pi, _ = select(SEL_URS, b["cu_seqlens"], p=0.5, seed=0)
    out = _run(b, mask, pi)
    # sum_v dz[n, v] = 0  =>  every column of dW sums to zero over the vocabulary
    assert np.abs(out["dW"].sum(0)).max() < 1e-12 * np.abs(out["dW"]).sum(0).max() + 1e-18
    # Euler identity: sum_n <dH_n, h_n> = <dW, W> (both equal sum_{n,v} dz z)
    si = compact(mask, b["cu_seqlens"])[0]
    lhs = (out["dH"] * b["hidden"][si].astype(np.float64)).sum()
    rhs = (out["dW"] * b["W"].astype(np.float64)).sum()
    assert abs(lhs - rhs) < 1e-12 * (abs(lhs) + 1e-6)
    # dense + one-hot parts recombine
    y = b["targets"][si]
    oh = out["g"][:, None] * b["W"].astype(np.float64)[y]
    np.testing.assert_allclose(out["dH_dense"] + oh, out["dH"], rtol=1e-10, atol=1e-15)


def test_saturated_clip_has_zero_gradient():
    # outside the trust region on the pessimistic side the surrogate is flat
    w, b = _tiny()
    ones_mask = np.ones(b["n_tot"], dtype=np.uint8)
    ones_pi = np.ones(b["n_tot"], dtype=np.float32)
    ref = _run(b, ones_mask, ones_pi, want_dW=False)
    A = np.repeat(b["adv"], np.diff(b["cu_seqlens"])).astype(np.float64)
    old = ref["logp"] - np.where(A > 0, 0.5, -0.5)      # r = e^{0.5} if A>0, e^{-0.5} if A<0
    b2 = dict(b, old_logp=old)
    out = _run(b2, ones_mask, ones_pi)
    assert np.all(out["g"] == 0) and np.all(out["dH"] == 0) and np.all(out["dW"] == 0)
    r = np.where(A > 0, 1.2, 0.8)
    want = -np.sum(out["w"] * r * A * (A != 0))
    assert abs(out["loss"] - want) < 1e-12
    # on the other side (r small with A > 0, r large with A < 0) the gradient is live
    old = ref["logp"] + np.where(A > 0, 0.5, -0.5)
    out = _run(dict(b, old_logp=old), ones_mask, ones_pi, want_dW=False)
    assert np.all((out["g"] != 0) == (A != 0))


# ---- Proposition 1: the HT estimator's expectation is the full-token value ----
def _full(b):
    ones_mask = np.ones(b["n_tot"], dtype=np.uint8)
    ones_pi = np.ones(b["n_tot"], dtype=np.float32)
    return _run(b, ones_mask, ones_pi)


def _scatter_dH(out, si, n_tot, d):
    full = np.zeros((n_tot, d))
    full[si] = out["dH"]
    return full


def test_urs_enumeration_is_unbiased():
    """All 2^T masks of every response, weighted p^k (1-p)^(T-k).

    The loss is a sum over responses and masks are independent across
    responses, so the expectation is taken response by response (the other
    responses held at the full mask scaled by their own expectation = dropped
    here: each response's contribution is compared separately).
    """
    T = [6, 9, 4, 7, 5, 8, 3, 10]
    w, b = _tiny(old_noise=0.3, lengths=T, rewards=[1, 0, 0, 1, 0, 1, 0, 0])
    cu = b["cu_seqlens"]
    p = 0.5
    pi = np.full(b["n_tot"], np.float32(p))
    second_moment = 0.0
    for i in range(w.B):
        # contribution of response i alone under the full mask
        only = np.zeros(b["n_tot"], dtype=np.uint8)
        only[cu[i]:cu[i + 1]] = 1
        full = _run(b, only, np.ones_like(pi))
        full_dH = _scatter_dH(full, np.nonzero(only)[0], b["n_tot"], w.d)
        e_loss, e_dH, e_dW, e_m = 0.0, 0.0, 0.0, np.zeros(T[i])
        for bits in itertools.product((0, 1), repeat=T[i]):
            k = sum(bits)
            pr = p ** k * (1 - p) ** (T[i] - k)
            m = np.zeros(b["n_tot"], dtype=np.uint8)
            m[cu[i]:cu[i + 1]] = bits
            e_m += pr * np.array(bits) / p
            if k == 0:
                continue
            out = _run(b, m, pi)
            e_loss += pr * out["loss"]
            e_dH = e_dH + pr * _scatter_dH(out, np.nonzero(m)[0], b["n_tot"], w.d)
            e_dW = e_dW + pr * out["dW"]
            if i == 0:
                second_moment += pr * (out["dW"] ** 2).sum()
        np.testing.assert_allclose(e_m, 1.0, rtol=1e-12)               # E[m/p] = 1
        assert abs(e_loss - full["loss"]) < 1e-12
        np.testing.assert_allclose(e_dH, full_dH, atol=1e-13 * np.abs(full_dH).max() + 1e-18)
        np.testing.assert_allclose(e_dW, full["dW"], atol=1e-12 * np.abs(full["dW"]).max())
        if i == 0:
            # independent masking: E||g_hat||^2 = ||g||^2 + sum_t (1-p)/p ||g_t||^2
            per_tok = 0.0
            for n in range(cu[0], cu[1]):
                one = np.zeros(b["n_tot"], dtype=np.uint8)
                one[n] = 1
                per_tok += (_run(b, one, np.ones_like(pi))["dW"] ** 2).sum()
            want = (full["dW"] ** 2).sum() + (1 - p) / p * per_tok
            assert abs(second_moment - want) < 1e-10 * want


def test_rpc_enumeration_is_unbiased_and_det_is_biased():
    w, b = _tiny(old_noise=0.3)
    cu = b["cu_seqlens"]
    for C in (1, 5):
        _, pi, _ = select(SEL_RPC, cu, min_cut=C, seed=0)
        for i in range(w.B):
            T = cu[i + 1] - cu[i]
            Ci = min(C, T)
            n_cuts = T - Ci + 1
            only = np.zeros(b["n_tot"], dtype=np.uint8)
            only[cu[i]:cu[i + 1]] = 1
            full = _run(b, only, np.ones_like(pi))
            e_loss, e_dW, e_dH = 0.0, 0.0, 0.0
            losses = []
            for L in range(Ci, T + 1):
                m = np.zeros(b["n_tot"], dtype=np.uint8)
                m[cu[i]:cu[i] + L] = 1
                out = _run(b, m, pi)
                losses.append(out["loss"])
                e_loss += out["loss"] / n_cuts
                e_dW = e_dW + out["dW"] / n_cuts
                e_dH = e_dH + _scatter_dH(out, np.nonzero(m)[0], b["n_tot"], w.d) / n_cuts
            scale = np.abs(full["dW"]).max()
            assert abs(e_loss - full["loss"]) < 2e-7 * abs(full["loss"]) + 1e-9   # pi is float32
            np.testing.assert_allclose(e_dW, full["dW"], atol=2e-7 * scale)
            full_dH = _scatter_dH(full, np.nonzero(only)[0], b["n_tot"], w.d)
            np.testing.assert_allclose(e_dH, full_dH, atol=2e-7 * np.abs(full_dH).max())
            # Variance in stopping-time form (Eq. rpc-variance-stopping, Appendix B.1),
            # evaluated from the per-token losses L_t of the full-token run and the
            # survival probabilities, not from the estimator's own realisations:
            #   Var[mu_hat] = (E[(sum_{t<=tau} L_t/p_t)^2] - (sum_t L_t)^2) / T^2,
            # tau uniform on {C..T}.  The loss of a batch whose mask covers response i
            # only is -mu_hat_i / B.
            Lt = full["L"]                                     # per-token losses, t = 1..T
            pt = pi[cu[i]:cu[i + 1]].astype(np.float64)
            partial = np.cumsum(Lt / pt)                       # sum_{t<=tau} L_t / p_t
            second = np.mean(partial[Ci - 1:] ** 2)            # E over tau = C..T
            var_formula = (second - Lt.sum() ** 2) / T ** 2 / w.B ** 2
            var_direct = np.mean((np.array(losses) - np.mean(losses)) ** 2)
            assert abs(var_direct - var_formula) < 2e-6 * abs(var_formula) + 1e-18
    # deterministic truncation: the "expectation" is the single realisation, and it
    # misses exactly the dropped suffix
    mask, pi, cut = select(SEL_DET, cu, beta=0.5)
    out = _run(b, mask, pi)
    full = _full(b)
    dropped = _run(b, 1 - mask, pi)
    assert abs((full["loss"] - out["loss"]) - dropped["loss"]) < 1e-12
    np.testing.assert_allclose(full["dW"] - out["dW"], dropped["dW"], atol=1e-14)
    assert np.abs(dropped["dW"]).max() > 1e-6                 # the bias is not small


def test_rpc_mask_covariance():
    # Cov(m_s, m_t) = p_t (1 - p_s) for s <= t, over all cuts of the uniform law
    T, C = 12, 3
    n = T - C + 1
    M = np.array([[1.0 if t <= L else 0.0 for t in range(1, T + 1)] for L in range(C, T + 1)])
    p = M.mean(0)
    _, pi, _ = select(SEL_RPC, np.array([0, T], dtype=np.int32), min_cut=C)
    np.testing.assert_allclose(pi, p, rtol=1e-7)
    cov = (M.T @ M) / n - np.outer(p, p)
    for s in range(T):
        for t in range(s, T):
            assert abs(cov[s, t] - p[t] * (1 - p[s])) < 1e-12


# ---- optional KL term (Eq. grpo-token-loss, sampled-token form of its footnote) ----
def test_kl_term_closed_form_and_gradient():
    w, b = _tiny(old_noise=0.3, lengths=[5, 9, 4, 7, 6, 8, 3, 10], rewards=[1, 0, 0, 1, 0, 1, 0, 0])
    mask, pi, _ = select(SEL_URS, b["cu_seqlens"], p=0.5, seed=2)
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    rng = np.random.default_rng(3)
    ref_logp = b["old_logp"].astype(np.float64) + rng.normal(0, 0.1, b["n_tot"])
    beta = 0.05
    base = _run(b, mask, pi)
    out = _run(b, mask, pi, kl_beta=beta, ref_logp=ref_logp)
    # loss differs from the beta = 0 loss by + beta * sum_n w_n (logp_n - ref_n)
    want = base["loss"] + beta * np.sum(base["w"] * (base["logp"] - ref_logp[si]))
    assert abs(out["loss"] - want) < 1e-12
    # with ref_logp equal to the current logp the penalty vanishes but its gradient does not
    ref_same = b["old_logp"].astype(np.float64).copy()
    ref_same[si] = base["logp"]
    same = _run(b, mask, pi, kl_beta=beta, ref_logp=ref_same)
    assert abs(same["loss"] - base["loss"]) < 1e-12
    np.testing.assert_allclose(same["g"] - base["g"], beta * base["w"], rtol=1e-12)

    # finite differences of the full loss
    def loss_at(H, W):
        return policy_loss_fwd(H, W, b["targets"], b["old_logp"], b["adv"], pi, b["cu_seqlens"],
                               si, sr, kl_beta=beta, ref_logp=ref_logp)["loss"]
    H0 = b["hidden"].astype(np.float64)
    W0 = b["W"].astype(np.float64)
    step = 1e-6
    for _ in range(8):
        k, j, v = rng.integers(n), rng.integers(w.d), rng.integers(w.V)
        Hp, Hm = H0.copy(), H0.copy()
        Hp[si[k], j] += step
        Hm[si[k], j] -= step
        fd = (loss_at(Hp, W0) - loss_at(Hm, W0)) / (2 * step)
        assert abs(fd - out["dH"][k, j]) < 1e-6 * np.abs(out["dH"]).max() + 1e-9
        Wp, Wm = W0.copy(), W0.copy()
        Wp[v, j] += step
        Wm[v, j] -= step
        fd = (loss_at(H0, Wp) - loss_at(H0, Wm)) / (2 * step)
        assert abs(fd - out["dW"][v, j]) < 1e-6 * np.abs(out["dW"]).max() + 1e-9


def test_general_cut_law_enumeration_is_unbiased():
    """Eq. rpc-survival with a non-uniform q: cuts weighted q(l) = p_l - p_{l+1} give the
    full-token loss and gradient in expectation when pi = p (Proposition 1)."""
    w, b = _tiny(old_noise=0.3, lengths=[6, 9, 5, 7, 4, 8, 3, 10], rewards=[1, 0, 0, 1, 0, 1, 0, 0])
    cu = b["cu_seqlens"]
    surv = np.concatenate([np.maximum(0.8 ** np.arange(T), 0.1) for T in np.diff(cu)])
    surv[cu[:-1]] = 1.0
    pi = surv.astype(np.float32)
    for i in range(w.B):
        T = cu[i + 1] - cu[i]
        p = pi[cu[i]:cu[i + 1]].astype(np.float64)
        q = p - np.append(p[1:], 0.0)                 # Pr(L = l), l = 1..T
        assert abs(q.sum() - 1.0) < 1e-12 and np.all(q >= 0)
        only = np.zeros(b["n_tot"], dtype=np.uint8)
        only[cu[i]:cu[i + 1]] = 1
        full = _run(b, only, np.ones_like(pi))
        e_loss, e_dW = 0.0, 0.0
        for L in range(1, T + 1):
            if q[L - 1] == 0:
                continue
            m = np.zeros(b["n_tot"], dtype=np.uint8)
            m[cu[i]:cu[i] + L] = 1
            out = _run(b, m, pi)
            e_loss += q[L - 1] * out["loss"]
            e_dW = e_dW + q[L - 1] * out["dW"]
        assert abs(e_loss - full["loss"]) < 2e-7 * abs(full["loss"]) + 1e-9
        np.testing.assert_allclose(e_dW, full["dW"], atol=2e-7 * np.abs(full["dW"]).max())


def test_cutlaw_enumeration_is_unbiased():
    """Proposition 1 under a non-uniform cut law given as masses q(l): weighting every cut by
    its probability k_l / S_1 and using select_cutlaw's pi gives the full-token loss and dW."""
    from oracle import cutlaw_counts
    w, b = _tiny(old_noise=0.3, lengths=[6, 9, 5, 7, 4, 8, 3, 10], rewards=[1, 0, 0, 1, 0, 1, 0, 0])
    cu = b["cu_seqlens"]
    q = np.concatenate([0.85 ** np.arange(T) + 0.05 for T in np.diff(cu)]).astype(np.float32) / 16
    _, pi, _ = select_cutlaw(cu, q, seed=0)
    k = cutlaw_counts(q)
    for i in range(w.B):
        T = cu[i + 1] - cu[i]
        kk = k[cu[i]:cu[i + 1]].astype(np.float64)
        prob = kk / kk.sum()                          # Pr(L = l), l = 1..T
        only = np.zeros(b["n_tot"], dtype=np.uint8)
        only[cu[i]:cu[i + 1]] = 1
        full = _run(b, only, np.ones_like(pi))
        e_loss, e_dW = 0.0, 0.0
        for L in range(1, T + 1):
            m = np.zeros(b["n_tot"], dtype=np.uint8)
            m[cu[i]:cu[i] + L] = 1
            out = _run(b, m, pi)
            e_loss += prob[L - 1] * out["loss"]
            e_dW = e_dW + prob[L - 1] * out["dW"]
        assert abs(e_loss - full["loss"]) < 2e-7 * abs(full["loss"]) + 1e-9
        np.testing.assert_allclose(e_dW, full["dW"], atol=2e-7 * np.abs(full["dW"]).max())


def test_dW_rows_match_full_dW_and_finite_differences():
    w, b = _tiny(old_noise=0.3)
    mask, pi, _ = select(SEL_URS, b["cu_seqlens"], p=0.5, seed=4)
    si, sr, so, n = compact(mask, b["cu_seqlens"])
    full = _run(b, mask, pi)
    y = b["targets"][si]
    v_ids = np.array([0, int(y[0]), int(y[n // 2]), 17, w.V - 1])
    A = b["adv"].astype(np.float64)[sr]
    g = grad_coeff(full["ratio"], A, full["w"], 0.2, 0.2)
    H = b["hidden"][si]
    blocks = [H[lo:lo + 37] for lo in range(0, n, 37)]          # streamed in ragged blocks
    rows, dense = policy_loss_dW_rows(blocks, b["W"][v_ids], v_ids, y, g, full["lse"])
    np.testing.assert_allclose(rows, full["dW"][v_ids], atol=1e-15 + 1e-12 * np.abs(full["dW"]).max())
    np.testing.assert_allclose(dense, full["dW_dense"][v_ids],
                               atol=1e-15 + 1e-12 * np.abs(full["dW_dense"]).max())
    assert np.abs(rows - dense).max() > 0                       # target rows are in the sample

    def loss_at(W):
        return policy_loss_fwd(b["hidden"], W, b["targets"], b["old_logp"], b["adv"], pi,
                               b["cu_seqlens"], si, sr)["loss"]
    W0 = b["W"].astype(np.float64)
    step = 1e-6
    rng = np.random.default_rng(0)
    for r, v in enumerate(v_ids):
        j = int(rng.integers(w.d))
        Wp, Wm = W0.copy(), W0.copy()
        Wp[v, j] += step
        Wm[v, j] -= step
        fd = (loss_at(Wp) - loss_at(Wm)) / (2 * step)
        assert abs(fd - rows[r, j]) < 1e-6 * np.abs(full["dW"]).max() + 1e-10
