"""fp64 oracle of the partial-token GRPO policy-gradient step (NAT).

TEST INFRASTRUCTURE ONLY: plain numpy, written from the paper's definitions,
independent of the CUDA library (no shared code, tables or helpers).  Every
function names the passage it follows.  Notation is the paper's: B = P*G
responses, response i has length T_i, packed token n belongs to response
resp(n) at 1-based position t; m is the mask, p (here ``pi``) the inclusion
probability, L_i the RPC cut, A_i the group-relative advantage.

Readings where the paper is silent (the CUDA library takes the same ones):
  * loss = -J (the paper maximises J, Section 2.2 sequence-level aggregation).
  * the batch mean runs over all B = P*G responses; each response keeps its
    FULL length T_i in the 1/T_i normaliser (Eq. ht-estimator, Eq. rpc-ht).
  * random draws come from Philox4x32-10 keyed by (seed, offset, response,
    position); see ``select``.
  * a clip bound is inclusive: a ratio exactly on the bound still has gradient.
"""
import math

import numpy as np

from .philox import philox4x32_10

SEL_URS = 0  # Uniform Random Sampling, Section 3.1
SEL_RPC = 1  # Random Prefix Cutting with minimum cut C, Section 4
SEL_DET = 2  # deterministic prefix truncation (the biased comparison), Section 4


# --------------------------------------------------------------------------
# Group-relative advantage, Eq. grpo-adv
# --------------------------------------------------------------------------
def grpo_adv(rewards, P, G, eps):
    """A_i = (R_i - mu) / (sigma + eps) inside each group of G responses.

    mu and sigma are the population mean and standard deviation (1/G) of the
    group's rewards.  Arithmetic is double, sums taken in index order, result
    rounded once to float32.
    """
    rewards = np.asarray(rewards, dtype=np.float32)
    assert rewards.shape == (P * G,)
    adv = np.zeros(P * G, dtype=np.float32)
    for g in range(P):
        R = [float(rewards[g * G + j]) for j in range(G)]
        s = 0.0
        for r in R:
            s = s + r
        mu = s / G
        v = 0.0
        for r in R:
            dlt = r - mu
            v = v + dlt * dlt
        sigma = math.sqrt(v / G)
        for j in range(G):
            adv[g * G + j] = np.float32((R[j] - mu) / (sigma + float(eps)))
    return adv


# --------------------------------------------------------------------------
# Token selection: URS (Section 3.1), RPC (Eq. rpc-mask, Eq. rpc-survival with
# the uniform / minimum-cutoff law), deterministic truncation
# --------------------------------------------------------------------------
def _key(seed, offset):
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    offset = int(offset) & 0xFFFFFFFFFFFFFFFF
    k0 = seed & 0xFFFFFFFF
    k1 = ((seed >> 32) ^ (offset >> 32)) & 0xFFFFFFFF
    return k0, k1, offset & 0xFFFFFFFF


def urs_threshold(p):
    """Integer threshold thr so that a 32-bit draw x is kept iff x < thr.

    thr = floor(p * 2^32) clamped to [1, 2^32]; the realised inclusion
    probability is exactly thr / 2^32.
    """
    if not (0.0 < p <= 1.0):
        raise ValueError("URS needs 0 < p <= 1")
    thr = int(math.floor(p * 4294967296.0))
    return min(max(thr, 1), 1 << 32)


def select(mode, cu_seqlens, *, p=1.0, min_cut=1, beta=1.0, seed=0, offset=0, resp_base=0):
    """Draw the mask m, the inclusion probabilities pi and the per-response cut.

    Returns (mask uint8 [N_tot], pi float32 [N_tot], cut_len int32 [B] or None).

    ``resp_base`` is the index, in the whole job's batch, of the first response of
    ``cu_seqlens``: the draws of local response i are those of response resp_base + i, so a
    shard of a batch realises the same mask as the whole batch does for those responses
    (masks of different responses are independent, Section 3.1).

    URS: token t of response i consumes word (t-1) mod 4 of the Philox block
    with counter ((t-1) div 4, i, 0, offset_lo); m = [x < thr], pi = thr/2^32.

    RPC: response i draws one block with counter (0, i, 1, offset_lo), forms
    u = x1*2^32 + x0 and L_i = C_i + floor(u * n / 2^64) with
    C_i = min(max(C, 1), T_i), n = T_i - C_i + 1, so L_i is uniform on
    {C_i..T_i}; m_t = [t <= L_i]; pi_t = 1 for t <= C_i and
    (T_i - t + 1) / (T_i - C_i + 1) afterwards (one float32 division).

    DET: K_i = max(1, floor(beta * T_i)), m_t = [t <= K_i], pi_t = 1.
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = cu.shape[0] - 1
    n_tot = int(cu[B])
    mask = np.zeros(n_tot, dtype=np.uint8)
    pi = np.zeros(n_tot, dtype=np.float32)
    k0, k1, off_lo = _key(seed, offset)
    if mode == SEL_URS:
        thr = urs_threshold(p)
        pi_val = np.float32(thr / 4294967296.0)
        for i in range(B):
            T = int(cu[i + 1] - cu[i])
            if T == 0:
                continue
            t0 = np.arange(T, dtype=np.uint64)          # t - 1
            words = philox4x32_10(t0 >> np.uint64(2), resp_base + i, 0, off_lo, k0, k1)
            x = np.choose((t0 & np.uint64(3)).astype(np.int64), words)
            mask[cu[i]:cu[i + 1]] = (x < np.uint64(thr)).astype(np.uint8)
            pi[cu[i]:cu[i + 1]] = pi_val
        return mask, pi, None
    cut_len = np.zeros(B, dtype=np.int32)
    for i in range(B):
        T = int(cu[i + 1] - cu[i])
        if T == 0:
            continue
        t = np.arange(1, T + 1, dtype=np.int64)
        if mode == SEL_RPC:
            C = min(max(int(min_cut), 1), T)
            n = T - C + 1
            x0, x1, _, _ = philox4x32_10(0, resp_base + i, 1, off_lo, k0, k1)
            u = (int(x1) << 32) | int(x0)
            L = C + ((u * n) >> 64)
            num = (T - t + 1).astype(np.float32)
            den = np.float32(n)
            surv = num / den                            # float32 IEEE division
            pi[cu[i]:cu[i + 1]] = np.where(t <= C, np.float32(1.0), surv)
        elif mode == SEL_DET:
            if not (0.0 < beta <= 1.0):
                raise ValueError("DET needs 0 < beta <= 1")
            L = max(1, int(math.floor(float(beta) * T)))
            pi[cu[i]:cu[i + 1]] = np.float32(1.0)
        else:
            raise ValueError("unknown selection mode")
        cut_len[i] = L
        mask[cu[i]:cu[i + 1]] = (t <= L).astype(np.uint8)
    return mask, pi, cut_len


def select_survival(cu_seqlens, surv, *, seed=0, offset=0, resp_base=0):
    """Random Prefix Cutting under a caller-given survival schedule (Eq. rpc-mask,
    Eq. rpc-survival with a general cut law q_i).

    ``surv[n]`` is p_{i,t} = Pr(L_i >= t) for packed token n: non-increasing inside a
    response, 1 at its first token, positive at its last.  Response i draws one uniform
    u = (x0 >> 8) * 2^-24 from the Philox block with counter (0, i, 2, offset_lo); then
    L_i >= t  <=>  u < p_{i,t}, so m_t = [u < surv[n]] (a prefix because surv is monotone)
    and Pr(L_i >= t) = ceil(p_{i,t} 2^24) / 2^24, within 2^-24 of the schedule.
    The inclusion probabilities are the schedule itself.  ``resp_base`` as in ``select``.

    Returns (mask uint8 [N_tot], cut_len int32 [B]).
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    surv = np.asarray(surv, dtype=np.float32)
    B = cu.shape[0] - 1
    mask = np.zeros(int(cu[B]), dtype=np.uint8)
    cut_len = np.zeros(B, dtype=np.int32)
    k0, k1, off_lo = _key(seed, offset)
    for i in range(B):
        lo, hi = int(cu[i]), int(cu[i + 1])
        if hi == lo:
            continue
        p = surv[lo:hi]
        if p[0] != 1.0 or np.any(np.diff(p) > 0) or p[-1] <= 0:
            raise ValueError("survival schedule must start at 1, not increase and stay positive")
        x0, _, _, _ = philox4x32_10(0, resp_base + i, 2, off_lo, k0, k1)
        u = np.float32(int(x0) >> 8) * np.float32(2.0 ** -24)
        m = u < p
        mask[lo:hi] = m.astype(np.uint8)
        cut_len[i] = int(m.sum())
    return mask, cut_len


def cutlaw_counts(q):
    """Cut-law masses in 32-bit fixed point: k = min(floor(q * 2^32), 2^32 - 1) for q > 0,
    else 0 (a negative or NaN mass counts as zero).

    The scaling by a power of two and the floor are exact, so the counts (and every sum of
    them, taken in 64-bit integers) do not depend on the order of evaluation.
    """
    q = np.asarray(q, dtype=np.float32)
    k = np.zeros(q.shape, dtype=np.uint64)
    pos = q > 0
    scaled = np.floor(q[pos].astype(np.float64) * 4294967296.0)
    k[pos] = np.minimum(scaled, 4294967295.0).astype(np.uint64)
    return k


def select_cutlaw(cu_seqlens, q, *, seed=0, offset=0, resp_base=0):
    """Random Prefix Cutting under a caller-given cut law q_i (Eq. rpc-mask, Eq. rpc-survival).

    ``q[n]`` is the (unnormalised) mass the cut law of token n's response puts on cutting
    right after that token, q_i(l) up to a common factor per response.  With the fixed-point
    counts k of ``cutlaw_counts``:
        S_t  = sum_{l >= t} k_l                 (Eq. rpc-survival's suffix sum, exact integers)
        u    = x1 2^32 + x0 from the Philox block with counter (0, resp_base + i, 3, offset_lo)
        r    = floor(u S_1 / 2^64)              uniform on {0 .. S_1 - 1} to within S_1 2^-64
        m_t  = [S_t > r]                        i.e. L_i = max{t : S_t > r}, Pr(L_i >= t) = S_t / S_1
        pi_t = float32(double(S_t) * (1 / double(S_1)))   (the reciprocal once per response;
               every operation IEEE round-to-nearest)
    so pi_1 = 1, pi never increases, and pi_t > 0 wherever the law still has mass at or
    after t.
    A response whose counts are all zero is kept whole with pi = 1.

    Returns (mask uint8 [N_tot], pi float32 [N_tot], cut_len int32 [B]).
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = cu.shape[0] - 1
    n_tot = int(cu[B])
    k = cutlaw_counts(q)
    assert k.shape == (n_tot,)
    mask = np.zeros(n_tot, dtype=np.uint8)
    pi = np.zeros(n_tot, dtype=np.float32)
    cut_len = np.zeros(B, dtype=np.int32)
    k0, k1, off_lo = _key(seed, offset)
    for i in range(B):
        lo, hi = int(cu[i]), int(cu[i + 1])
        if hi == lo:
            continue
        S = [0] * (hi - lo)                         # Python integers: exact
        run = 0
        for t in range(hi - lo - 1, -1, -1):
            run += int(k[lo + t])
            S[t] = run
        total = S[0]
        if total == 0:
            mask[lo:hi] = 1
            pi[lo:hi] = np.float32(1.0)
            cut_len[i] = hi - lo
            continue
        x0, x1, _, _ = philox4x32_10(0, resp_base + i, 3, off_lo, k0, k1)
        u = (int(x1) << 32) | int(x0)
        r = (u * total) >> 64
        S64 = np.array(S, dtype=np.uint64)
        mask[lo:hi] = (S64 > np.uint64(r)).astype(np.uint8)
        inv_total = np.float64(1.0) / np.float64(np.uint64(total))
        pi[lo:hi] = (S64.astype(np.float64) * inv_total).astype(np.float32)
        cut_len[i] = int(mask[lo:hi].sum())
    return mask, pi, cut_len


# --------------------------------------------------------------------------
# Compaction of the selected token indices
# --------------------------------------------------------------------------
def compact(mask, cu_seqlens):
    """Ascending indices of the kept tokens, their responses, per-response
    offsets into that list, and the count.

    Returns (sel_idx int32 [n_sel], sel_resp int32 [n_sel],
             sel_offsets int32 [B+1], n_sel int).
    """
    mask = np.asarray(mask)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = cu.shape[0] - 1
    sel_idx = []
    sel_resp = []
    sel_offsets = np.zeros(B + 1, dtype=np.int32)
    for i in range(B):
        sel_offsets[i] = len(sel_idx)
        for n in range(int(cu[i]), int(cu[i + 1])):
            if mask[n] != 0:
                sel_idx.append(n)
                sel_resp.append(i)
    sel_offsets[B] = len(sel_idx)
    return (np.asarray(sel_idx, dtype=np.int32), np.asarray(sel_resp, dtype=np.int32),
            sel_offsets, len(sel_idx))


# --------------------------------------------------------------------------
# Packing for prefix-truncated computation (Section 4, "Compute savings": under
# RPC the model only processes the prefix 1..L_i of each response)
# --------------------------------------------------------------------------
def gather_rows(src, sel_idx):
    """Compact copy: row k of the result is row sel_idx[k] of ``src``."""
    src = np.asarray(src)
    out = np.zeros((len(sel_idx),) + src.shape[1:], dtype=src.dtype)
    for k, n in enumerate(sel_idx):
        out[k] = src[int(n)]
    return out


def scatter_rows(src, sel_idx, n_tot):
    """Inverse placement: row sel_idx[k] of the result is row k of ``src``; every other
    row is zero (a token that was not selected receives no gradient)."""
    src = np.asarray(src)
    out = np.zeros((int(n_tot),) + src.shape[1:], dtype=src.dtype)
    for k, n in enumerate(sel_idx):
        out[int(n)] = src[k]
    return out


# --------------------------------------------------------------------------
# Policy loss over the selected tokens: forward
#   ratio Eq. ratio, surrogate Eq. grpo-surrogate, aggregation Eq. grpo-obj,
#   Horvitz-Thompson weights Eq. ht-estimator / Eq. rpc-ht
# --------------------------------------------------------------------------
_ROW_BATCH = 256  # rows evaluated per matmul call; rows are independent


def _rows(hidden, sel_idx, hidden_is_compact, lo, hi):
    if hidden_is_compact:
        return np.asarray(hidden[lo:hi], dtype=np.float64)
    return np.asarray(hidden[np.asarray(sel_idx[lo:hi], dtype=np.int64)], dtype=np.float64)


def _token_weights(pi, cu_seqlens, sel_idx, sel_resp):
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    B = cu.shape[0] - 1
    T = (cu[1:] - cu[:-1]).astype(np.float64)
    sel_idx = np.asarray(sel_idx, dtype=np.int64)
    sel_resp = np.asarray(sel_resp, dtype=np.int64)
    pin = np.asarray(pi, dtype=np.float64)[sel_idx]
    return 1.0 / (pin * T[sel_resp] * float(B))          # w_n = 1 / (pi_n T_i B)


def policy_loss_fwd(hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx, sel_resp,
                    clip_lo=0.2, clip_hi=0.2, hidden_is_compact=False, kl_beta=0.0,
                    ref_logp=None):
    """Loss and per-token statistics over the selected tokens.

    For selected token n (row h_n of ``hidden``):
        z      = W h_n                      (V logits)
        lse    = log sum_v exp(z_v)
        logp   = z[y_n] - lse
        r      = exp(logp - old_logp[n])
        S      = min(r A, clip(r, 1-clip_lo, 1+clip_hi) A),  A = adv[resp(n)]
        w      = 1 / (pi[n] * T_resp(n) * B)
        L      = S - kl_beta * (logp - ref_logp[n])     (Eq. grpo-token-loss with the
                 per-token KL taken in the sampled-token form of its footnote;
                 kl_beta = 0, the paper's experimental setting, drops it)
        loss   = - sum_n w L

    ``hidden`` is [N_tot, d] (rows picked by sel_idx) or, with
    hidden_is_compact, [n_sel, d] with row k belonging to sel_idx[k].
    Returns a dict: loss (float), logp, lse, ratio, S, w (float64 [n_sel]).
    """
    W64 = np.asarray(W, dtype=np.float64)
    sel_idx = np.asarray(sel_idx, dtype=np.int64)
    sel_resp = np.asarray(sel_resp, dtype=np.int64)
    n_sel = sel_idx.shape[0]
    y = np.asarray(targets, dtype=np.int64)[sel_idx]
    old = np.asarray(old_logp, dtype=np.float64)[sel_idx]
    A = np.asarray(adv, dtype=np.float64)[sel_resp]
    w = _token_weights(pi, cu_seqlens, sel_idx, sel_resp)
    lse = np.zeros(n_sel)
    logp = np.zeros(n_sel)
    for lo in range(0, n_sel, _ROW_BATCH):
        hi = min(lo + _ROW_BATCH, n_sel)
        z = _rows(hidden, sel_idx, hidden_is_compact, lo, hi) @ W64.T
        M = z.max(axis=1)
        lse[lo:hi] = M + np.log(np.exp(z - M[:, None]).sum(axis=1))
        logp[lo:hi] = z[np.arange(hi - lo), y[lo:hi]] - lse[lo:hi]
    ratio = np.exp(logp - old)
    clipped = np.minimum(np.maximum(ratio, 1.0 - clip_lo), 1.0 + clip_hi)
    S = np.minimum(ratio * A, clipped * A)
    L = S
    if kl_beta != 0.0:
        ref = np.asarray(ref_logp, dtype=np.float64)[sel_idx]
        L = S - float(kl_beta) * (logp - ref)
    loss = -float(np.sum(w * L))
    return dict(loss=loss, logp=logp, lse=lse, ratio=ratio, S=S, w=w, L=L)


# --------------------------------------------------------------------------
# Policy loss over the selected tokens: backward
# --------------------------------------------------------------------------
def grad_coeff(ratio, A, w, clip_lo, clip_hi, dloss=1.0, kl_beta=0.0):
    """g_n = d loss / d logp_n.

    The min in the surrogate picks r*A (which has gradient A*r w.r.t. logp)
    unless the clipped branch is the smaller one: A > 0 and r > 1+clip_hi, or
    A < 0 and r < 1-clip_lo, where the surrogate is flat.  A = 0 gives zero.
    """
    active = ((A > 0) & (ratio <= 1.0 + clip_hi)) | ((A < 0) & (ratio >= 1.0 - clip_lo))
    # the KL term -kl_beta (logp - ref_logp) has derivative -kl_beta w.r.t. logp
    return np.where(active, -dloss * w * A * ratio, 0.0) + dloss * w * float(kl_beta)


def policy_loss_bwd(hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx, sel_resp,
                    clip_lo=0.2, clip_hi=0.2, hidden_is_compact=False, dloss=1.0,
                    want_dW=True, kl_beta=0.0, ref_logp=None):
    """Gradients of ``policy_loss_fwd``'s loss.

        dz[n, v]  = g_n (1[v = y_n] - softmax(z_n)[v])
        dH[n, :]  = sum_v dz[n, v] W[v, :]        (compact: row k <-> sel_idx[k])
        dW[v, :]  = sum_n dz[n, v] h_n

    Returns a dict: dH float64 [n_sel, d], dW float64 [V, d] (None unless
    want_dW), g float64 [n_sel], and the dense (softmax-only) parts dH_dense,
    dW_dense that exclude the one-hot target terms.
    """
    fwd = policy_loss_fwd(hidden, W, targets, old_logp, adv, pi, cu_seqlens, sel_idx, sel_resp,
                          clip_lo, clip_hi, hidden_is_compact, kl_beta, ref_logp)
    W64 = np.asarray(W, dtype=np.float64)
    V, d = W64.shape
    sel_idx = np.asarray(sel_idx, dtype=np.int64)
    sel_resp = np.asarray(sel_resp, dtype=np.int64)
    n_sel = sel_idx.shape[0]
    y = np.asarray(targets, dtype=np.int64)[sel_idx]
    A = np.asarray(adv, dtype=np.float64)[sel_resp]
    g = grad_coeff(fwd["ratio"], A, fwd["w"], clip_lo, clip_hi, dloss, kl_beta)
    dH = np.zeros((n_sel, d))
    dH_dense = np.zeros((n_sel, d))
    dW = np.zeros((V, d)) if want_dW else None
    dW_dense = np.zeros((V, d)) if want_dW else None
    for lo in range(0, n_sel, _ROW_BATCH):
        hi = min(lo + _ROW_BATCH, n_sel)
        h = _rows(hidden, sel_idx, hidden_is_compact, lo, hi)
        z = h @ W64.T
        prob = np.exp(z - fwd["lse"][lo:hi, None])
        dz_dense = -g[lo:hi, None] * prob
        dz = dz_dense.copy()
        dz[np.arange(hi - lo), y[lo:hi]] += g[lo:hi]
        dH[lo:hi] = dz @ W64
        dH_dense[lo:hi] = dz_dense @ W64
        if want_dW:
            dW += dz.T @ h
            dW_dense += dz_dense.T @ h
    out = dict(fwd)
    out.update(dH=dH, dW=dW, g=g, dH_dense=dH_dense, dW_dense=dW_dense)
    return out


def policy_loss_dW_rows(hidden_blocks, W_rows, v_ids, y, g, lse):
    """Rows ``v_ids`` of dW, summed over ALL selected tokens, from per-token scalars.

        dW[v, :] = sum_n g_n (1[v = y_n] - exp(W_v . h_n - lse_n)) h_n

    which is ``policy_loss_bwd``'s dW restricted to a few vocabulary rows: the softmax
    probability of entry v needs only W_v, h_n and the row's lse_n.  ``hidden_blocks``
    yields the selected rows in order as consecutive arrays [rows, d] (so a caller can
    stream them), ``W_rows`` is W[v_ids] (float [len(v_ids), d]), ``y`` the selected tokens'
    targets, ``g`` their gradient coefficients (``grad_coeff``) and ``lse`` their
    log-sum-exp, all [n_sel].

    Returns (dW_rows, dW_rows_dense) float64 [len(v_ids), d]; the second leaves out the
    one-hot target term.
    """
    Wv = np.asarray(W_rows, dtype=np.float64)
    v_ids = np.asarray(v_ids, dtype=np.int64)
    y = np.asarray(y, dtype=np.int64)
    g = np.asarray(g, dtype=np.float64)
    lse = np.asarray(lse, dtype=np.float64)
    out = np.zeros(Wv.shape)
    dense = np.zeros(Wv.shape)
    lo = 0
    for blk in hidden_blocks:
        h = np.asarray(blk, dtype=np.float64)
        hi = lo + h.shape[0]
        z = h @ Wv.T                                         # [rows, len(v_ids)]
        dz_dense = -g[lo:hi, None] * np.exp(z - lse[lo:hi, None])
        hit = (y[lo:hi, None] == v_ids[None, :])
        dz = dz_dense + np.where(hit, g[lo:hi, None], 0.0)
        out += dz.T @ h
        dense += dz_dense.T @ h
        lo = hi
    assert lo == y.shape[0]
    return out, dense
