"""GPU parity: advantages, selection and compaction are bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_06619_b200 import nat
from paper_2603_06619_b200 import workloads as wl
from paper_2603_06619_b200.step import NatStep

from parity import MODE_ID

pytestmark = pytest.mark.gpu


def _select_compact(T, mode, P, G, seed=0, offset=0, p=0.5, min_cut=1, beta=0.5, cap=None,
                    rewards=None):
    T = np.asarray(T, dtype=np.int32)
    cu = wl.cu_from_lengths(T)
    n_tot = int(cu[-1])
    st = NatStep(P, G, 64, 512, torch.float32, n_tot, n_sel_cap=cap, want_grads=False)
    cu_d = torch.from_numpy(cu).cuda()
    if rewards is None:
        rewards = (np.random.default_rng(seed).random(P * G) < 0.4).astype(np.float32)
    st.grpo_adv(torch.from_numpy(rewards).cuda())
    st.select(cu_d, mode, p=p, min_cut=min_cut, beta=beta, seed=seed, offset=offset)
    for t in (st.sel_idx, st.sel_resp, st.sel_offsets, st.n_sel):
        t.fill_(-9)
    st.compact(cu_d)
    torch.cuda.synchronize()
    adv = oracle.grpo_adv(rewards, P, G, 1e-6)
    mask, pi, cut = oracle.select(MODE_ID[mode], cu, p=p, min_cut=min_cut, beta=beta, seed=seed,
                                  offset=offset)
    si, sr, so, n = oracle.compact(mask, cu)
    assert np.array_equal(st.adv.cpu().numpy().view(np.uint32), adv.view(np.uint32))
    assert np.array_equal(st.mask[:n_tot].cpu().numpy(), mask)
    assert np.array_equal(st.pi[:n_tot].cpu().numpy().view(np.uint32), pi.view(np.uint32))
    if cut is not None:
        assert np.array_equal(st.cut_len[:P * G].cpu().numpy(), cut)
    m = n if cap is None else min(n, cap)

    def check_lists():
        assert int(st.n_sel.item()) == n
        assert np.array_equal(st.sel_idx[:m].cpu().numpy(), si[:m])
        assert np.array_equal(st.sel_resp[:m].cpu().numpy(), sr[:m])
        assert np.array_equal(st.sel_offsets.cpu().numpy(), so)
        if m < st.sel_idx.numel():
            assert int(st.sel_idx[m:].max()) == -9       # nothing written past the lists' end

    check_lists()
    if mode != "urs":
        # prefix modes: st.compact() built the lists from the cut lengths alone; the
        # generic compaction of the mask must give the same lists
        for t in (st.sel_idx, st.sel_resp, st.sel_offsets, st.n_sel):
            t.fill_(-9)
        st.compact(cu_d, from_mask=True)
        torch.cuda.synchronize()
        check_lists()
    return n


@pytest.mark.parametrize("mode", ["urs", "rpc", "det"])
def test_tiny_lengths(mode):
    w = wl.WORKLOADS["tiny"]
    _select_compact(wl.make_lengths(w, 0), mode, w.P, w.G, seed=0)
    _select_compact(wl.make_lengths(w, 1), mode, w.P, w.G, seed=1, offset=(7 << 32) + 3)


@pytest.mark.parametrize("name", ["qwen3_0p6b", "qwen3_8b", "long_cot"])
@pytest.mark.parametrize("mode", ["urs", "rpc", "det"])
def test_config_lengths(name, mode):
    w = wl.WORKLOADS[name]
    n = _select_compact(wl.make_lengths(w, 0), mode, w.P, w.G, seed=0, p=0.5, min_cut=100)
    assert n > 0


@pytest.mark.parametrize("p", [0.25, 0.75, 1.0, 0.3, 1e-9])
def test_urs_probabilities(p):
    w = wl.WORKLOADS["qwen3_0p6b"]
    _select_compact(wl.make_lengths(w, 3), "urs", w.P, w.G, seed=5, p=p)


def test_edge_cases():
    # empty responses at the start, middle and end; single tokens; chunk-edge sizes
    _select_compact([0, 5, 0, 0, 3, 1, 0, 0], "urs", 2, 4, seed=2)
    _select_compact([0, 5, 0, 0, 3, 1, 0, 0], "rpc", 2, 4, seed=2, min_cut=2)
    _select_compact([0, 0, 0, 0], "rpc", 1, 4)
    _select_compact([4096, 4096], "urs", 1, 2, seed=3)
    _select_compact([4095, 1, 4096, 17], "det", 2, 2, seed=3)
    _select_compact([1] * 64, "rpc", 8, 8, seed=4, min_cut=0)
    _select_compact([30, 100, 101, 250], "rpc", 1, 4, seed=4, min_cut=100)
    _select_compact([32768, 9], "rpc", 1, 2, seed=9, min_cut=1)


def test_rpc_every_length_up_to_4096():
    # every denominator T - C + 1 <= 4096 with every numerator: the kernel forms pi by an FMA
    # sequence instead of a division and must still give the correctly rounded quotient
    T = np.random.default_rng(0).permutation(np.arange(1, 4097))
    _select_compact(T, "rpc", 512, 8, seed=3, min_cut=1)


def test_rpc_pi_is_the_rounded_quotient_for_every_length_up_to_32768():
    # all 5.4e8 quotients (T-t+1)/T with T <= 32768 (the longest response of the workloads)
    # against numpy's float32 division, which is what the oracle's definition of pi is
    Tmax = 32768
    T = np.arange(1, Tmax + 1, dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(T)])
    n_tot, B = int(cu[-1]), Tmax
    mask = torch.empty(n_tot, dtype=torch.uint8, device="cuda")
    pi = torch.empty(n_tot, dtype=torch.float32, device="cuda")
    cut = torch.empty(B, dtype=torch.int32, device="cuda")
    nat.nat_select(nat.select_params("rpc", min_cut=1, seed=3), B,
                   torch.from_numpy(cu.astype(np.int32)).cuda(), n_tot, mask, pi, cut)
    torch.cuda.synchronize()
    pi_h, mask_h, cut_h = pi.cpu().numpy(), mask.cpu().numpy(), cut.cpu().numpy()
    del mask, pi
    for i in range(B):
        Ti = int(T[i])
        t = np.arange(1, Ti + 1, dtype=np.int64)
        ref = (Ti - t + 1).astype(np.float32) / np.float32(Ti)
        assert np.array_equal(pi_h[cu[i]:cu[i + 1]].view(np.uint32), ref.view(np.uint32)), Ti
        assert np.array_equal(mask_h[cu[i]:cu[i + 1]], (t <= cut_h[i]).astype(np.uint8)), Ti
        assert 1 <= cut_h[i] <= Ti


def test_skewed_lengths_miss_the_proportional_window():
    # one very long response among many short ones: the blocks' proportional guess of the
    # owning response is far off, so the general search runs
    T = [3] * 500 + [40000] + [5] * 300 + [0] * 40 + [9000] + [2] * 182
    assert len(T) == 1024
    for mode in ("urs", "rpc", "det"):
        _select_compact(T, mode, 128, 8, seed=11, min_cut=4)


def test_capacity_smaller_than_selection():
    n = _select_compact([300, 200, 100, 50], "urs", 2, 2, seed=1, p=0.9, cap=64)
    assert n > 64
    n = _select_compact([300, 200, 100, 50], "det", 2, 2, seed=1, beta=0.9, cap=64)
    assert n > 64
    n = _select_compact([5000, 9000, 100, 50], "rpc", 2, 2, seed=1, min_cut=4000, cap=4099)
    assert n > 4099


def test_rewards_real_valued():
    r = np.random.default_rng(0).normal(size=48).astype(np.float32)
    _select_compact([3] * 48, "urs", 6, 8, rewards=r)
    _select_compact([3] * 48, "urs", 6, 8, rewards=np.full(48, 0.7, dtype=np.float32))


def test_invalid_arguments_are_rejected():
    cu = torch.zeros(3, dtype=torch.int32, device="cuda")
    buf = torch.zeros(16, dtype=torch.uint8, device="cuda")
    pi = torch.zeros(16, dtype=torch.float32, device="cuda")
    for kw in (dict(mode="urs", p=0.0), dict(mode="urs", p=1.5), dict(mode="det", beta=0.0),
               dict(mode="rpc", min_cut=-1), dict(mode=7)):
        with pytest.raises(nat.NatError):
            nat.nat_select(nat.select_params(**kw), 2, cu, 0, buf, pi, cu)
    with pytest.raises(nat.NatError):
        nat.nat_grpo_adv(2, 0, pi, 1e-6, pi)


# --------------------------------------------- general survival schedules (RPC)
def _schedule(T, rho, floor):
    p = np.maximum(rho ** np.arange(T), floor).astype(np.float32)
    if T:
        p[0] = 1.0
    return p


@pytest.mark.parametrize("lengths", [[1, 5, 64, 300, 0, 17, 4096, 33], [0, 0, 7, 0],
                                     "qwen3_0p6b"])
def test_survival_schedule_selection(lengths):
    if isinstance(lengths, str):
        lengths = wl.make_lengths(wl.WORKLOADS[lengths], 0)
    T = np.asarray(lengths, dtype=np.int32)
    cu = wl.cu_from_lengths(T)
    n_tot, B = int(cu[-1]), len(T)
    surv = np.concatenate([_schedule(int(t), 0.999 if t > 200 else 0.9, 0.03) for t in T])
    mask = torch.full((max(n_tot, 16),), 7, dtype=torch.uint8, device="cuda")
    cut = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    surv_d = torch.from_numpy(surv).cuda() if n_tot else torch.zeros(16, device="cuda")
    for seed, offset in ((3, 0), (3, (5 << 32) + 9)):
        nat.nat_select_survival(B, torch.from_numpy(cu).cuda(), n_tot, surv_d, seed, offset,
                                mask, cut, resp_base=offset & 7)
        torch.cuda.synchronize()
        ref_mask, ref_cut = oracle.select_survival(cu, surv, seed=seed, offset=offset,
                                                   resp_base=offset & 7)
        assert np.array_equal(mask[:n_tot].cpu().numpy(), ref_mask)
        assert np.array_equal(cut.cpu().numpy(), ref_cut)


def test_survival_schedule_feeds_the_loss():
    # pi = the schedule: selection, compaction and the loss agree with the oracle
    import parity
    w = wl.WORKLOADS["mid"]
    batch = wl.make_batch(w, seed=2, device="cuda")
    nb = wl.to_numpy(batch)
    cu = nb["cu_seqlens"]
    surv = np.concatenate([_schedule(int(t), 0.97, 0.05) for t in np.diff(cu)])
    st = NatStep(w.P, w.G, w.d, w.V, torch.bfloat16, batch["n_tot"])
    st.grpo_adv(batch["rewards"])
    st.pi.copy_(torch.from_numpy(surv).cuda())
    nat.nat_select_survival(w.B, batch["cu_seqlens"], batch["n_tot"], st.pi, 4, 0, st.mask,
                            st.cut_len)
    st.compact(batch["cu_seqlens"])
    st.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"],
                    batch["cu_seqlens"])
    torch.cuda.synchronize()
    mask, cut = oracle.select_survival(cu, surv, seed=4)
    si, sr, so, n = oracle.compact(mask, cu)
    ref_sel = dict(adv=oracle.grpo_adv(nb["rewards"], w.P, w.G, 1e-6), mask=mask, pi=surv, cut=cut,
                   sel_idx=si, sel_resp=sr, sel_offsets=so, n_sel=n)
    parity.check_selection(st, ref_sel, w)
    parity.check_loss(st, ref_sel, nb, w)


# ----------------------------------------------------- packing of selected rows
@pytest.mark.parametrize("d,dtype", [(64, torch.float32), (1024, torch.bfloat16), (8, torch.bfloat16)])
def test_gather_and_scatter_rows(d, dtype):
    w = wl.WORKLOADS["mid"]
    T = wl.make_lengths(w, 1)
    cu = wl.cu_from_lengths(T)
    n_tot = int(cu[-1])
    st = NatStep(w.P, w.G, 64, 512, torch.float32, n_tot, want_grads=False)
    cu_d = torch.from_numpy(cu).cuda()
    st.select(cu_d, "rpc", min_cut=3, seed=2)
    st.compact(cu_d)
    g = torch.Generator(device="cuda")
    g.manual_seed(0)
    x = torch.randn(n_tot, d, generator=g, device="cuda").to(dtype)
    n = int(st.n_sel.item())
    packed = torch.full((n_tot, d), 9.0, device="cuda").to(dtype)
    nat.nat_gather_rows(x, st.sel_idx, st.n_sel, n_tot, packed)
    back = torch.full((n_tot, d), 9.0, device="cuda").to(dtype)
    nat.nat_scatter_rows(packed, st.sel_idx, st.n_sel, n_tot, n_tot, back)
    torch.cuda.synchronize()
    si = st.sel_idx[:n].cpu().numpy()
    xn = x.float().cpu().numpy()
    assert np.array_equal(packed[:n].float().cpu().numpy(), oracle.gather_rows(xn, si))
    assert torch.all(packed[n:] == 9.0)                      # rows past n_sel untouched
    assert np.array_equal(back.float().cpu().numpy(),
                          oracle.scatter_rows(oracle.gather_rows(xn, si), si, n_tot))
    # the packed rows are the per-response prefixes, delimited by sel_offsets
    so = st.sel_offsets.cpu().numpy()
    cut = st.cut_len[:w.B].cpu().numpy()
    assert np.array_equal(np.diff(so), cut)
    # row_bytes must be a multiple of 16
    assert nat.load().nat_gather_rows(x.data_ptr(), 24, st.sel_idx.data_ptr(), st.n_sel.data_ptr(), 3,
                                      packed.data_ptr(), None) == -1


# ------------------------------------------------- sharding: response-index base
@pytest.mark.parametrize("mode", ["urs", "rpc", "det"])
def test_shards_realise_slices_of_the_whole_batch_selection(mode):
    """Two data-parallel shards of one batch, each passing only its own responses and the
    global index of its first one, draw exactly the whole batch's mask, pi and cuts."""
    w = wl.WORKLOADS["qwen3_0p6b"]
    T = wl.make_lengths(w, 2)
    cu = wl.cu_from_lengths(T)
    kw = dict(p=0.5, min_cut=100, beta=0.5, seed=5, offset=(3 << 32) + 1)
    mask, pi, cut = oracle.select(MODE_ID[mode], cu, **kw)
    for lo, hi in ((0, 24), (24, 64)):
        cu_s = wl.cu_from_lengths(T[lo:hi])
        n_s = int(cu_s[-1])
        st = NatStep((hi - lo) // w.G, w.G, 64, 512, torch.float32, n_s, want_grads=False,
                     B_global=w.B, resp_base=lo)
        cu_d = torch.from_numpy(cu_s).cuda()
        st.select(cu_d, mode, **kw)
        st.compact(cu_d)
        torch.cuda.synchronize()
        assert np.array_equal(st.mask[:n_s].cpu().numpy(), mask[cu[lo]:cu[hi]])
        assert np.array_equal(st.pi[:n_s].cpu().numpy().view(np.uint32),
                              pi[cu[lo]:cu[hi]].view(np.uint32))
        if cut is not None:
            assert np.array_equal(st.cut_len[:hi - lo].cpu().numpy(), cut[lo:hi])
        si, sr, so, n = oracle.compact(mask[cu[lo]:cu[hi]], cu_s)
        assert int(st.n_sel.item()) == n
        assert np.array_equal(st.sel_idx[:n].cpu().numpy(), si)
        assert np.array_equal(st.sel_resp[:n].cpu().numpy(), sr)


# ------------------------------------------------------------ general cut laws
def _law(T, rng):
    q = (np.maximum(0.995 ** np.arange(T), 0.05) * rng.uniform(0.5, 1.0, T) / max(T, 1))
    return q.astype(np.float32)


@pytest.mark.parametrize("lengths", [[1, 5, 64, 300, 0, 17, 4096, 33, 4095, 1, 0, 8193],
                                     [0, 0, 7, 0], [0, 0, 0], "qwen3_0p6b", "long_cot"])
def test_cut_law_selection(lengths):
    """nat_select_cutlaw against the oracle, bit for bit: pi is the suffix sum of the law
    over each response (a scan over the packed stream on the device), one cut per response."""
    if isinstance(lengths, str):
        lengths = wl.make_lengths(wl.WORKLOADS[lengths], 0)
    T = np.asarray(lengths, dtype=np.int32)
    cu = wl.cu_from_lengths(T)
    n_tot, B = int(cu[-1]), len(T)
    rng = np.random.default_rng(3)
    q = np.concatenate([_law(int(t), rng) for t in T] + [np.zeros(0, np.float32)])
    if n_tot > 40:
        q[7] = 0.0                      # a zero mass inside a response
        q[11] = -1.0                    # negative and NaN count as zero
        q[13] = np.nan
        q[15] = 2.0                     # masses of 1 and above saturate at 2^32 - 1
        q[16] = 1.0
        q[17] = 1e-40                   # subnormal: below the fixed-point quantum
        q[18] = np.float32(2.0 ** -33)  # just below one quantum, and exactly one
        q[19] = np.float32(2.0 ** -32)
        q[20] = np.inf
        q[cu[2]:cu[3]] = 0.0            # a response whose law has no mass at all: kept whole
    if B > 7:
        q[cu[7]:cu[8]] = 1.0 / 64       # dyadic uniform law
        q[cu[6] + 2000:cu[7]] = 0.0     # no mass after position 2000: pi = 0 there
    pad = max(n_tot, 16)
    mask = torch.full((pad,), 7, dtype=torch.uint8, device="cuda")
    pi = torch.full((pad,), -1.0, dtype=torch.float32, device="cuda")
    cut = torch.full((max(B, 1),), -1, dtype=torch.int32, device="cuda")
    q_d = torch.zeros(pad, device="cuda")
    q_d[:n_tot] = torch.from_numpy(q)
    ws = nat.alloc_workspace(nat.nat_select_cutlaw_workspace_bytes(B, n_tot), "cuda")
    cu_d = torch.from_numpy(cu).cuda()
    for seed, offset, base in ((3, 0, 0), (4, (5 << 32) + 9, 17)):
        nat.nat_select_cutlaw(B, cu_d, n_tot, q_d, seed, offset, mask, pi, cut, ws, resp_base=base)
        torch.cuda.synchronize()
        rm, rp, rc = oracle.select_cutlaw(cu, q, seed=seed, offset=offset, resp_base=base)
        assert np.array_equal(mask[:n_tot].cpu().numpy(), rm)
        assert np.array_equal(pi[:n_tot].cpu().numpy().view(np.uint32), rp.view(np.uint32))
        assert np.array_equal(cut[:B].cpu().numpy(), rc)
    # the cut lengths feed the prefix compaction
    st = NatStep(1, max(B, 1), 64, 512, torch.float32, n_tot, want_grads=False)
    nat.nat_compact_prefix(B, cu_d, n_tot, cut, st.sel_idx, st.sel_resp, st.sel_offsets, st.n_sel,
                           st.cap)
    torch.cuda.synchronize()
    si, sr, so, n = oracle.compact(rm, cu)
    assert int(st.n_sel.item()) == n
    assert np.array_equal(st.sel_idx[:n].cpu().numpy(), si)
    assert np.array_equal(st.sel_resp[:n].cpu().numpy(), sr)
    assert np.array_equal(st.sel_offsets[:B + 1].cpu().numpy(), so)


# ------------------------------------------------------------ maximum sizes
@pytest.mark.parametrize("mode", ["urs", "rpc"])
def test_stream_close_to_the_int32_limit(mode):
    """n_tot = 65535 responses of 32767 tokens = 2,147,385,345 (< 2^31): the largest packed
    stream the int32 indices can address.  The oracle evaluates a sample of responses on
    their own (their draws depend only on the global response index); the lists are checked
    in full against plain torch reductions of the mask and on sampled segments."""
    B, T = 65535, 32767
    n_tot = B * T
    assert n_tot < 2 ** 31 and n_tot > 2 ** 31 - 2 ** 17
    cu = torch.arange(0, n_tot + 1, T, dtype=torch.int64, device="cuda").to(torch.int32)
    st = NatStep(B // 5, 5, 64, 512, torch.float32, n_tot, want_grads=False)
    kw = dict(p=0.5, min_cut=100, seed=21, offset=(1 << 33) + 5)
    st.select(cu, mode, **kw)
    st.compact(cu)
    torch.cuda.synchronize()
    n_sel = int(st.n_sel.item())
    per_resp = st.mask[:n_tot].view(B, T).sum(dim=1, dtype=torch.int64)
    assert n_sel == int(per_resp.sum().item())
    offs = torch.zeros(B + 1, dtype=torch.int64, device="cuda")
    offs[1:] = per_resp.cumsum(0)
    assert torch.equal(st.sel_offsets.to(torch.int64), offs)
    rng = np.random.default_rng(3)
    one = wl.cu_from_lengths(np.array([T], dtype=np.int32))
    for i in [0, 1, B - 1, B - 2] + [int(x) for x in rng.integers(2, B - 2, size=4)]:
        m, p, c = oracle.select(MODE_ID[mode], one, resp_base=i, **kw)
        lo = i * T
        assert np.array_equal(st.mask[lo:lo + T].cpu().numpy(), m), i
        assert np.array_equal(st.pi[lo:lo + T].cpu().numpy().view(np.uint32), p.view(np.uint32)), i
        if c is not None:
            assert int(st.cut_len[i].item()) == int(c[0])
        k0, k1 = int(offs[i].item()), int(offs[i + 1].item())
        want = torch.nonzero(st.mask[lo:lo + T]).flatten() + lo
        assert torch.equal(st.sel_idx[k0:k1].to(torch.int64), want), i
        assert bool((st.sel_resp[k0:k1] == i).all()), i
    if mode == "rpc":
        # the generic compaction of the same mask gives the same lists
        idx_prefix = st.sel_idx[:n_sel].clone()
        st.sel_idx.fill_(-1)
        st.compact(cu, from_mask=True)
        torch.cuda.synchronize()
        assert int(st.n_sel.item()) == n_sel
        assert torch.equal(st.sel_idx[:n_sel], idx_prefix)


def test_prefix_compaction_clamps_cut_lengths():
    # cut lengths outside [0, T_i] (a caller's mistake) are clamped, never used as they are
    T = np.array([5, 0, 9, 3], dtype=np.int32)
    cu = wl.cu_from_lengths(T)
    n_tot = int(cu[-1])
    cut = torch.tensor([7, 4, -2, 3], dtype=torch.int32, device="cuda")      # -> 5, 0, 0, 3
    st = NatStep(1, 4, 64, 512, torch.float32, n_tot, want_grads=False)
    for t in (st.sel_idx, st.sel_resp):
        t.fill_(-9)
    nat.nat_compact_prefix(4, torch.from_numpy(cu).cuda(), n_tot, cut, st.sel_idx, st.sel_resp,
                           st.sel_offsets, st.n_sel, st.cap)
    torch.cuda.synchronize()
    assert int(st.n_sel.item()) == 8
    assert st.sel_offsets.cpu().tolist() == [0, 5, 5, 5, 8]
    assert st.sel_idx[:8].cpu().tolist() == [0, 1, 2, 3, 4, 14, 15, 16]
    assert st.sel_resp[:8].cpu().tolist() == [0] * 5 + [3] * 3
    assert int(st.sel_idx[8:].max()) == -9
