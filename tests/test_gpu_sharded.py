"""Data-parallel sharding through the CUDA path, played on one device.

Ranks of a data-parallel job take whole prompt groups.  Each passes only its own responses
to the library, with the job's batch size as the batch mean's divisor (Eq. grpo-obj: the
mean runs over all responses of the batch) and the global index of its first response as
the base of the selection's random draws (the masks of different responses are independent,
Section 3.1, so a shard must reproduce the whole batch's mask for its responses).  Then the
ranks' losses and dW add up to the single-rank step's, and their dHidden rows are its rows:
the one exchange of a trainer is a sum (all-reduce) of loss and dW.  Here the two ranks
run one after the other on the same GPU, the second accumulating into the first's dW.
"""
import numpy as np
import pytest
import torch

from paper_2603_06619_b200 import sharding
from paper_2603_06619_b200 import workloads as wl
from paper_2603_06619_b200.step import NatStep

import parity

pytestmark = pytest.mark.gpu


def _shard(batch, cu, lo, hi):
    a, b = int(cu[lo]), int(cu[hi])
    cu_s = (cu[lo:hi + 1] - cu[lo]).astype(np.int32)
    return dict(hidden=batch["hidden"][a:b].contiguous(), W=batch["W"],
                targets=batch["targets"][a:b].contiguous(),
                old_logp=batch["old_logp"][a:b].contiguous(),
                rewards=batch["rewards"][lo:hi].contiguous(),
                cu_seqlens=torch.from_numpy(cu_s).cuda(), n_tot=b - a)


@pytest.mark.parametrize("mode,fused", [("urs", True), ("rpc", True), ("urs", False)])
def test_two_shards_add_up_to_the_single_rank_step(mode, fused):
    w = wl.variant(wl.WORKLOADS["mid"], sel_mode=mode, min_cut=5, old_noise=0.3)
    seed, offset = 3, 2
    batch = wl.make_batch(w, seed=seed, device="cuda")
    nb = wl.to_numpy(batch)
    cu = nb["cu_seqlens"]
    ref_sel = parity.oracle_selection(w, nb, seed, offset)
    single = parity.gpu_step(w, batch, seed, offset, fused=fused)
    parity.check_selection(single, ref_sel, w)
    out, ref = parity.check_loss(single, ref_sel, nb, w)          # the single rank is right

    world = 2
    dtype = torch.bfloat16
    dW = torch.zeros_like(single.dW)
    loss_sum, rows = 0.0, []
    for rank in range(world):
        lo, hi = sharding.response_range(w.P, w.G, rank, world)
        sb = _shard(batch, cu, lo, hi)
        st = NatStep((hi - lo) // w.G, w.G, w.d, w.V, dtype, sb["n_tot"], B_global=w.B,
                     resp_base=lo)
        st.dW = dW                                                # the job's gradient buffer
        cu_d = sb["cu_seqlens"]
        st.grpo_adv(sb["rewards"])
        st.select(cu_d, mode, p=w.p, min_cut=w.min_cut, seed=seed, offset=offset)
        st.compact(cu_d)
        args = (sb["hidden"], sb["W"], sb["targets"], sb["old_logp"], cu_d)
        if fused:
            st.loss_fwd_bwd(*args, accumulate_dW=rank > 0)
        else:
            st.loss_fwd(*args)
            st.loss_bwd(*args, accumulate_dW=rank > 0)
        torch.cuda.synchronize()
        assert st.status() & ~4 == 0
        # the shard's selection is the whole batch's, restricted to its responses
        a, b = int(cu[lo]), int(cu[hi])
        assert torch.equal(st.mask[:b - a], single.mask[a:b])
        assert torch.equal(st.pi[:b - a], single.pi[a:b])
        assert torch.equal(st.adv, single.adv[lo:hi])
        n = int(st.n_sel.item())
        k0 = int(ref_sel["sel_offsets"][lo])
        assert n == int(ref_sel["sel_offsets"][hi]) - k0
        assert torch.equal(st.sel_idx[:n] + a, single.sel_idx[k0:k0 + n])
        # per-token outputs are the single rank's rows (the vocabulary may be split
        # differently for a smaller batch, so fp32 sums can differ in their last bits)
        assert float((st.logp[:n] - single.logp[k0:k0 + n]).abs().max()) <= 2e-5
        assert parity.rel_fro(st.dH[:n].float().cpu().numpy(),
                              single.dH[k0:k0 + n].float().cpu().numpy()) < 1e-3
        loss_sum += float(st.loss.item())
        rows.append(st.dH[:n].float().cpu().numpy())
    n_all = ref_sel["n_sel"]
    floor = 1e-2 * float(np.sum(ref["w"] * np.abs(ref["L"])))
    assert abs(loss_sum - ref["loss"]) <= parity.TOL_LOSS * max(abs(ref["loss"]), floor)
    assert parity.rel_fro(dW.cpu().numpy(), single.dW.cpu().numpy()) < 1e-3
    # and against the oracle's single-rank gradients
    assert parity.rel_fro(dW.cpu().numpy(), ref["dW"]) <= parity.TOL_GRAD
    assert parity.rel_fro(np.concatenate(rows), ref["dH"]) <= parity.TOL_GRAD
    assert sum(r.shape[0] for r in rows) == n_all
