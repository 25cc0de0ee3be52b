"""One partial-token GRPO policy-gradient step through the C-ABI library.

``NatStep`` owns the device buffers of one batch shape (torch is only the
allocator and the stream) and exposes the five calls of the path in the order
a trainer makes them: advantages, select, compact, loss forward, loss backward.
"""
import torch

from . import nat


class NatStep:
    def __init__(self, P, G, d, V, dtype, n_tot, device="cuda", n_sel_cap=None,
                 clip_lo=0.2, clip_hi=0.2, eps=1e-6, hidden_is_compact=False, want_grads=True,
                 kl_beta=0.0, ref_logp=None, B_global=None, resp_base=0):
        """``B_global`` / ``resp_base``: for a data-parallel shard, the number of responses of
        the whole job's batch (the batch mean's divisor) and the global index of this
        shard's first response (the selection draws are keyed by it)."""
        self.P, self.G, self.B = P, G, P * G
        self.B_global = self.B if B_global is None else int(B_global)
        self.resp_base = int(resp_base)
        self.prefix_mode = False
        self.d, self.V, self.dtype = d, V, dtype
        self.n_tot = int(n_tot)
        self.cap = int(n_tot if n_sel_cap is None else n_sel_cap)
        self.eps = eps
        dev = torch.device(device)
        self.device = dev
        i32, f32 = torch.int32, torch.float32
        self.adv = torch.empty(self.B, dtype=f32, device=dev)
        self.mask = torch.empty(max(self.n_tot, 1), dtype=torch.uint8, device=dev)
        self.pi = torch.empty(max(self.n_tot, 1), dtype=f32, device=dev)
        self.cut_len = torch.zeros(max(self.B, 1), dtype=i32, device=dev)
        self.sel_idx = torch.empty(max(self.cap, 1), dtype=i32, device=dev)
        self.sel_resp = torch.empty(max(self.cap, 1), dtype=i32, device=dev)
        self.sel_offsets = torch.empty(self.B + 1, dtype=i32, device=dev)
        self.n_sel = torch.zeros(1, dtype=i32, device=dev)
        self.compact_ws = nat.alloc_workspace(nat.nat_compact_workspace_bytes(self.n_tot), dev)
        self.ref_logp = ref_logp            # keeps the tensor alive while params point at it
        self.params = nat.loss_params(d, V, dtype, self.B_global, clip_lo, clip_hi, hidden_is_compact,
                                      kl_beta=kl_beta, ref_logp=ref_logp)
        self.loss = torch.zeros(1, dtype=f32, device=dev)
        self.logp = torch.empty(max(self.cap, 1), dtype=f32, device=dev)
        self.lse = torch.empty(max(self.cap, 1), dtype=f32, device=dev)
        self.loss_ws = nat.alloc_workspace(
            nat.nat_policy_loss_workspace_bytes(self.params, self.cap), dev)
        self.dH = self.dW = None
        if want_grads:
            self.dH = torch.empty(max(self.cap, 1), d, dtype=dtype, device=dev)
            self.dW = torch.empty(V, d, dtype=f32, device=dev)

    # -- the five calls ----------------------------------------------------
    def grpo_adv(self, rewards):
        nat.nat_grpo_adv(self.P, self.G, rewards, self.eps, self.adv)
        return self.adv

    def select(self, cu_seqlens, mode, p=1.0, min_cut=1, beta=1.0, seed=0, offset=0):
        sp = nat.select_params(mode, p=p, min_cut=min_cut, beta=beta, seed=seed, offset=offset,
                               resp_base=self.resp_base)
        self.prefix_mode = sp.mode != nat.NAT_SEL_URS
        cut = self.cut_len if self.prefix_mode else None
        nat.nat_select(sp, self.B, cu_seqlens, self.n_tot, self.mask, self.pi, cut)

    def compact(self, cu_seqlens, from_mask=False):
        """Compacted lists of the last selection: straight from the cut lengths after a
        prefix mode (RPC, truncation), from the mask otherwise (or when asked to)."""
        if self.prefix_mode and not from_mask:
            nat.nat_compact_prefix(self.B, cu_seqlens, self.n_tot, self.cut_len, self.sel_idx,
                                   self.sel_resp, self.sel_offsets, self.n_sel, self.cap)
        else:
            nat.nat_compact(self.B, cu_seqlens, self.n_tot, self.mask, self.sel_idx,
                            self.sel_resp, self.sel_offsets, self.n_sel, self.cap,
                            self.compact_ws)

    def loss_fwd(self, hidden, W, targets, old_logp, cu_seqlens):
        nat.nat_policy_loss_fwd(self.params, hidden, W, targets, old_logp, self.adv, self.pi,
                                cu_seqlens, self.sel_idx, self.sel_resp, self.n_sel, self.cap,
                                self.loss, self.logp, self.lse, self.loss_ws)

    def loss_bwd(self, hidden, W, targets, old_logp, cu_seqlens, dloss=None, accumulate_dW=False):
        self.params.accumulate_dW = int(accumulate_dW)
        nat.nat_policy_loss_bwd(self.params, hidden, W, targets, old_logp, self.adv, self.pi,
                                cu_seqlens, self.sel_idx, self.sel_resp, self.n_sel, self.cap,
                                self.logp, self.lse, dloss, self.dH, self.dW, self.loss_ws)

    def loss_fwd_bwd(self, hidden, W, targets, old_logp, cu_seqlens, dloss=None,
                     accumulate_dW=False):
        self.params.accumulate_dW = int(accumulate_dW)
        nat.nat_policy_loss_fwd_bwd(self.params, hidden, W, targets, old_logp, self.adv, self.pi,
                                    cu_seqlens, self.sel_idx, self.sel_resp, self.n_sel, self.cap,
                                    dloss, self.loss, self.logp, self.lse, self.dH, self.dW,
                                    self.loss_ws)

    def run(self, batch, mode, p=1.0, min_cut=1, beta=1.0, seed=0, offset=0, backward=True,
            fused=False):
        """All steps of the path on one batch (a dict from ``workloads.make_batch``)."""
        cu = batch["cu_seqlens"]
        self.grpo_adv(batch["rewards"])
        self.select(cu, mode, p=p, min_cut=min_cut, beta=beta, seed=seed, offset=offset)
        self.compact(cu)
        if fused:
            self.loss_fwd_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
            return
        self.loss_fwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)
        if backward:
            self.loss_bwd(batch["hidden"], batch["W"], batch["targets"], batch["old_logp"], cu)

    def status(self):
        return nat.device_status(self.loss_ws)
