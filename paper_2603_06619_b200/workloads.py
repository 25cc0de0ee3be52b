"""Seeded synthetic workloads shaped like the paper's Qwen3 GRPO batches.

This module only draws inputs (lengths, hidden states, LM-head weights,
targets, rewards, behaviour-policy log-probs).  It holds none of the method's
arithmetic: selection, weighting, the surrogate and its gradients live in the
CUDA library (and, separately, in the test oracle).  The one derived input,
``old_logp``, is a library log-softmax of the drawn logits plus noise (torch's
matmul and logsumexp: the only place in the package where a library GEMM runs,
and only to make an input); it is an input like any other and both sides
receive the same bytes.

Shapes follow the paper's training recipe (8 rollouts per prompt, responses up
to 8192 tokens for Qwen3-8B, Appendix C) and the Qwen3 head sizes
(d = 1024 / 4096, V = 151936).
"""
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    P: int                    # prompts
    G: int                    # responses per prompt
    d: int
    V: int
    dtype: str                # "f32" | "bf16"
    length_law: str           # "uniform" | "lognormal"
    len_lo: int
    len_hi: int
    len_median: int = 0
    len_sigma: float = 0.75   # log-normal shape (only median and cap are given)
    sel_mode: str = "urs"     # "urs" | "rpc" | "det"
    p: float = 0.5
    min_cut: int = 1
    beta: float = 0.5
    w_scale: float = 0.02
    old_noise: float = 0.05
    reward_p: float = 0.4

    @property
    def B(self):
        return self.P * self.G


WORKLOADS = {
    # Tiny fp32 case: small enough to enumerate every mask / cut.
    "tiny": Workload("tiny", P=2, G=4, d=64, V=512, dtype="f32", length_law="uniform",
                     len_lo=8, len_hi=64, sel_mode="urs", p=0.5),
    "tiny_rpc": Workload("tiny_rpc", P=2, G=4, d=64, V=512, dtype="f32", length_law="uniform",
                         len_lo=8, len_hi=64, sel_mode="rpc", min_cut=1),
    # Qwen3-0.6B-shaped head.
    "qwen3_0p6b": Workload("qwen3_0p6b", P=8, G=8, d=1024, V=151936, dtype="bf16",
                           length_law="uniform", len_lo=256, len_hi=2048, sel_mode="urs", p=0.5),
    # Qwen3-8B-shaped head, RPC with the paper's minimum cut of 100 tokens.
    "qwen3_8b": Workload("qwen3_8b", P=16, G=8, d=4096, V=151936, dtype="bf16",
                         length_law="lognormal", len_lo=16, len_hi=8192, len_median=2048,
                         sel_mode="rpc", min_cut=100),
    # Long chain-of-thought.
    "long_cot": Workload("long_cot", P=4, G=16, d=4096, V=151936, dtype="bf16",
                         length_law="uniform", len_lo=8192, len_hi=32768, sel_mode="rpc",
                         min_cut=100),
    # Reduced twins: same head (d, V, dtype) with few, short responses, so the
    # fp64 oracle can evaluate every row.  Row counts are not tile multiples.
    "twin_0p6b": Workload("twin_0p6b", P=2, G=4, d=1024, V=151936, dtype="bf16",
                          length_law="uniform", len_lo=40, len_hi=130, sel_mode="urs", p=0.5),
    "twin_8b": Workload("twin_8b", P=2, G=4, d=4096, V=151936, dtype="bf16",
                        length_law="uniform", len_lo=30, len_hi=90, sel_mode="rpc", min_cut=10),
    # Mid-size bf16 head with ragged V and d used by the element-by-element
    # parity tests (several row tiles, several vocab tiles, a ragged tail).
    "mid": Workload("mid", P=3, G=4, d=256, V=5000, dtype="bf16", length_law="uniform",
                    len_lo=20, len_hi=120, sel_mode="urs", p=0.5),
}


def variant(w: Workload, **kw) -> Workload:
    return replace(w, **kw)


def make_lengths(w: Workload, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64([seed, 101]))
    if w.length_law == "uniform":
        T = rng.integers(w.len_lo, w.len_hi + 1, size=w.B)
    elif w.length_law == "lognormal":
        T = np.rint(np.exp(rng.normal(np.log(w.len_median), w.len_sigma, size=w.B)))
        T = np.clip(T, w.len_lo, w.len_hi)
    else:
        raise ValueError(w.length_law)
    return T.astype(np.int32)


def cu_from_lengths(T: np.ndarray) -> np.ndarray:
    cu = np.zeros(T.shape[0] + 1, dtype=np.int32)
    np.cumsum(T, out=cu[1:])
    return cu


def _torch_dtype(w: Workload):
    return torch.float32 if w.dtype == "f32" else torch.bfloat16


def library_logp(hidden, W, targets, rows_per_chunk=4096):
    """log-softmax(hidden @ W^T)[target] via plain torch library calls.

    Only used to place ``old_logp`` near the current log-probability, as the
    workload recipe asks; its accuracy does not matter (it is an input).
    """
    out = torch.empty(hidden.shape[0], dtype=torch.float32, device=hidden.device)
    for lo in range(0, hidden.shape[0], rows_per_chunk):
        hi = min(lo + rows_per_chunk, hidden.shape[0])
        if hidden.is_cuda:
            z = (hidden[lo:hi] @ W.t()).float()
        else:
            z = hidden[lo:hi].float() @ W.float().t()
        lse = torch.logsumexp(z, dim=1)
        out[lo:hi] = z.gather(1, targets[lo:hi].long()[:, None])[:, 0] - lse
    return out


def make_batch(w: Workload, seed: int = 0, device="cpu", lengths=None, W_seed=None):
    """Draw one batch.  Returns a dict of torch tensors on ``device``:

    lengths/cu_seqlens int32, hidden [N_tot, d], W [V, d] (dtype of the
    workload), targets int32 [N_tot], rewards float32 [B], old_logp float32
    [N_tot].

    ``W_seed``: draw W from a generator of its own with this seed, so that data-parallel
    ranks that draw different shards (different ``seed``) hold the same replicated W.
    """
    T = make_lengths(w, seed) if lengths is None else np.asarray(lengths, dtype=np.int32)
    cu = cu_from_lengths(T)
    n_tot = int(cu[-1])
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(1000003 * seed + 17)
    dt = _torch_dtype(w)
    hidden = torch.randn(n_tot, w.d, generator=g, device=dev, dtype=torch.float32).to(dt)
    gW = g
    if W_seed is not None:
        gW = torch.Generator(device=dev)
        gW.manual_seed(1000003 * int(W_seed) + 29)
    W = (torch.randn(w.V, w.d, generator=gW, device=dev, dtype=torch.float32) * w.w_scale).to(dt)
    targets = torch.randint(0, w.V, (n_tot,), generator=g, device=dev, dtype=torch.int32)
    rewards = (torch.rand(w.B, generator=g, device=dev) < w.reward_p).float()
    noise = torch.randn(n_tot, generator=g, device=dev, dtype=torch.float32) * w.old_noise
    old_logp = library_logp(hidden, W, targets) + noise
    return dict(
        lengths=torch.from_numpy(T.copy()),
        cu_seqlens=torch.from_numpy(cu.copy()).to(dev),
        hidden=hidden, W=W, targets=targets, rewards=rewards, old_logp=old_logp,
        n_tot=n_tot,
    )


def to_numpy(batch):
    """Host copies as numpy arrays (bf16 widened exactly to float32)."""
    out = {}
    for k, v in batch.items():
        if isinstance(v, torch.Tensor):
            v = v.detach().cpu()
            out[k] = (v.float() if v.dtype == torch.bfloat16 else v).numpy()
        else:
            out[k] = v
    return out
