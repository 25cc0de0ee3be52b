"""Seeded random draws from the space of packed streams (batch shape, length mix with empty
responses and lengths on the 16-token and 4096-token boundaries of the kernels' layout,
selection rule and parameters, 64-bit seeds and offsets, capacities): advantages, masks,
inclusion probabilities, cuts and compacted lists are bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_06619_b200 import nat
from paper_2603_06619_b200 import workloads as wl

from test_gpu_select import _select_compact

pytestmark = pytest.mark.gpu


def _lengths(rng, B):
    kind = int(rng.integers(0, 6))
    if kind == 0:
        T = rng.integers(0, 50, size=B)
    elif kind == 1:
        T = rng.integers(0, 3, size=B) * rng.integers(0, 9000, size=B)
    elif kind == 2:
        T = 16 * rng.integers(0, 600, size=B) + rng.integers(0, 2, size=B)
    elif kind == 3:
        T = 4096 * rng.integers(0, 4, size=B) + rng.integers(0, 3, size=B)
    elif kind == 4:
        T = np.rint(np.exp(rng.normal(6, 2, size=B))).clip(0, 40000)
    else:
        T = rng.integers(1, 20000, size=B)
    T = np.asarray(T, dtype=np.int64).clip(0)
    if T.sum() == 0:
        T[0] = 1
    return T.astype(np.int32)


@pytest.mark.parametrize("block", range(4))
def test_random_selection_and_compaction(block):
    rng = np.random.default_rng(2000 + block)
    for _ in range(12):
        P, G = int(rng.integers(1, 6)), int(rng.integers(1, 9))
        T = _lengths(rng, P * G)
        kw = dict(seed=int(rng.integers(0, 2 ** 62)), offset=int(rng.integers(0, 2 ** 63)),
                  p=float(rng.choice([1e-6, 0.1, 0.25, 0.5, 0.77, 0.999, 1.0])),
                  min_cut=int(rng.choice([0, 1, 2, 15, 16, 17, 100, 5000])),
                  beta=float(rng.choice([0.01, 0.3, 0.5, 0.99, 1.0])))
        if rng.random() < 0.2:
            kw["cap"] = int(rng.integers(1, max(2, int(T.sum()))))
        _select_compact(T, str(rng.choice(["urs", "rpc", "det"])), P, G, **kw)


@pytest.mark.parametrize("block", range(3))
def test_random_cut_laws(block):
    rng = np.random.default_rng(3000 + block)
    for _ in range(10):
        B = int(rng.integers(1, 40))
        T = _lengths(rng, B)
        cu = wl.cu_from_lengths(T)
        n_tot = int(cu[-1])
        style = int(rng.integers(0, 4))
        if style == 0:
            q = rng.random(n_tot)
        elif style == 1:
            q = rng.random(n_tot) * (rng.random(n_tot) < 0.1)          # sparse laws
        elif style == 2:
            q = np.exp(rng.normal(-20, 8, n_tot))                      # masses around the quantum
        else:
            q = rng.choice([0.0, 1.0, 2.0 ** -32, 0.5, 3.0, -1.0], n_tot)
        q = q.astype(np.float32)
        seed, offset = int(rng.integers(0, 2 ** 62)), int(rng.integers(0, 2 ** 63))
        base = int(rng.integers(0, 1000))
        pad = max(n_tot, 16)
        mask = torch.full((pad,), 7, dtype=torch.uint8, device="cuda")
        pi = torch.full((pad,), -1.0, dtype=torch.float32, device="cuda")
        cut = torch.full((B,), -1, dtype=torch.int32, device="cuda")
        q_d = torch.zeros(pad, device="cuda")
        q_d[:n_tot] = torch.from_numpy(q)
        ws = nat.alloc_workspace(nat.nat_select_cutlaw_workspace_bytes(B, n_tot), "cuda")
        nat.nat_select_cutlaw(B, torch.from_numpy(cu).cuda(), n_tot, q_d, seed, offset, mask, pi,
                              cut, ws, resp_base=base)
        torch.cuda.synchronize()
        rm, rp, rc = oracle.select_cutlaw(cu, q, seed=seed, offset=offset, resp_base=base)
        assert np.array_equal(mask[:n_tot].cpu().numpy(), rm)
        assert np.array_equal(pi[:n_tot].cpu().numpy().view(np.uint32), rp.view(np.uint32))
        assert np.array_equal(cut[:B].cpu().numpy(), rc)
