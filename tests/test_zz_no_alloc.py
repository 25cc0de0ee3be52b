"""nat_compact_static: compaction for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits when the call is
made: inside a framework that already owns all of the GPU's memory, in a
callback that must not synchronise the device, or in a loop that has to stay
clear of any allocator.  For them the library keeps its scan scratch in a fixed
array of its own.  This test drives that entry point through the C ABI and
checks it against nat_compact (integer outputs, so bit for bit), twice in a
row because all calls share the one array and the second call must not be
disturbed by what the first left behind.

The file sorts last on purpose: a run that stops at the first failure has then
already gone through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2603_06619_b200 import nat
from paper_2603_06619_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _both(T, p, seed):
    T = np.asarray(T, dtype=np.int32)
    cu_h = wl.cu_from_lengths(T)
    B, n_tot = len(T), int(cu_h[-1])
    cu = torch.from_numpy(cu_h).cuda()
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    mask = (torch.rand(max(n_tot, 1), generator=g, device="cuda") < p).to(torch.uint8)
    outs = []
    for static in (False, True):
        # poison the outputs so that a call which writes nothing cannot pass
        idx = torch.full((max(n_tot, 1),), -7, dtype=torch.int32, device="cuda")
        resp = torch.full((max(n_tot, 1),), -7, dtype=torch.int32, device="cuda")
        offs = torch.full((B + 1,), -7, dtype=torch.int32, device="cuda")
        n_sel = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        if static:
            nat.nat_compact_static(B, cu, n_tot, mask, idx, resp, offs, n_sel, n_tot)
        else:
            ws = nat.alloc_workspace(nat.nat_compact_workspace_bytes(n_tot), "cuda")
            nat.nat_compact(B, cu, n_tot, mask, idx, resp, offs, n_sel, n_tot, ws)
        torch.cuda.synchronize()
        outs.append((idx, resp, offs, n_sel))
    (i0, r0, o0, n0), (i1, r1, o1, n1) = outs
    n = int(n0.item())
    assert n == int(mask[:n_tot].sum().item())
    assert int(n1.item()) == n
    assert torch.equal(i0[:n], i1[:n]) and torch.equal(r0[:n], r1[:n]) and torch.equal(o0, o1)
    return n


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # a long input first, a short one second: the second call sees the first one's
    # leftovers in the shared scratch and must ignore them
    lengths = wl.make_lengths(wl.WORKLOADS["qwen3_8b"], 0)
    n_long = _both(lengths, 0.5, seed=1)
    n_short = _both([5, 0, 4097, 33, 0], 0.3, seed=2)
    assert n_long > 4096 * 8 and 0 < n_short < 4200
    # and the long one again, after the short one
    assert _both(lengths, 0.5, seed=1) == n_long


def test_static_scratch_rejects_oversized_input():
    limit = nat.nat_compact_static_max_tokens()
    assert limit == 16384 * 4096
    t = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(nat.NatError, match="exceeds the built-in scratch"):
        nat.nat_compact_static(1, t, limit + 1, t, t, t, t, t, 8)
