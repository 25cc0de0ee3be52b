"""bf16 loss parity at the edges of the shape space: vocabularies of one entry up to a few
tiles with ragged tails, hidden sizes that are not a power of two, row counts on and around
the 512-row padding and the 8192-row chunk, empty responses.  Every case runs both routes
(forward + backward calls, single-pass call) against the oracle, element by element."""
import numpy as np
import pytest

import parity
from paper_2603_06619_b200 import workloads as wl

pytestmark = pytest.mark.gpu

BASE = wl.WORKLOADS["mid"]

CASES = [
    # d,   V,    P, G, len_lo, len_hi, mode,  extra
    (64,   1,    2, 4, 3,   20,  "urs", {}),
    (64,   2,    2, 4, 3,   20,  "rpc", {}),
    (64,   7,    2, 4, 0,   30,  "urs", {"w_scale": 0.5}),
    (128,  255,  2, 4, 5,   40,  "rpc", {"min_cut": 3}),
    (128,  256,  2, 4, 5,   40,  "urs", {"p": 0.75}),
    (128,  257,  2, 4, 5,   40,  "det", {"w_scale": 0.5}),
    (192,  513,  1, 2, 1,   1,   "urs", {"p": 1.0}),
    (1088, 700,  2, 4, 20,  60,  "rpc", {"min_cut": 10, "w_scale": 0.1}),
    (64,   300,  1, 8, 64,  64,  "urs", {"p": 1.0}),          # exactly 512 selected rows
    (64,   300,  1, 8, 64,  65,  "urs", {"p": 1.0}),          # just past the 512-row padding
    (64,   130,  2, 8, 500, 530, "urs", {"p": 1.0}),          # a full row chunk and a few rows
]


@pytest.mark.parametrize("d,V,P,G,lo,hi,mode,extra", CASES)
def test_edge_shapes(d, V, P, G, lo, hi, mode, extra):
    w = wl.variant(BASE, d=d, V=V, P=P, G=G, len_lo=lo, len_hi=hi, sel_mode=mode, old_noise=0.2,
                   **extra)
    out, _ = parity.run_case(w, seed=d + V, routes=(False, True))
    assert out["status"] & ~4 == 0


def _random_case(rng):
    d = 64 * int(rng.integers(1, 25))
    V = int(rng.choice([rng.integers(1, 64), rng.integers(64, 700), rng.integers(700, 6000)]))
    lo = int(rng.integers(0, 40))
    hi = lo + int(rng.integers(0, 200))
    if rng.random() < 0.2:
        lo, hi = 400, 700                       # more than one row chunk when there are many responses
    return dict(d=d, V=V, P=int(rng.integers(1, 4)), G=int(rng.integers(2, 9)), len_lo=lo, len_hi=hi,
                sel_mode=str(rng.choice(["urs", "rpc", "det"])),
                old_noise=float(rng.choice([0.05, 0.3])), w_scale=float(rng.choice([0.02, 0.1, 0.5])),
                p=float(rng.choice([0.25, 0.5, 0.9, 1.0])), min_cut=int(rng.integers(0, 50)),
                beta=float(rng.choice([0.3, 0.5, 1.0])))


@pytest.mark.parametrize("block", range(4))
def test_random_shapes(block):
    """Seeded random draws from the shape space (hidden size, vocabulary, batch, length mix,
    selection rule and its parameter, logit scale), eight per block, both routes."""
    rng = np.random.default_rng(1000 + block)
    for it in range(8):
        kw = _random_case(rng)
        out, _ = parity.run_case(wl.variant(BASE, **kw), seed=100 * block + it, routes=(False, True))
        assert out["status"] & ~4 == 0, kw
