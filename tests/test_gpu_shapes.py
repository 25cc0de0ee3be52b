"""bf16 loss parity at the edges of the shape space: vocabularies of one entry up to a few
tiles with ragged tails, hidden sizes that are not a power of two, row counts on and around
the 512-row padding and the 8192-row chunk, empty responses.  Every case runs both routes
(forward + backward calls, single-pass call) against the oracle, element by element."""
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
