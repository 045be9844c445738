"""The chunked algebra (tests/chunked_math.py) must equal the per-timestep oracle to rounding:
a check of the derivation the CUDA kernels follow, independent of both."""
import numpy as np
import pytest

from oracle import ssd_oracle as orc
from tests.chunked_math import chunked_bwd, chunked_fwd
from tests.test_oracle_pins import rand_problem


@pytest.mark.parametrize("Q", [4, 16])
def test_chunked_equals_recurrence(Q):
    rng = np.random.default_rng(9)
    d = rand_problem(rng, B=2, L=48, H=4, P=3, N=5, G=2)
    y, hf, _ = orc.ssd_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"])
    y2, hf2 = chunked_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], Q)
    np.testing.assert_allclose(y2, y, rtol=0, atol=1e-12)
    np.testing.assert_allclose(hf2, hf, rtol=0, atol=1e-12)
    g = orc.ssd_bwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], d["dy"], d["dh_final"])
    g2 = chunked_bwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], d["dy"], d["dh_final"], Q)
    for k in g:
        np.testing.assert_allclose(g2[k], g[k], rtol=0, atol=1e-11 * max(1.0, np.abs(g[k]).max()), err_msg=k)
