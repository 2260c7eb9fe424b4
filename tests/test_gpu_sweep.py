"""Two cells of the parameter sweep (paper_2109_09868_b200/sweep.py; the grid of Section 4.2 and Appendix B on
synthetic stand-ins), one with a linear stand-in model and one with a softmax behind it, run through the library
and checked against the oracle: located sets on every group the oracle calls solid, decoded values on every group."""
import numpy as np
import pytest
import torch

import oracle
from paper_2109_09868_b200 import sweep

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,S,E,sigma,softmax", [(8, 0, 2, 10.0, False), (10, 1, 1, 100.0, True)])
def test_sweep_cell_matches_oracle(K, S, E, sigma, softmax):
    G, C = 512, 10
    cell = sweep.run_cell(K, S, E, sigma, softmax, G, C, 64, 4242 + K, torch.device("cuda:0"), keep_tensors=True)
    t = cell["tensors"]
    W = cell["W"]
    Yt = t["Yt"].cpu().numpy()
    ref = oracle.locate(K, W, E, Yt, t["mask"])
    solid = (ref["min_gap"] > 1.0 + 1e-6) & (ref["vote_margin"] > 0) & ((ref["status"] & oracle.ST_ORACLE_RANK_DEFICIENT) == 0)
    assert solid.mean() > 0.9
    adv = t["adv"].cpu().numpy()
    np.testing.assert_array_equal(adv[solid], ref["adv"][solid])
    if not softmax:  # a linear model makes the honest predictions exactly rational: Theorem 1 applies
        assert solid.all() and np.array_equal(adv, t["injected"]) and cell["located_equals_injected"] == 1.0
    trusted = t["trusted"].cpu().numpy().view(np.uint32)
    want, _, _ = oracle.decode(K, W, Yt, trusted)
    got = t["Yhat"].cpu().numpy().astype(np.float64)
    err = np.abs(got - want).reshape(G, -1).max(axis=1)
    assert np.all(err <= 1e-4 * np.abs(want).reshape(G, -1).max(axis=1))
