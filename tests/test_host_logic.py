"""Host-side algebra of the package that needs no GPU."""
import numpy as np
import torch

import oracle
from paper_2509_09679_b200.composite import cayley_pullback


def test_cayley_pullback_matches_central_differences_of_the_oracle():
    rng = np.random.default_rng(0)
    for n1 in (2, 5, 9):
        par = rng.standard_normal(n1 * (n1 - 1) // 2) * 0.4
        Gq = rng.standard_normal((n1, n1))  # dL/dQ1 of L = sum(Gq * Q1)
        loss = lambda q: float(np.sum(Gq * oracle.cayley(q, n1)))
        fd = np.zeros_like(par)
        for k in range(par.size):
            e = np.zeros_like(par)
            e[k] = 1e-6
            fd[k] = (loss(par + e) - loss(par - e)) / 2e-6
        got = cayley_pullback(torch.from_numpy(par), n1, torch.from_numpy(Gq)).numpy()
        assert np.abs(got - fd).max() <= 1e-7 * max(1.0, np.abs(fd).max())
