"""ESS-floor weight shrinkage on the GPU against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,p_width", [(128000, 1024), (4097, 128), (100, 128), (70000, 20 * 128)])
def test_ess_weights_match_oracle(n, p_width):
    g = torch.Generator().manual_seed(n)
    sig = torch.tensor([0.0, 0.1, 1.0, 2.5, 4.0, 1.0])[:, None]
    r = torch.exp(sig * torch.randn(6, n, generator=g)) * torch.tensor([1.0, 3.0, 0.01, 1.0, 50.0, 1.0])[:, None]
    r[5] = 0.0                                                     # a row without sensitivity
    w = torch.full((6, n), float("nan"), device="cuda")
    alpha = torch.full((6,), float("nan"), device="cuda")
    cb.cb_ess_weights(r.cuda(), p_width, w, alpha)
    torch.cuda.synchronize()
    wo, ao, _ = oracle.ess_weights(r.double().numpy(), p_width)
    np.testing.assert_allclose(alpha.cpu().numpy(), ao, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(w.cpu().numpy(), wo, rtol=2e-6, atol=1e-6)
    wk = w.double().cpu().numpy()
    kish = wk.sum(1) ** 2 / (wk ** 2).sum(1)
    assert (kish >= min(n, 2 * p_width) * (1 - 1e-5)).all()        # the floor holds on the fp32 output too
