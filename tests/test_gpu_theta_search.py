"""Adaptive threshold search (Algorithm 1) on the GPU path against the oracle's search."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw,P", [("c1", dict(N=128), 8),
                                       ("c2", dict(M=48, K=512, N=96, n_outlier=4, calib_tokens=0), 6)])
def test_search_matches_oracle(name, kw, P):
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS[name].scaled(**kw)
    x = synth.activations(cfg)
    gamma, beta = synth.layernorm_params(cfg)
    W = synth.weights(cfg)
    absmax = oracle.channel_absmax(oracle.layernorm(x, gamma, beta, cfg.ln_eps))
    ref_theta, ref_losses = oracle.search_theta(x, gamma, beta, cfg.ln_eps, W, absmax, cfg.a_bits, cfg.w_bits, P)
    theta, losses = B.qllm_search_theta(G.dev_x(x), gamma, beta, absmax, W, cfg.a_bits, cfg.w_bits, P, ln_eps=cfg.ln_eps)
    assert B.qllm_poll_status() == 0
    # the same thresholds are feasible on both sides
    assert np.array_equal(np.isfinite(losses), np.isfinite(ref_losses)) and np.isfinite(ref_losses).any()
    fin = np.isfinite(ref_losses)
    # errors: the GPU's fp32 path may flip a few codes inside the flip band and sums the reference product in
    # fp32; both move the error by far less than the spacing between candidates
    np.testing.assert_allclose(losses[fin], ref_losses[fin], rtol=5e-3)
    # the selected threshold is the oracle's unless two candidates are closer than that tolerance
    grid = oracle.theta_grid(absmax, P)
    order = np.argsort(np.where(fin, ref_losses, np.inf), kind="stable")
    if ref_losses[order[1]] > ref_losses[order[0]] * 1.02:
        assert theta == ref_theta
    else:
        assert theta in (float(grid[order[0]]), float(grid[order[1]]))
    print(name, "theta*", theta, "losses", losses)
