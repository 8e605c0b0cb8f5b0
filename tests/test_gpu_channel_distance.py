"""Eq. 5 on the device: the distance table bit for bit against the oracle's, then the map built from it."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kw", [dict(K=256, N=80, calib_tokens=24), dict(K=250, N=33, calib_tokens=37),
                                dict(K=512, N=130, calib_tokens=64)])
def test_distance_table_and_map(kw):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS["c2"].scaled(M=8, n_outlier=4, **kw)
    g, b = synth.layernorm_params(cfg)
    xc = synth.calibration_tokens(cfg)
    W = synth.weights(cfg)
    C = cfg.K
    # the layer's input of the calibration tokens, on the device
    y = torch.empty((xc.shape[0], C), dtype=torch.float32, device=G.DEV)
    B.qllm_layernorm_rows(G.dev_x(xc), G.dev(g), None if b is None else G.dev(b), y, ln_eps=cfg.ln_eps)
    y_ref = oracle.layernorm(xc, g, b, cfg.ln_eps)
    np.testing.assert_allclose(y.cpu().numpy(), y_ref, rtol=2e-5, atol=2e-6)
    # the table is defined on float32 inputs in a fixed order: same inputs, same bits
    y_np = y.cpu().numpy()
    D = torch.empty((C, C), dtype=torch.float32, device=G.DEV)
    B.qllm_channel_distance(y, G.dev(W), D)
    torch.cuda.synchronize()
    D_np = D.cpu().numpy()
    D_ref = oracle.channel_distance(y_np, W)
    assert np.array_equal(D_np, D_ref)
    # and the map built from it is the oracle's
    absmax = oracle.channel_absmax(y_np)
    theta = oracle.theta_percentile(absmax, 0.98)
    ptr, src, coef, st = oracle.build_map(absmax, theta, dist=D_ref)
    assert st["E"] > 0
    h = B.qllm_build_reassembly(absmax, theta, W, w_bits=cfg.w_bits, dist=D_np)
    p2, s2, c2 = h.map()
    assert np.array_equal(p2, ptr) and np.array_equal(s2, src) and np.array_equal(c2, coef)
