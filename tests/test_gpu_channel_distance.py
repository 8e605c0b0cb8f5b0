"""Eq. 5 on the device against the oracle's plain fp64 statement: the distance table at a stated tolerance, and
the map that the builder makes with the nearest-neighbour search on the device.

The product evaluates D(i, j) in float32 (sums of 10^2 .. 10^4 squares: relative error of order 1e-6), the
oracle in fp64 from its own fp64 LayerNorm.  A decision of the matching (which b is nearest to a; which edges are
among the E shortest) is therefore compared only where the oracle's margin exceeds TOL; the decisions inside TOL
are counted and reported, and there the product's choice must be one of the near-tied candidates."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-4      # relative margin below which two Eq. 5 distances count as tied between fp32 and fp64


def _setup(kw):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS["c2"].scaled(M=8, n_outlier=4, **kw)
    g, b = synth.layernorm_params(cfg)
    xc = synth.calibration_tokens(cfg)
    W = synth.weights(cfg)
    y = torch.empty((xc.shape[0], cfg.K), dtype=torch.float32, device=G.DEV)
    B.qllm_layernorm_rows(G.dev_x(xc), G.dev(g), None if b is None else G.dev(b), y, ln_eps=cfg.ln_eps)
    y_ref = oracle.layernorm(xc, g, b, cfg.ln_eps)
    np.testing.assert_allclose(y.cpu().numpy(), y_ref, rtol=2e-5, atol=2e-6)
    return cfg, W, y, y_ref


@pytest.mark.parametrize("kw", [dict(K=256, N=80, calib_tokens=24), dict(K=250, N=33, calib_tokens=37),
                                dict(K=512, N=130, calib_tokens=64)])
def test_distance_table_against_fp64(kw):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg, W, y, y_ref = _setup(kw)
    C = cfg.K
    D = torch.empty((C, C), dtype=torch.float32, device=G.DEV)
    B.qllm_channel_distance(y, G.dev(W), D)
    torch.cuda.synchronize()
    D_ref = oracle.channel_distance(y_ref, W)
    np.testing.assert_allclose(D.cpu().numpy(), D_ref, rtol=2e-5, atol=0)


@pytest.mark.parametrize("kw", [dict(K=256, N=80, calib_tokens=24), dict(K=512, N=130, calib_tokens=64),
                                dict(K=1024, N=272, calib_tokens=128)])
def test_map_from_the_device_search_against_the_oracle(kw):
    from paper_2310_08041_b200 import binding as B
    cfg, W, y, y_ref = _setup(kw)
    C = cfg.K
    absmax = oracle.channel_absmax(y_ref)
    theta = oracle.theta_percentile(absmax, 0.98)
    D = oracle.channel_distance(y_ref, W)                 # fp64, from the oracle's own LayerNorm
    ptr, src, coef, st = oracle.build_map(absmax, theta, dist=D)
    E = st["E"]
    assert E > 0 and st["rounds"] == 1
    h = B.qllm_build_reassembly(absmax, theta, W, w_bits=cfg.w_bits, calib_y=y)
    p2, s2, c2 = h.map()
    # the margins of the oracle's decisions (Appendix A steps 2-3 on its table)
    T = np.maximum(1, np.ceil(absmax.astype(np.float64) / np.float64(theta))).astype(int)
    pos_src = np.repeat(np.arange(C), T)
    elig = [p for p in range(len(pos_src)) if T[pos_src[p]] == 1]
    A = [p for p in elig if p % 2 == 0]
    Bs = np.array([pos_src[p] for p in elig if p % 2 == 1])
    best, near_nearest = [], 0
    for p in A:
        d = np.sort(D[pos_src[p], Bs])
        best.append(d[0])
        near_nearest += int(len(d) > 1 and d[1] - d[0] <= TOL * d[0])
    ranked = np.sort(np.array(best))
    near_rank = int(E < len(ranked) and ranked[E] - ranked[E - 1] <= TOL * ranked[E - 1])
    print(f"C={C}: E={E}, |A|={len(A)}, near-tied nearest neighbours {near_nearest}, near-tied cut {near_rank}")
    if near_nearest == 0 and near_rank == 0:
        assert np.array_equal(p2, ptr) and np.array_equal(s2, src) and np.array_equal(c2, coef)
    else:
        # every merge the product made is one the oracle's table allows within TOL
        assert p2[-1] == ptr[-1] and int((np.diff(p2) > 1).sum()) > 0
        for c in np.nonzero(np.diff(p2) > 1)[0]:
            mem = s2[p2[c]:p2[c + 1]]
            for a in mem[1:]:
                assert D[a, mem[0]] <= D[a, Bs].min() * (1 + TOL)
    wc, ws, wz, wcs = h.weights()
    ref_w = oracle.prepare_weights(W, p2, s2, cfg.w_bits)
    assert np.array_equal(wc, oracle.pack4(ref_w["codes"]) if cfg.w_bits == 4 else ref_w["codes"])
