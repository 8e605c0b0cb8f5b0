"""Host builder of the library against the oracle's builder: identical integer arrays,
bit-equal coefficients, identical weight codes / scales / zero-points / column sums."""
import os

import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import binding as B
from paper_2310_08041_b200 import synth

from test_oracle_pins import _records, _frac


def _absmax(cfg):
    g, b = synth.layernorm_params(cfg)
    return oracle.channel_absmax(oracle.layernorm(synth.calibration_tokens(cfg), g, b, cfg.ln_eps))


def _theta(cfg, absmax, use_lib):
    if cfg.theta_rule == "extra8":
        return B.qllm_theta_for_extra(absmax, 8) if use_lib else oracle.theta_for_extra(absmax, 8)
    return B.qllm_theta_percentile(absmax, 0.99) if use_lib else oracle.theta_percentile(absmax, 0.99)


CASES = [
    ("c1", {}),
    ("c2", dict(K=1024, N=96, n_outlier=5)),
    ("c4", dict(K=640, N=64, n_outlier=4)),
    ("c5", dict(K=2048, N=48, n_outlier=10)),
]


@pytest.mark.parametrize("name,kw", CASES)
def test_builder_matches_oracle(name, kw):
    cfg = synth.CONFIGS[name].scaled(**kw)
    absmax = _absmax(cfg)
    th_o, th_l = _theta(cfg, absmax, False), _theta(cfg, absmax, True)
    assert th_o == th_l and th_o > 0
    W = synth.weights(cfg)
    A, Bm = synth.low_rank(cfg)
    ptr, src, coef, st = oracle.build_map(absmax, th_o)
    ow = oracle.prepare_weights(W, ptr, src, cfg.w_bits, A, Bm)
    h = B.qllm_build_reassembly(absmax, th_l, W, A, Bm, cfg.w_bits)
    lp, ls, lc = h.map()
    assert np.array_equal(lp, ptr) and np.array_equal(ls, src)
    assert np.array_equal(lc.view(np.uint32), coef.view(np.uint32))
    s = h.stats()
    assert (s["E"], s["merged_rows"], s["rounds"]) == (st["E"], st["merged_rows"], st["rounds"])
    assert st["E"] > 0
    wc, ws, wz, wcs = h.weights()
    ocodes = oracle.pack4(ow["codes"]) if cfg.w_bits == 4 else ow["codes"]
    assert np.array_equal(wc, ocodes)
    assert np.array_equal(ws.view(np.uint32), ow["scale"].view(np.uint32))
    assert np.array_equal(wz, ow["zero"]) and np.array_equal(wcs, ow["colsum"])
    assert B.qllm_validate_map(lp, ls, cfg.K) == B.QLLM_OK


def test_builder_hand_cases_and_ties():
    recs = _records("matching_hand.txt")
    i = 0
    while i < len(recs):
        absmax = np.array(recs[i][1], np.float32)
        theta = float(recs[i + 1][1][0])
        W = np.ones((2, len(absmax)), np.float32)
        if recs[i + 2][0] == "infeasible":
            with pytest.raises(B.QllmError) as e:
                B.qllm_build_reassembly(absmax, theta, W, w_bits=8)
            assert e.value.status == B.QLLM_ERR_INFEASIBLE
            i += 3
            continue
        d = {k: v for k, v in recs[i + 2:i + 6]}
        h = B.qllm_build_reassembly(absmax, theta, W, w_bits=8)
        p, s, c = h.map()
        assert p.tolist() == [int(t) for t in d["ptr"]] and s.tolist() == [int(t) for t in d["src"]]
        assert c.tolist() == [_frac(t) for t in d["coef"]]
        assert h.stats()["rounds"] == int(d["rounds"][0])
        i += 6
    # many exact ties (quantised maxima): sorted search must agree with the exhaustive search
    rng = np.random.default_rng(21)
    for trial in range(20):
        C = int(rng.integers(16, 200))
        absmax = (rng.integers(1, 12, C) * 0.25).astype(np.float32)
        absmax[rng.integers(0, C, 3)] *= rng.integers(4, 30)
        theta = float(rng.uniform(2.8, 6.0))
        W = np.ones((1, C), np.float32)
        try:
            ptr, src, coef, st = oracle.build_map(absmax, theta)
        except oracle.Infeasible:
            with pytest.raises(B.QllmError):
                B.qllm_build_reassembly(absmax, theta, W, w_bits=8)
            continue
        h = B.qllm_build_reassembly(absmax, theta, W, w_bits=8)
        p, s, c = h.map()
        assert np.array_equal(p, ptr) and np.array_equal(s, src) and np.array_equal(c, coef), trial
        assert h.stats()["rounds"] == st["rounds"]


def test_theta_helpers_match():
    rng = np.random.default_rng(22)
    a = rng.uniform(0.1, 5, 300).astype(np.float32)
    for pct in (0.5, 0.99, 1.0):
        assert B.qllm_theta_percentile(a, pct) == oracle.theta_percentile(a, pct)
    for extra in (1, 8, 50):
        assert B.qllm_theta_for_extra(a, extra) == oracle.theta_for_extra(a, extra)
    assert B.qllm_theta_for_extra(np.array([1.0, 1.0], np.float32), 1) == 0.0   # empty interval


def test_builder_with_eq5_table_matches_oracle():
    """Host builder driven by a distance table (here the oracle's Eq. 5 table, rounded to the float32 the builder
    takes) against the oracle's table-driven builder."""
    cfg = synth.CONFIGS["c2"].scaled(M=32, K=256, N=48, n_outlier=4, calib_tokens=24)
    g, b = synth.layernorm_params(cfg)
    y = oracle.layernorm(synth.calibration_tokens(cfg), g, b, cfg.ln_eps)
    absmax = oracle.channel_absmax(y)
    W = synth.weights(cfg)
    D = oracle.channel_distance(y, W).astype(np.float32)   # the table the product's builder takes is float32: both sides get these values
    theta = oracle.theta_percentile(absmax, 0.97)
    ptr, src, coef, st = oracle.build_map(absmax, theta, dist=D)
    assert st["E"] > 0 and st["rounds"] == 1
    plain = oracle.build_map(absmax, theta)
    assert not np.array_equal(plain[1], src)             # the Eq. 5 table picks other partners than |m_a - m_b|
    h = B.qllm_build_reassembly(absmax, theta, W, w_bits=4, dist=D)
    p2, s2, c2 = h.map()
    assert np.array_equal(p2, ptr) and np.array_equal(s2, src) and np.array_equal(c2, coef)
    ref_w = oracle.prepare_weights(W, ptr, src, 4)
    wc, ws, wz, wcs = h.weights()
    assert np.array_equal(wc, oracle.pack4(ref_w["codes"])) and np.array_equal(ws, ref_w["scale"])
    # one round only: a threshold that needs two is refused
    big = absmax.copy()
    big[int(np.argmax(absmax))] *= 60.0
    with pytest.raises(oracle.NeedsMoreRounds):
        oracle.build_map(big, theta, dist=D)
    with pytest.raises(B.QllmError):
        B.qllm_build_reassembly(big, theta, W, w_bits=4, dist=D)
    # a row of the table without a finite distance is refused, not indexed with
    bad = D.copy()
    bad[:, :] = np.inf
    with pytest.raises(B.QllmError) as e:
        B.qllm_build_reassembly(absmax, theta, W, w_bits=4, dist=bad)
    assert e.value.status == B.QLLM_ERR_MAP
