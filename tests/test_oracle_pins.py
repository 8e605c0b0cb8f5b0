"""Pins of the CPU oracle against what the paper and the mathematics fix.

Every oracle function is checked against something other than itself: hand-worked
fixtures (tests/golden), closed forms (Eq. 4-5 merge error), exactness claims
(Eq. 3 keeps the layer output), invariants, library routines (numpy) on special
cases, and brute force on tiny inputs.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _records(name):
    """Parse 'key: values' lines of a golden file into a list of (key, [tokens])."""
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":", 1)
            out.append((k.strip(), v.split()))
    return out


# --------------------------------------------------------------------------- O1
def test_layernorm_hand_rows():
    recs = _records("layernorm_hand.txt")
    for (kx, vx), (ky, vy) in zip(recs[0::2], recs[1::2]):
        assert kx == "x" and ky == "y"
        x = np.array([vx], np.float32)
        y = oracle.layernorm(x, np.ones(x.shape[1], np.float32), None, eps=0.0)
        np.testing.assert_allclose(y[0], np.array(vy, np.float64), rtol=1e-14)


def test_layernorm_moments_and_affine():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((5, 64)) * 3 + 7).astype(np.float32)
    g = rng.standard_normal(64).astype(np.float32)
    b = rng.standard_normal(64).astype(np.float32)
    eps = 1e-5
    y1 = oracle.layernorm(x, np.ones(64, np.float32), None, eps)
    # gamma = 1, beta = 0: mean 0, variance var/(var+eps)
    var = x.astype(np.float64).var(axis=1)
    np.testing.assert_allclose(y1.mean(1), 0, atol=1e-14)
    np.testing.assert_allclose(y1.var(1), var / (var + eps), rtol=1e-12)
    # affine part is applied per channel after normalisation
    y2 = oracle.layernorm(x, g, b, eps)
    np.testing.assert_allclose(y2, y1 * g.astype(np.float64) + b.astype(np.float64), rtol=1e-13, atol=1e-13)
    # shift invariance and scale invariance (eps = 0)
    y3 = oracle.layernorm((x * 4).astype(np.float32), g, b, 0.0)
    y4 = oracle.layernorm(x, g, b, 0.0)
    np.testing.assert_allclose(y3, y4, rtol=1e-10, atol=1e-12)


def test_layernorm_bf16_is_widened_exactly():
    rng = np.random.default_rng(2)
    xb = synth.f32_to_bf16_bits(rng.standard_normal((3, 32)).astype(np.float32))
    g = np.ones(32, np.float32)
    y_b = oracle.layernorm(xb, g)
    y_f = oracle.layernorm(synth.bf16_bits_to_f32(xb), g)
    assert np.array_equal(y_b, y_f)


def test_channel_absmax_matches_numpy():
    y = np.random.default_rng(3).standard_normal((17, 9))
    np.testing.assert_array_equal(oracle.channel_absmax(y), np.abs(y).max(0).astype(np.float32))


# --------------------------------------------------------------------------- O2 / O4
def _disassembly_only_map(T):
    """Expanded map of Eq. 3 without any assembly: channel i -> T_i rows (i, 1/T_i)."""
    src = np.repeat(np.arange(len(T)), T).astype(np.int32)
    coef = np.repeat(1.0 / np.asarray(T, np.float64), T).astype(np.float32)
    ptr = np.arange(len(src) + 1, dtype=np.int32)
    return ptr, src, coef


def test_disassembly_preserves_layer_output():
    """Eq. 3: splitting channels and duplicating weight rows leaves X W unchanged."""
    rng = np.random.default_rng(4)
    C, N, M = 24, 10, 7
    X = rng.standard_normal((M, C))
    X[:, [3, 17]] *= 50
    W = rng.standard_normal((N, C)).astype(np.float32)
    T = np.ones(C, np.int64); T[3] = 4; T[17] = 8      # powers of two: coefficients exact in float
    ptr, src, coef = _disassembly_only_map(T)
    Xr = oracle.map_apply(X, ptr, src, coef)
    Wr = oracle.weight_transform(W, ptr, src)
    assert Xr.shape == (M, C + 10) and Wr.shape == (N, C + 10)
    ref = oracle.dense_linear(X, W.astype(np.float64))
    got = oracle.dense_linear(Xr, Wr)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-12
    # non power-of-two split counts: float(1/T) rounding only
    T[3] = 3; T[17] = 7
    ptr, src, coef = _disassembly_only_map(T)
    got = oracle.dense_linear(oracle.map_apply(X, ptr, src, coef), oracle.weight_transform(W, ptr, src))
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    # reduces to numpy on the dense map matrix P (rows = output channels)
    P = np.zeros((len(src), C)); P[np.arange(len(src)), src] = coef.astype(np.float64)
    np.testing.assert_allclose(oracle.map_apply(X, ptr, src, coef), X @ P.T, rtol=1e-13, atol=1e-13)
    S = (P != 0).astype(np.float64)
    np.testing.assert_allclose(P.T @ S, np.eye(C), atol=1e-7)   # the pattern undoes the split


def test_single_merge_closed_form():
    """Eq. 4-5: merging channels i, j changes X W by (x_i - x_j)(W_i - W_j)/2, so
    ||XW - X'W'||_F^2 = 1/4 ||x_i - x_j||^2 ||W_i - W_j||^2; identical channels merge exactly."""
    rng = np.random.default_rng(5)
    C, N, M = 12, 6, 9
    X = rng.standard_normal((M, C))
    W = rng.standard_normal((N, C)).astype(np.float32)
    i, j = 2, 7
    rows = [[c] for c in range(C) if c not in (i, j)] + [[j, i]]
    ptr = np.cumsum([0] + [len(r) for r in rows]).astype(np.int32)
    src = np.concatenate(rows).astype(np.int32)
    coef = np.concatenate([[1.0 / len(r)] * len(r) for r in rows]).astype(np.float32)
    Xr = oracle.map_apply(X, ptr, src, coef)
    Wr = oracle.weight_transform(W, ptr, src)
    ref = oracle.dense_linear(X, W.astype(np.float64))
    got = oracle.dense_linear(Xr, Wr)
    lhs = np.linalg.norm(ref - got) ** 2
    W64 = W.astype(np.float64)
    rhs = 0.25 * np.linalg.norm(X[:, i] - X[:, j]) ** 2 * np.linalg.norm(W64[:, i] - W64[:, j]) ** 2
    assert abs(lhs - rhs) <= 1e-10 * rhs
    X2 = X.copy(); X2[:, j] = X2[:, i]
    got2 = oracle.dense_linear(oracle.map_apply(X2, ptr, src, coef), Wr)
    ref2 = oracle.dense_linear(X2, W64)
    assert np.linalg.norm(got2 - ref2) <= 1e-12 * np.linalg.norm(ref2)


def test_low_rank_fold_matches_numpy():
    rng = np.random.default_rng(6)
    C, N, r = 10, 5, 4
    W = rng.standard_normal((N, C)).astype(np.float32)
    A = rng.standard_normal((C, r)).astype(np.float32)
    B = rng.standard_normal((r, N)).astype(np.float32)
    ptr = np.arange(C + 1, dtype=np.int32); src = np.arange(C, dtype=np.int32)
    got = oracle.weight_transform(W, ptr, src, A, B)
    ref = W.astype(np.float64) + (A.astype(np.float64) @ B.astype(np.float64)).T
    np.testing.assert_allclose(got, ref, rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------- O3
def test_quantizer_hand_cases():
    recs = _records("quant_hand.txt")
    assert len(recs) % 5 == 0
    for i in range(0, len(recs), 5):
        d = {k: v for k, v in recs[i:i + 5]}
        bits = int(d["bits"][0])
        x = np.array([d["x"]], np.float64)
        q = oracle.quant_rows(x, bits)
        assert q["scale"][0] == np.float32(d["alpha"][0])
        assert q["zero"][0] == np.float32(d["beta"][0])
        assert q["codes"][0].tolist() == [int(t) for t in d["q"]]
        assert q["sum"][0] == sum(int(t) for t in d["q"])


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_quantizer_grid_round_trip(bits):
    """Values on the code grid alpha (q - beta), alpha a power of two, come back exactly."""
    rng = np.random.default_rng(7 + bits)
    qmax = (1 << bits) - 1
    R, C = 6, 80
    for alpha, beta in [(0.25, 5), (2.0 ** -7, 0), (8.0, qmax), (1.0, -40), (0.5, qmax + 9)]:
        q = rng.integers(0, qmax + 1, size=(R, C))
        q[:, 0] = 0; q[:, 1] = qmax
        x = alpha * (q - beta).astype(np.float64)
        out = oracle.quant_rows(x, bits)
        assert np.array_equal(out["codes"], q.astype(np.uint8))
        assert np.all(out["scale"] == np.float32(alpha))
        assert np.all(out["zero"] == np.float32(beta))
        assert np.array_equal(out["sum"], q.sum(1).astype(np.int32))


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_quantizer_error_bound_and_ties(bits):
    rng = np.random.default_rng(17 + bits)
    qmax = (1 << bits) - 1
    x = rng.standard_normal((8, 300)) * rng.uniform(0.1, 30, size=(8, 1)) + rng.uniform(-3, 3, size=(8, 1))
    out = oracle.quant_rows(x, bits, want_pre=True)
    a = out["scale"].astype(np.float64)[:, None]
    z = out["zero"].astype(np.float64)[:, None]
    codes = out["codes"].astype(np.float64)
    assert codes.min() >= 0 and codes.max() <= qmax
    err = np.abs(x - a * (codes - z))
    unclamped = (np.rint(out["pre"]) + z >= 0) & (np.rint(out["pre"]) + z <= qmax)
    assert np.all(err[unclamped] <= a.repeat(300, 1)[unclamped] * 0.5 * (1 + 1e-9))
    assert np.all(err <= 1.5 * a * (1 + 1e-9))
    assert np.all(out["codes"].min(1) <= 1) and np.all(out["codes"].max(1) >= qmax - 1)
    # ties go to even: 0.5 -> 0, 1.5 -> 2, 2.5 -> 2  (alpha = 1, beta = 0)
    t = np.array([[0.0, 0.5, 1.5, 2.5, float(qmax)]])
    assert oracle.quant_rows(t, bits)["codes"][0].tolist() == [0, 0, 2, 2, qmax]


def test_quantizer_constant_rows():
    for v in (0.0, 3.5, -2.25):
        out = oracle.quant_rows(np.full((1, 5), v), 4)
        a, z, q = float(out["scale"][0]), float(out["zero"][0]), out["codes"][0].astype(np.float64)
        assert np.all(q == 0)
        assert np.all(a * (q - z) == v)


def test_pack4_layout():
    c = np.array([[1, 2, 15, 0, 7, 9]], np.uint8)
    assert oracle.pack4(c)[0].tolist() == [0x21, 0x0F, 0x97]
    assert np.array_equal(oracle.pack4(c), synth.pack_nibbles(c))


# --------------------------------------------------------------------------- O5
def test_int_matmul_brute_force():
    rng = np.random.default_rng(8)
    M, N, K = 5, 7, 16
    qa = rng.integers(0, 16, (M, K), dtype=np.uint8)
    qw = rng.integers(0, 16, (N, K), dtype=np.uint8)
    ref = [[sum(int(qa[m, k]) * int(qw[n, k]) for k in range(K)) for n in range(N)] for m in range(M)]
    assert oracle.int_matmul(qa, qw).tolist() == ref
    # library routine on a larger case; extremes; sampled variant
    qa = rng.integers(0, 256, (9, 200), dtype=np.uint8); qw = rng.integers(0, 256, (11, 200), dtype=np.uint8)
    full = oracle.int_matmul(qa, qw)
    assert np.array_equal(full, qa.astype(np.int64) @ qw.astype(np.int64).T)
    ms = np.array([0, 8, 3, 3]); ns = np.array([10, 0, 5, 6])
    assert np.array_equal(oracle.int_matmul_at(qa, qw, ms, ns), full[ms, ns])
    ones = np.full((2, 64), 255, np.uint8)
    assert np.all(oracle.int_matmul(ones, ones) == 64 * 255 * 255)


@pytest.mark.parametrize("bits", [4, 6])
def test_epilogue_is_the_dense_product_of_dequantized_operands(bits):
    rng = np.random.default_rng(9 + bits)
    M, N, K = 6, 8, 48
    qmax = (1 << bits) - 1
    qa = rng.integers(0, qmax + 1, (M, K), dtype=np.uint8)
    qw = rng.integers(0, qmax + 1, (N, K), dtype=np.uint8)
    a_s = rng.uniform(0.01, 1, M).astype(np.float32); w_s = rng.uniform(0.001, 0.1, N).astype(np.float32)
    a_z = rng.integers(-3, qmax + 3, M).astype(np.float32); w_z = rng.integers(0, qmax + 1, N).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    acc = oracle.int_matmul(qa, qw)
    out = oracle.epilogue(acc, K, a_s, a_z, qa.sum(1, dtype=np.int32), w_s, w_z, qw.sum(1, dtype=np.int32), bias)
    A = a_s.astype(np.float64)[:, None] * (qa.astype(np.float64) - a_z.astype(np.float64)[:, None])
    Wd = w_s.astype(np.float64)[:, None] * (qw.astype(np.float64) - w_z.astype(np.float64)[:, None])
    ref = A @ Wd.T + bias.astype(np.float64)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-12)
    out0 = oracle.epilogue(acc, K, a_s, a_z, qa.sum(1, dtype=np.int32), w_s, w_z, qw.sum(1, dtype=np.int32), None)
    np.testing.assert_allclose(out0, A @ Wd.T, rtol=1e-12, atol=1e-12)


def test_casts():
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -3.14159, 1e-3, 65504.0, 0.0])
    b = oracle.cast_bf16(v)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 is a tie -> 1 + 2^-6
    assert b[0] == 0x3F80 and b[1] == 0x3F80 and b[2] == 0x3F82
    back = synth.bf16_bits_to_f32(b).astype(np.float64)
    assert np.all(np.abs(back - v) <= np.abs(v) * 2.0 ** -8)
    # agrees with the float32 route when no double rounding is involved
    r = np.random.default_rng(10).standard_normal(1000).astype(np.float32)
    assert np.array_equal(oracle.cast_bf16(r.astype(np.float64)), synth.f32_to_bf16_bits(r))
    assert np.array_equal(oracle.cast_f32(v), v.astype(np.float32))


# --------------------------------------------------------------------------- O6 + thresholds
def _frac(tok):
    n, d = tok.split("/")
    return np.float32(float(Fraction(int(n), int(d))))


def test_builder_hand_cases():
    recs = _records("matching_hand.txt")
    i = 0
    seen = 0
    while i < len(recs):
        assert recs[i][0] == "absmax" and recs[i + 1][0] == "theta"
        absmax = np.array(recs[i][1], np.float32)
        theta = float(recs[i + 1][1][0])
        if recs[i + 2][0] == "infeasible":
            with pytest.raises(oracle.Infeasible):
                oracle.build_map(absmax, theta)
            i += 3
        else:
            d = {k: v for k, v in recs[i + 2:i + 6]}
            ptr, src, coef, st = oracle.build_map(absmax, theta)
            assert ptr.tolist() == [int(t) for t in d["ptr"]]
            assert src.tolist() == [int(t) for t in d["src"]]
            assert coef.tolist() == [_frac(t) for t in d["coef"]]
            assert st["rounds"] == int(d["rounds"][0])
            i += 6
        seen += 1
    assert seen == 3


def _check_map_invariants(absmax, theta, ptr, src, coef, st):
    C = len(absmax)
    T = np.maximum(1, np.ceil(absmax.astype(np.float64) / np.float64(np.float32(theta)))).astype(np.int64)
    E = int((T - 1).sum())
    assert st["E"] == E
    assert len(ptr) == C + 1 and ptr[0] == 0 and ptr[-1] == len(src) == C + E
    lens = np.diff(ptr)
    assert lens.min() >= 1
    assert np.array_equal(np.bincount(src, minlength=C), T)          # channel i appears T_i times
    assert np.all(T * np.float64(np.float32(theta)) >= absmax)       # sub-channel maxima <= theta
    P = np.zeros((C, C)); np.add.at(P, (np.repeat(np.arange(C), lens), src), coef.astype(np.float64))
    for c in range(C):
        members = src[ptr[c]:ptr[c + 1]]
        if lens[c] > 1:
            assert np.all(T[members] == 1)                           # sub-channels are never merged
            assert len(set(members.tolist())) == lens[c]
            assert np.all(coef[ptr[c]:ptr[c + 1]] == np.float32(1.0 / lens[c]))
            assert abs(P[c].sum() - 1) < 1e-6
        else:
            assert coef[ptr[c]] == np.float32(1.0 / T[members[0]])
    colsum = P.sum(0)
    merged_src = np.zeros(C, bool)
    for c in np.nonzero(lens > 1)[0]:
        merged_src[src[ptr[c]:ptr[c + 1]]] = True
    assert np.allclose(colsum[~merged_src], 1, atol=1e-5)            # untouched and disassembled
    assert st["merged_rows"] == int((lens > 1).sum())
    assert int((lens - 1).sum()) == E                                # E members were merged away


def test_builder_invariants_on_synthetic_layers():
    for name, K in (("c1", None), ("c2", 1024), ("c5", 2048)):
        cfg = synth.CONFIGS[name]
        if K:
            cfg = cfg.scaled(K=K, n_outlier=max(2, cfg.n_outlier * K // cfg.K))
        g, b = synth.layernorm_params(cfg)
        absmax = oracle.channel_absmax(oracle.layernorm(synth.calibration_tokens(cfg), g, b, cfg.ln_eps))
        theta = oracle.theta_for_extra(absmax, 8) if cfg.theta_rule == "extra8" else oracle.theta_percentile(absmax, 0.99)
        ptr, src, coef, st = oracle.build_map(absmax, theta)
        if cfg.theta_rule == "extra8":
            assert st["E"] == 8 and st["merged_rows"] >= 1
        _check_map_invariants(absmax, theta, ptr, src, coef, st)


def test_builder_picks_nearest_and_shortest_edges():
    """Brute-force statement of Appendix A steps 2-3 on a single-round case."""
    rng = np.random.default_rng(11)
    C = 40
    absmax = rng.uniform(0.5, 2.0, C).astype(np.float32)
    absmax[[5, 22]] = [9.0, 14.0]
    theta = 2.5
    ptr, src, coef, st = oracle.build_map(absmax, theta)
    assert st["rounds"] == 1
    T = np.maximum(1, np.ceil(absmax / np.float32(theta))).astype(int)
    pos_src = np.repeat(np.arange(C), T)
    elig = [p for p in range(len(pos_src)) if T[pos_src[p]] == 1]
    A = [p for p in elig if p % 2 == 0]; B = [p for p in elig if p % 2 == 1]
    edges = []
    for a in A:
        d = [abs(float(absmax[pos_src[a]]) - float(absmax[pos_src[b]])) for b in B]
        edges.append((min(d), a, B[int(np.argmin(d))]))
    edges.sort()
    kept = edges[:st["E"]]
    merged = {}
    for _, a, b in sorted(kept, key=lambda e: e[1]):
        merged.setdefault(b, [pos_src[b]]).append(pos_src[a])
    gone = {a for _, a, _ in kept}
    rows = [merged.get(p, [pos_src[p]]) for p in range(len(pos_src)) if p not in gone]
    assert [src[ptr[c]:ptr[c + 1]].tolist() for c in range(C)] == [list(map(int, r)) for r in rows]


def test_theta_helpers():
    rng = np.random.default_rng(12)
    a = rng.uniform(0.1, 5, 257).astype(np.float32)
    for pct in (0.5, 0.9, 0.99, 1.0):
        assert oracle.theta_percentile(a, pct) == np.float32(np.percentile(a, pct * 100, method="inverted_cdf"))
    for extra in (1, 8, 33):
        th = oracle.theta_for_extra(a, extra)
        assert th > 0
        T = np.maximum(1, np.ceil(a.astype(np.float64) / np.float64(np.float32(th))))
        assert int((T - 1).sum()) == extra == oracle.extra_channels(a, th)
    # T rule of Sec. 4.1.1: below theta unchanged, above split by ceil
    assert oracle.extra_channels(np.array([1.0, 2.0, 2.0001, 7.9, 0.0], np.float32), 2.0) == 0 + 0 + 1 + 3 + 0


# ---------------------------------------------------------------------------
# Adaptive threshold search (Algorithm 1)
# ---------------------------------------------------------------------------
def _search_case(seed=7, T=24, C=64, N=40):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, C)).astype(np.float32)
    x[:, [3, 17]] *= 30.0
    gamma = (1 + 0.1 * rng.standard_normal(C)).astype(np.float32)
    W = (0.05 * rng.standard_normal((N, C))).astype(np.float32)
    absmax = oracle.channel_absmax(oracle.layernorm(x, gamma, None, 1e-5))
    return x, gamma, W, absmax


def test_theta_grid_closed_form():
    """Algorithm 1: P evenly spaced thresholds ending at max(m); the first lies one step above min(m)."""
    m = np.array([0.5, 4.0, 1.25, 2.0], np.float32)
    g = oracle.theta_grid(m, 7)
    assert g.shape == (7,) and g[-1] == np.float32(4.0)
    np.testing.assert_allclose(np.diff(g.astype(np.float64)), 0.5, rtol=1e-6)
    assert g[0] == np.float32(1.0)


def test_reassembly_loss_without_outlier_channels_is_plain_quantization_error():
    """At theta = max(m) every T_i = 1, the map is the identity, and the loss reduces to the error of
    quantizing both operands: recomputed here from the dequantized operands with numpy."""
    x, gamma, W, absmax = _search_case()
    theta = float(absmax.max())
    ptr, src, coef, st = oracle.build_map(absmax, theta)
    assert st["E"] == 0 and np.array_equal(src, np.arange(len(absmax)))
    y = oracle.layernorm(x, gamma, None, 1e-5)
    qa = oracle.quant_rows(y, 4)
    qw = oracle.quant_rows(W.astype(np.float64), 4)
    A = qa["scale"].astype(np.float64)[:, None] * (qa["codes"].astype(np.float64) - qa["zero"].astype(np.float64)[:, None])
    Wd = qw["scale"].astype(np.float64)[:, None] * (qw["codes"].astype(np.float64) - qw["zero"].astype(np.float64)[:, None])
    want = float(((y @ W.astype(np.float64).T - A @ Wd.T) ** 2).sum())
    got = oracle.reassembly_loss(x, gamma, None, 1e-5, W, absmax, theta, 4, 4)
    assert abs(got - want) <= 1e-9 * want


def test_search_theta_is_the_first_minimum_of_the_grid_losses():
    x, gamma, W, absmax = _search_case()
    P = 9
    theta, losses = oracle.search_theta(x, gamma, None, 1e-5, W, absmax, 4, 4, P)
    grid = oracle.theta_grid(absmax, P)
    assert losses.shape == (P,)
    finite = np.isfinite(losses)
    assert finite[-1]                                   # theta = max(m) never needs assembly
    best = min(range(P), key=lambda p: (losses[p], p))  # brute force with the tie rule of Algorithm 1
    assert theta == float(grid[best])
    # every finite loss is reproduced by evaluating its grid point on its own
    for p in np.nonzero(finite)[0][:3]:
        assert losses[p] == oracle.reassembly_loss(x, gamma, None, 1e-5, W, absmax, float(grid[p]), 4, 4)
    # splitting the outlier channels helps on this input: some interior threshold beats "no reassembly"
    assert losses[best] < losses[-1]


# ---------------------------------------------------------------------------
# Appendix B: reassembly folded into a preceding linear layer
# ---------------------------------------------------------------------------
def test_fold_previous_closed_forms_and_function_preservation():
    """Appendix B's two rules on a hand-made map (channel 1 split in T = 3, channels 2 and 4 merged), then
    the defining property: the folded layer's output equals the map applied to the original output."""
    rng = np.random.default_rng(5)
    C_src, C_in = 5, 7
    Wp = rng.standard_normal((C_src, C_in)).astype(np.float32)
    bp = rng.standard_normal(C_src).astype(np.float32)
    third = np.float32(1.0 / 3.0)
    rows = [[(0, 1.0)], [(1, third)], [(1, third)], [(1, third)], [(2, 0.5), (4, 0.5)]]   # 5 rows: 3 stays out
    ptr = np.array([0, 1, 2, 3, 4, 6], np.int32)
    src = np.array([s for r in rows for s, _ in r], np.int32)
    coef = np.array([c for r in rows for _, c in r], np.float32)
    Wo, bo = oracle.fold_previous(Wp, bp, ptr, src, coef)
    assert np.array_equal(Wo[0], Wp[0])                                             # untouched channel
    for c in (1, 2, 3):                                                             # W / T
        np.testing.assert_allclose(Wo[c], Wp[1].astype(np.float64) * float(third), rtol=1e-7)
    np.testing.assert_allclose(Wo[4], (Wp[2].astype(np.float64) + Wp[4]) / 2, rtol=1e-7)   # (W_i + W_j) / 2
    np.testing.assert_allclose(bo[4], (float(bp[2]) + float(bp[4])) / 2, rtol=1e-6)
    X = rng.standard_normal((9, C_in))
    y_prev = X @ Wp.astype(np.float64).T + bp
    want = oracle.map_apply(y_prev, ptr, src, coef)
    got = X @ Wo.astype(np.float64).T + bo
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)                        # fp32 storage of the rows


# ---------------------------------------------------------------------------
# Eq. 5: distance between channels, and the builder driven by it
# ---------------------------------------------------------------------------
def _eq5_case(seed=21, T=20, C=24, N=18):
    rng = np.random.default_rng(seed)
    y = rng.standard_normal((T, C)).astype(np.float32)
    W = (0.2 * rng.standard_normal((N, C))).astype(np.float32)
    return y, W


def test_channel_distance_is_eq5_and_equals_the_error_of_the_merge():
    y, W = _eq5_case()
    D = oracle.channel_distance(y, W)
    C = y.shape[1]
    y64, W64 = y.astype(np.float64), W.astype(np.float64)
    ref = np.array([[0.25 * ((y64[:, i] - y64[:, j]) ** 2).sum() * ((W64[:, i] - W64[:, j]) ** 2).sum()
                     for j in range(C)] for i in range(C)])
    np.testing.assert_allclose(D, ref, rtol=1e-12, atol=0)
    assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0)
    # Eq. 5 is the output error of assembling the two channels (Eq. 4): build that map by hand and measure it
    i, j = 3, 10
    rows = [[c] for c in range(C) if c != j]
    rows[i] = [i, j]
    rows.append([j])                                    # keep C rows: channel j again as its own row, then drop its effect
    ptr = np.zeros(C + 1, np.int32); ptr[1:] = np.cumsum([len(r) for r in rows])
    src = np.array([s for r in rows for s in r], np.int32)
    coef = np.array([1.0 / len(r) for r in rows for _ in r], np.float32)
    xr = oracle.map_apply(y64, ptr, src, coef)[:, :C - 1]            # the C - 1 assembled channels
    Wr = oracle.weight_transform(W, ptr, src)[:, :C - 1]
    err = ((y64 @ W64.T - xr @ Wr.T) ** 2).sum()
    assert abs(err - ref[i, j]) <= 1e-9 * ref[i, j]


def test_builder_with_a_distance_table():
    """With the table |m_i - m_j| the table-driven builder is the plain one (integer maxima keep the table exact);
    with an Eq. 5 table it follows the brute-force statement of Appendix A steps 2-3 on that table."""
    rng = np.random.default_rng(22)
    C = 36
    absmax = rng.integers(1, 9, C).astype(np.float32)
    absmax[[4, 19]] = [40.0, 23.0]
    theta = 9.0
    table = np.abs(absmax[:, None] - absmax[None, :]).astype(np.float32)
    a = oracle.build_map(absmax, theta)
    b = oracle.build_map(absmax, theta, dist=table)
    assert a[3]["rounds"] == 1 and all(np.array_equal(u, v) for u, v in zip(a[:3], b[:3]))
    y, W = _eq5_case(seed=23, C=C)
    D = oracle.channel_distance(y, W)
    ptr, src, coef, st = oracle.build_map(absmax, theta, dist=D)
    T = np.maximum(1, np.ceil(absmax / np.float32(theta))).astype(int)
    pos_src = np.repeat(np.arange(C), T)
    elig = [p for p in range(len(pos_src)) if T[pos_src[p]] == 1]
    A = [p for p in elig if p % 2 == 0]; B = [p for p in elig if p % 2 == 1]
    edges = []
    for p in A:
        d = [float(D[pos_src[p], pos_src[q]]) for q in B]
        edges.append((min(d), p, B[int(np.argmin(d))]))
    edges.sort()
    kept = edges[:st["E"]]
    merged = {}
    for _, p, q in sorted(kept, key=lambda e: e[1]):
        merged.setdefault(q, [pos_src[q]]).append(pos_src[p])
    gone = {p for _, p, _ in kept}
    rows = [merged.get(p, [pos_src[p]]) for p in range(len(pos_src)) if p not in gone]
    assert [src[ptr[c]:ptr[c + 1]].tolist() for c in range(C)] == [list(map(int, r)) for r in rows]
    _check_map_invariants(absmax, theta, ptr, src, coef, st)
    # a threshold that needs a second round has no Eq. 5 reading
    big = absmax.copy()
    big[4] = 200.0                                      # 24 extra channels against 17 candidates in the first round
    assert oracle.build_map(big, theta)[3]["rounds"] > 1
    with pytest.raises(oracle.NeedsMoreRounds):
        oracle.build_map(big, theta, dist=D)
