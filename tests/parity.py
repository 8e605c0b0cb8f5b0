"""Helpers shared by the GPU parity tests: oracle-side preparation of a synthetic layer and
the comparison rules.

Rules (per the acceptance criteria of the path):
  * int32 accumulators: bit-exact given identical codes;
  * activation codes: bit-exact except +-1 flips where the oracle's pre-round quotient lies
    within 1e-4 of a rounding boundary, at most 1e-4 of the entries; a row whose zero-point
    differs by +-1 because the oracle's min/alpha is within 1e-4 of a boundary counts as one
    row flip and its codes are compared relative to the zero-point;
  * fp32 outputs: relative Frobenius error <= 1e-5 given identical codes; bf16: <= 1 ULP.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2310_08041_b200 import synth

FLIP_BAND = 1e-4        # distance of the oracle's pre-round value to a rounding boundary
FLIP_FRACTION = 1e-4    # allowed share of flipped entries
SCALE_RTOL = 2e-5       # a_scale: fp32 LayerNorm / min-max against the fp64 oracle


def oracle_layer(cfg: synth.LayerConfig, with_weights=True):
    """Everything the oracle derives offline for a synthetic layer."""
    gamma, beta = synth.layernorm_params(cfg)
    ycal = oracle.layernorm(synth.calibration_tokens(cfg), gamma, beta, cfg.ln_eps)
    absmax = oracle.channel_absmax(ycal)
    theta = oracle.theta_for_extra(absmax, 8) if cfg.theta_rule == "extra8" else oracle.theta_percentile(absmax, 0.99)
    ptr, src, coef, stats = oracle.build_map(absmax, theta)
    out = dict(cfg=cfg, gamma=gamma, beta=beta, absmax=absmax, theta=theta, ptr=ptr, src=src, coef=coef, stats=stats)
    if with_weights:
        W = synth.weights(cfg)
        A, B = synth.low_rank(cfg)
        w = oracle.prepare_weights(W, ptr, src, cfg.w_bits, A, B)
        out.update(W=W, lrA=A, lrB=B, w_codes=w["codes"], w_scale=w["scale"], w_zero=w["zero"], w_colsum=w["colsum"])
        out["w_packed"] = oracle.pack4(w["codes"]) if cfg.w_bits == 4 else w["codes"]
    return out


def unpack_codes(stored: np.ndarray, bits: int) -> np.ndarray:
    return synth.unpack_nibbles(stored) if bits == 4 else stored


def check_activation_codes(got_codes, got_scale, got_zero, got_rowsum, ref, bits):
    """got_*: numpy copies of the GPU outputs (codes one per byte).  ref: oracle.quant_rows(...,
    want_pre=True).  Returns dict(flips, row_flips, entries); raises AssertionError on violation."""
    qmax = (1 << bits) - 1
    R, C = ref["codes"].shape
    assert got_codes.shape == (R, C)
    np.testing.assert_allclose(got_scale, ref["scale"], rtol=SCALE_RTOL, atol=0)
    dz = got_zero.astype(np.int64) - ref["zero"].astype(np.int64)
    zfrac = np.abs(np.abs(ref["zpre"] - np.floor(ref["zpre"])) - 0.5)
    bad_rows = np.nonzero(dz != 0)[0]
    for r in bad_rows:
        assert abs(dz[r]) == 1 and zfrac[r] <= FLIP_BAND, f"zero-point of row {r}: {got_zero[r]} vs {ref['zero'][r]}"
    # compare relative to the zero-point on flipped rows (interior codes only: the clamp
    # positions move with the zero-point)
    g = got_codes.astype(np.int64)
    o = ref["codes"].astype(np.int64)
    diff = g - o
    if len(bad_rows):
        diff[bad_rows] -= dz[bad_rows, None]
        edge = (g[bad_rows] == 0) | (g[bad_rows] == qmax) | (o[bad_rows] == 0) | (o[bad_rows] == qmax)
        sub = diff[bad_rows]
        sub[edge & (np.abs(sub) <= 1)] = 0
        diff[bad_rows] = sub
    mism = np.nonzero(diff)
    pre = ref["pre"][mism]
    frac = np.abs(np.abs(pre - np.floor(pre)) - 0.5)
    assert np.all(np.abs(diff[mism]) == 1), "code differs by more than one step"
    assert np.all(frac <= FLIP_BAND), f"flip away from a rounding boundary (max distance {frac.max() if len(frac) else 0})"
    flips = len(pre)
    assert flips <= max(1, int(FLIP_FRACTION * R * C)), f"{flips} flips in {R * C} entries"
    if got_rowsum is not None:
        assert np.array_equal(got_rowsum, got_codes.sum(1, dtype=np.int64).astype(np.int32)), "rowsum != sum of the codes written"
    return dict(flips=flips, row_flips=len(bad_rows), entries=R * C)


def bf16_ulp_distance(got_bits: np.ndarray, ref_bits: np.ndarray) -> np.ndarray:
    """Distance in units of bf16 steps between two arrays of bf16 bit patterns."""
    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(got_bits) - key(ref_bits))


def check_output(got, ref64, out_dtype):
    """got: float32 array, or uint16 bf16 bit patterns.  ref64: the oracle's fp64 result."""
    if out_dtype == "f32":
        rel = np.linalg.norm(got.astype(np.float64) - ref64) / max(np.linalg.norm(ref64), 1e-300)
        assert rel <= 1e-5, f"relative Frobenius error {rel}"
        return rel
    d = bf16_ulp_distance(got, oracle.cast_bf16(ref64))
    assert d.max() <= 1, f"bf16 output off by {d.max()} ULP"
    return int(d.max())
