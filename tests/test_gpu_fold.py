"""Appendix B on the product path: the host fold against the oracle's, and the run-time half (per-token
quantization without LayerNorm on an identity map) against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

import parity

pytestmark = pytest.mark.gpu


def test_fold_previous_matches_oracle_and_quantizes_without_layernorm():
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS["c1"].scaled(M=40, K=256)
    L = parity.oracle_layer(cfg, with_weights=False)
    rng = np.random.default_rng(9)
    C_in = 96
    Wp = (0.3 * rng.standard_normal((cfg.K, C_in))).astype(np.float32)     # preceding layer: C_in -> K channels
    bp = (0.1 * rng.standard_normal(cfg.K)).astype(np.float32)
    ref_W, ref_b = oracle.fold_previous(Wp, bp, L["ptr"], L["src"], L["coef"])
    W2, b2 = B.qllm_fold_previous(L["ptr"], L["src"], L["coef"], Wp, bp)
    assert np.array_equal(W2, ref_W) and np.array_equal(b2, ref_b)
    # run time: the folded layer's output already is the reassembled activation; quantize it as it is
    X = rng.standard_normal((cfg.M, C_in)).astype(np.float32)
    X[:, 5] *= 40.0
    xr = (X.astype(np.float64) @ W2.astype(np.float64).T + b2).astype(np.float32)
    C = cfg.K
    ident = (np.arange(C + 1, dtype=np.int32), np.arange(C, dtype=np.int32), np.ones(C, np.float32))
    for bits in (4, 8):
        got = G.run_reassemble_quant(xr, None, None, 0.0, *ident, bits)
        ref = oracle.quant_rows(xr.astype(np.float64), bits, want_pre=True)
        ref["xr"] = xr
        old = parity.FLIP_BAND
        parity.FLIP_BAND = old * (17 if bits == 8 else 1)
        try:
            parity.check_activation_codes(got["codes"], got["scale"], got["zero"], got["rowsum"], ref, bits)
        finally:
            parity.FLIP_BAND = old


@pytest.mark.parametrize("M,C,dtype,bits", [(40, 256, "f32", 4), (33, 4096, "bf16", 4), (19, 5120, "bf16", 6),
                                            (9, 8192, "bf16", 8), (21, 250, "f32", 6), (5, 77, "bf16", 8),
                                            (3, 4096, "f32", 4)])
def test_quantize_rows_alone(M, C, dtype, bits):
    """The run-time stage of a folded layer through its own entry point: Eq. 2 per row, no LayerNorm, no map,
    against the oracle's quantizer on the same values (constant and all-zero rows included)."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    rng = np.random.default_rng(C + bits)
    x = (rng.standard_normal((M, C)) * (1 + 25 * (rng.random(C) < 0.02))).astype(np.float32)
    x[0] = 0.0
    if M > 2:
        x[2] = -3.25
    if dtype == "bf16":
        xb = synth.f32_to_bf16_bits(x)
        x64 = synth.bf16_bits_to_f32(xb).astype(np.float64)
        xd = G.dev_x(xb)
    else:
        x64 = x.astype(np.float64)
        xd = G.dev(x)
    guards = [G.Guarded((M, C // 2 if bits == 4 else C), torch.uint8, 0xAB), G.Guarded((M,), torch.float32, 0),
              G.Guarded((M,), torch.float32, 0), G.Guarded((M,), torch.int32, 0)]
    codes, sc, ze, rs = (g.t for g in guards)
    B.qllm_quantize_rows(xd, bits, codes, sc, ze, rs)
    torch.cuda.synchronize()
    for g, what in zip(guards, ("codes", "a_scale", "a_zero", "a_rowsum")):
        g.check(what)
    got = codes.cpu().numpy()
    got = parity.unpack_codes(got, 4) if bits == 4 else got
    ref = oracle.quant_rows(x64, bits, want_pre=True)
    old = parity.FLIP_BAND
    parity.FLIP_BAND = old * (17 if bits == 8 else 1)
    try:
        parity.check_activation_codes(got, sc.cpu().numpy(), ze.cpu().numpy(), rs.cpu().numpy(), ref, bits)
    finally:
        parity.FLIP_BAND = old


def test_quantize_rows_far_from_zero():
    """A row far from zero with a tiny range (quotients of ~1.5e7, zero-point of the same size): fp32 cannot resolve
    the oracle's decisions there, so the check is on what must hold whatever the rounding: codes inside the range, the
    row sum of exactly those codes, alpha from the row's range, and every value reproduced to within a few steps."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    C, bits = 4096, 4
    rng = np.random.default_rng(11)
    x = np.zeros((4, C), np.float32)
    x[0] = 1000.0 + 1e-3 * rng.random(C)
    x[1] = -2500.0 + 4e-3 * rng.random(C)
    x[2] = rng.standard_normal(C)                        # an ordinary row beside them
    x[3] = 1000.0
    codes = torch.zeros((4, C // 2), dtype=torch.uint8, device=G.DEV)
    sc = torch.zeros(4, device=G.DEV); ze = torch.zeros(4, device=G.DEV); rs = torch.zeros(4, dtype=torch.int32, device=G.DEV)
    B.qllm_quantize_rows(G.dev(x), bits, codes, sc, ze, rs)
    torch.cuda.synchronize()
    q = parity.unpack_codes(codes.cpu().numpy(), 4).astype(np.int64)
    alpha, zero = sc.cpu().numpy().astype(np.float64), ze.cpu().numpy().astype(np.float64)
    assert q.min() >= 0 and q.max() <= 15
    assert np.array_equal(q.sum(1), rs.cpu().numpy())
    x64 = x.astype(np.float64)
    for m in range(3):
        np.testing.assert_allclose(alpha[m], (x64[m].max() - x64[m].min()) / 15, rtol=2e-5)
        assert zero[m] == np.rint(zero[m])
        assert np.abs(x64[m] - alpha[m] * (q[m] - zero[m])).max() <= 2.5 * alpha[m] + 2e-4 * abs(x64[m]).max() * (m < 2)
    assert alpha[3] == 1000.0 and np.all(q[3] == 0)
    ref = oracle.quant_rows(x64[2:3], bits, want_pre=True)
    parity.check_activation_codes(q[2:3].astype(np.uint8), sc.cpu().numpy()[2:3], ze.cpu().numpy()[2:3], rs.cpu().numpy()[2:3], ref, bits)
