"""End to end: builder -> layer object -> fused kernel -> GEMM, against the oracle's path."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw,out_dtype", [("c1", {}, "f32"), ("c1", {}, "bf16"),
                                               ("c2", dict(M=150, N=528), "f32"),
                                               ("c3", dict(M=8, N=1024), "bf16"),
                                               ("c4", dict(M=133, N=272), "bf16")])
def test_layer_forward_matches_oracle(name, kw, out_dtype):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS[name].scaled(**kw)
    L = parity.oracle_layer(cfg)
    x = synth.activations(cfg)
    # the product path derives its own calibration statistic, threshold, map and weights
    xc = G.dev_x(synth.calibration_tokens(cfg))
    absmax = torch.zeros(cfg.K, dtype=torch.float32, device=G.DEV)
    B.qllm_calib_absmax(xc, G.dev(L["gamma"]), None if L["beta"] is None else G.dev(L["beta"]), absmax, ln_eps=cfg.ln_eps)
    am = absmax.cpu().numpy()
    np.testing.assert_allclose(am, L["absmax"], rtol=5e-6)
    # build from the oracle's statistic so that both sides hold the same map (the statistic
    # itself was compared just above; a last-bit difference could move a merge)
    theta = B.qllm_theta_for_extra(L["absmax"], 8) if cfg.theta_rule == "extra8" else B.qllm_theta_percentile(L["absmax"], 0.99)
    assert theta == L["theta"]
    h = B.qllm_build_reassembly(L["absmax"], theta, L["W"], L["lrA"], L["lrB"], cfg.w_bits)
    wc, ws, wz, wcs = h.weights()
    assert np.array_equal(wc, L["w_packed"])
    xdt = B.QLLM_F32 if cfg.x_dtype == "f32" else B.QLLM_BF16
    odt = B.QLLM_F32 if out_dtype == "f32" else B.QLLM_BF16
    bias = np.random.default_rng(1).standard_normal(cfg.N).astype(np.float32)
    layer = B.Layer(h, L["gamma"], L["beta"], cfg.ln_eps, bias, cfg.a_bits, xdt, odt, max_M=cfg.M)
    tdt = torch.float32 if out_dtype == "f32" else torch.bfloat16
    out = torch.zeros((cfg.M, cfg.N), dtype=tdt, device=G.DEV)
    layer.forward(G.dev_x(x), out)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    # activations: the flip rule
    ref_q = oracle.reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits, want_pre=True)
    got = G.run_reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits)
    parity.check_activation_codes(got["codes"], got["scale"], got["zero"], got["rowsum"], ref_q, cfg.a_bits)
    # outputs: the oracle's GEMM + epilogue on the codes the GPU produced (identical codes)
    acc = oracle.int_matmul(got["codes"], L["w_codes"])
    ref = oracle.epilogue(acc, cfg.K, got["scale"], got["zero"], got["rowsum"], L["w_scale"], L["w_zero"], L["w_colsum"], bias)
    o = out.cpu()
    parity.check_output(o.numpy() if out_dtype == "f32" else G.bf16_bits(o), ref, out_dtype)
    # host-buffer entry point gives the same bytes
    xh = torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).pin_memory()
    oh = torch.zeros((cfg.M, cfg.N), dtype=tdt).pin_memory()
    layer.forward_host(xh, oh, cfg.M)
    assert torch.equal(oh.view(torch.int16 if out_dtype == "bf16" else torch.int32), o.view(torch.int16 if out_dtype == "bf16" else torch.int32))
    # informational: the quantized layer approximates the fp64 layer
    y = oracle.layernorm(x, L["gamma"], L["beta"], cfg.ln_eps)
    dense = oracle.dense_linear(y, L["W"].astype(np.float64)) + bias
    rel = np.linalg.norm(ref - dense) / np.linalg.norm(dense)
    print(name, "quantized-vs-fp64 relative error", rel)
    layer.destroy()
