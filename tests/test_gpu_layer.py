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
    # activations: the flip rule, on the direct entry point and on what the layer's own pass left in its workspace
    # (larger batches may hold one code per byte there)
    ref_q = oracle.reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits, want_pre=True)
    direct = G.run_reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits)
    parity.check_activation_codes(direct["codes"], direct["scale"], direct["zero"], direct["rowsum"], ref_q, cfg.a_bits)
    pc, ps, pz, pr, lanes = layer.workspace_ptrs()

    def from_dev(p, shape, typestr):
        class View:
            __cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(p), False), version=2)
        return torch.as_tensor(View(), device=G.DEV).cpu().numpy().copy()

    wcodes = from_dev(pc, (cfg.M, cfg.K if lanes == 8 else cfg.K // 2), "|u1")
    got = dict(codes=parity.unpack_codes(wcodes, 4) if lanes == 4 else wcodes, scale=from_dev(ps, (cfg.M,), "<f4"),
               zero=from_dev(pz, (cfg.M,), "<f4"), rowsum=from_dev(pr, (cfg.M,), "<i4"))
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
    # the resident byte copy of 4-bit weights changes which kernel variant runs, not a bit of the result
    layer.keep_byte_weights(True)
    out2 = torch.zeros_like(out)
    layer.forward(G.dev_x(x), out2)
    torch.cuda.synchronize()
    assert torch.equal(out2, out)
    layer.keep_byte_weights(False)
    # informational: the quantized layer approximates the fp64 layer
    y = oracle.layernorm(x, L["gamma"], L["beta"], cfg.ln_eps)
    dense = oracle.dense_linear(y, L["W"].astype(np.float64)) + bias
    rel = np.linalg.norm(ref - dense) / np.linalg.norm(dense)
    print(name, "quantized-vs-fp64 relative error", rel)
    layer.destroy()


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5", "c2_w4a8"])
def test_layer_full_size_two_halves_sampled(name):
    """The launch configuration the benchmark times: layer object, full-size workload, the two half-step
    calls.  Activation codes are compared in full under the flip rule (whatever lane width the layer
    chose for its workspace); outputs are checked on sampled (m, n) entries with the oracle's integer
    dot product and epilogue evaluated on the codes the GPU produced."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS[name]
    M, N, K = cfg.M, cfg.N, cfg.K
    L = parity.oracle_layer(cfg)
    x = synth.activations(cfg)
    theta = B.qllm_theta_percentile(L["absmax"], 0.99)
    assert theta == L["theta"]
    h = B.qllm_build_reassembly(L["absmax"], theta, L["W"], L["lrA"], L["lrB"], cfg.w_bits)
    assert np.array_equal(h.weights()[0], L["w_packed"])
    layer = B.Layer(h, L["gamma"], L["beta"], cfg.ln_eps, None, cfg.a_bits, B.QLLM_BF16, B.QLLM_BF16, max_M=M)
    out = torch.zeros((M, N), dtype=torch.bfloat16, device=G.DEV)
    xd = G.dev_x(x)
    for _ in range(2):          # the second pass reuses scratch and the side stream like a steady-state step
        layer.reassemble_quant(xd)
        layer.qgemm(M, out)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    pc, ps, pz, pr, lanes = layer.workspace_ptrs()
    assert lanes == (8 if cfg.a_bits != 4 or M > 16 else 4)

    def from_dev(ptr, shape, typestr):
        # view the layer's borrowed device workspace through the CUDA array interface and copy it out
        class View:
            __cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(ptr), False), version=2)
        return torch.as_tensor(View(), device=G.DEV).cpu().numpy().copy()

    codes = from_dev(pc, (M, K if lanes == 8 else K // 2), "|u1")
    if lanes == 4:
        codes = parity.unpack_codes(codes, 4)
    scale = from_dev(ps, (M,), "<f4")
    zero = from_dev(pz, (M,), "<f4")
    rowsum = from_dev(pr, (M,), "<i4")
    ref_q = oracle.reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits, want_pre=True)
    # 8-bit codes: the pre-round values are 17x larger than 4-bit ones, so the fp32 error scales with them;
    # the band is widened in proportion (255/15) for this bit-width only
    old_band = parity.FLIP_BAND
    parity.FLIP_BAND = old_band * (17 if cfg.a_bits == 8 else 1)
    try:
        parity.check_activation_codes(codes, scale, zero, rowsum, ref_q, cfg.a_bits)
    finally:
        parity.FLIP_BAND = old_band
    rng = np.random.default_rng(cfg.seed + 100)
    ms = np.concatenate([rng.integers(0, M, 600), [0, 0, M - 1, M - 1]]).astype(np.int64)
    ns = np.concatenate([rng.integers(0, N, 600), [0, N - 1, 0, N - 1]]).astype(np.int32)
    acc = oracle.int_matmul_at(codes, L["w_codes"], ms, ns)
    ref = np.array([oracle.epilogue(np.array([[a]], np.int32), K, scale[m:m + 1], zero[m:m + 1], rowsum[m:m + 1],
                                    L["w_scale"][n:n + 1], L["w_zero"][n:n + 1], L["w_colsum"][n:n + 1])[0, 0]
                    for a, m, n in zip(acc, ms, ns)])
    parity.check_output(G.bf16_bits(out.cpu())[ms, ns], ref, "bf16")
    # the host-buffer entry point (chunked and overlapped at this size) returns the same bytes as the one call with
    # device buffers
    xh = torch.from_numpy(x.view(np.int16)).pin_memory()
    oh = torch.zeros((M, N), dtype=torch.bfloat16).pin_memory()
    layer.forward_host(xh, oh, M)
    layer.forward(xd, out)
    torch.cuda.synchronize()
    diff = oh.view(torch.int16) != out.cpu().view(torch.int16)
    assert not bool(diff.any()), (f"{int(diff.sum())} entries differ, rows {torch.nonzero(diff.any(1)).flatten()[:8].tolist()}"
                                  f" cols {torch.nonzero(diff.any(0)).flatten()[:8].tolist()}")
    # with the resident byte copy of the weights (no per-call widening) the step returns the same bytes, on both
    # entry points, and so does the layer after the copy has been given back
    want = out.cpu().view(torch.int16).clone()
    layer.keep_byte_weights(True)
    for step in ("resident", "resident-host", "released"):
        out.zero_()
        if step == "resident-host":
            oh.zero_()
            layer.forward_host(xh, oh, M)
            got = oh.view(torch.int16)
        else:
            if step == "released":
                layer.keep_byte_weights(False)
            layer.reassemble_quant(xd)
            layer.qgemm(M, out)
            torch.cuda.synchronize()
            got = out.cpu().view(torch.int16)
        assert torch.equal(got, want), step
    assert B.qllm_poll_status() == 0
    layer.destroy()


def test_two_layers_interleaved_on_one_stream():
    """The byte expansion of 4-bit weights lives in scratch memory shared by everything on a stream.  Two layers
    whose half-step calls interleave (A pre-GEMM, B pre-GEMM, A GEMM, B GEMM) must each still multiply with their
    own weights, exactly as when they run one after the other."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    layers, xs, refs = [], [], []
    for seed, N in ((31, 256), (32, 384)):
        cfg = synth.CONFIGS["c2"].scaled(M=520, K=512, N=N, n_outlier=4, seed=seed)
        L = parity.oracle_layer(cfg)
        h = B.qllm_build_reassembly(L["absmax"], L["theta"], L["W"], L["lrA"], L["lrB"], cfg.w_bits)
        layer = B.Layer(h, L["gamma"], L["beta"], cfg.ln_eps, None, cfg.a_bits, B.QLLM_BF16, B.QLLM_F32, max_M=cfg.M)
        x = G.dev_x(synth.activations(cfg))
        ref = torch.zeros((cfg.M, N), dtype=torch.float32, device=G.DEV)
        layer.forward(x, ref)
        layers.append(layer); xs.append(x); refs.append(ref)
    torch.cuda.synchronize()
    for _ in range(3):
        outs = [torch.zeros_like(r) for r in refs]
        layers[0].reassemble_quant(xs[0])
        layers[1].reassemble_quant(xs[1])
        layers[0].qgemm(xs[0].shape[0], outs[0])
        layers[1].qgemm(xs[1].shape[0], outs[1])
        torch.cuda.synchronize()
        assert B.qllm_poll_status() == 0
        # each layer's workspace is its own, so the activations are right either way; the weights are what is shared
        assert torch.equal(outs[0], refs[0]) and torch.equal(outs[1], refs[1])
    for layer in layers:
        layer.destroy()


def test_forward_under_stream_capture():
    """qllm_layer_forward issues only capturable work once its buffers are warm (launches, and the fork/join
    of the side stream that expands 4-bit weights): a CUDA graph of two layers replays to the same bits as the
    direct calls, before and after other direct calls on the stream."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    layers, xs, refs = [], [], []
    for seed, N in ((41, 256), (42, 384)):
        cfg = synth.CONFIGS["c2"].scaled(M=520, K=512, N=N, n_outlier=4, seed=seed)
        L = parity.oracle_layer(cfg)
        h = B.qllm_build_reassembly(L["absmax"], L["theta"], L["W"], L["lrA"], L["lrB"], cfg.w_bits)
        layers.append(B.Layer(h, L["gamma"], L["beta"], cfg.ln_eps, None, cfg.a_bits, B.QLLM_BF16, B.QLLM_F32,
                              max_M=cfg.M))
        xs.append(G.dev_x(synth.activations(cfg)))
        refs.append(torch.zeros((cfg.M, N), dtype=torch.float32, device=G.DEV))
    s = torch.cuda.Stream()
    outs = [torch.zeros_like(r) for r in refs]
    with torch.cuda.stream(s):
        for layer, x, ref in zip(layers, xs, refs):      # warm: scratch sized, attributes set
            layer.forward(x, ref)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for layer, x, out in zip(layers, xs, outs):
            layer.forward(x, out)
    torch.cuda.synchronize()
    for rep in range(3):
        for o in outs:
            o.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert B.qllm_poll_status() == 0
        assert torch.equal(outs[0], refs[0]) and torch.equal(outs[1], refs[1]), rep
        with torch.cuda.stream(s):                        # a direct call between replays
            chk = torch.zeros_like(refs[rep % 2])
            layers[rep % 2].forward(xs[rep % 2], chk)
        torch.cuda.synchronize()
        assert torch.equal(chk, refs[rep % 2])
    for layer in layers:
        layer.destroy()


def test_decode_calls_back_to_back_see_their_own_tokens():
    """The decode GEMM starts its prologue while the pre-GEMM kernel of the same call still runs (a programmatic
    dependent launch) and must wait for that kernel before it reads the tokens: forward calls issued back to back
    with alternating inputs return, every time, the bits of the same call made alone."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS["c3"].scaled(M=16, N=2048)
    L = parity.oracle_layer(cfg)
    h = B.qllm_build_reassembly(L["absmax"], L["theta"], L["W"], L["lrA"], L["lrB"], cfg.w_bits)
    layer = B.Layer(h, L["gamma"], L["beta"], cfg.ln_eps, None, cfg.a_bits, B.QLLM_BF16, B.QLLM_BF16, max_M=cfg.M)
    xs = [G.dev_x(synth.activations(cfg, stream=s)) for s in (1, 5, 6)]
    refs = []
    for x in xs:
        ref = torch.zeros((cfg.M, cfg.N), dtype=torch.bfloat16, device=G.DEV)
        layer.forward(x, ref)
        torch.cuda.synchronize()
        refs.append(ref)
    assert not torch.equal(refs[0], refs[1])
    outs = [torch.zeros_like(refs[0]) for _ in range(60)]
    for i, o in enumerate(outs):                        # no synchronisation between the calls
        layer.forward(xs[i % 3], o)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    for i, o in enumerate(outs):
        assert torch.equal(o, refs[i % 3]), i
    layer.destroy()


@pytest.mark.parametrize("name,kw", [("c2", dict(M=600, N=272)), ("c4", dict(M=150, N=144))])
def test_product_pipeline_end_to_end_as_the_benchmark_runs_it(name, kw):
    """Calibration statistic on the GPU -> threshold -> host builder -> layer -> forward, nothing taken from the
    oracle on the way (the benchmark's set-up).  The oracle then runs on the SAME statistic: same threshold, same
    map, same weight codes; activation codes under the flip rule; outputs from the oracle's integer product and
    epilogue on the codes the GPU produced."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS[name].scaled(**kw)
    gamma, beta = synth.layernorm_params(cfg)
    absmax = torch.zeros(cfg.K, dtype=torch.float32, device=G.DEV)
    B.qllm_calib_absmax(G.dev_x(synth.calibration_tokens(cfg)), G.dev(gamma), None, absmax, ln_eps=cfg.ln_eps)
    am = absmax.cpu().numpy()
    theta = B.qllm_theta_percentile(am, 0.99)
    W = synth.weights(cfg)
    A, Bm = synth.low_rank(cfg)
    h = B.qllm_build_reassembly(am, theta, W, A, Bm, cfg.w_bits)
    layer = B.Layer(h, gamma, beta, cfg.ln_eps, None, cfg.a_bits, B.QLLM_BF16, B.QLLM_BF16, max_M=cfg.M)
    x = synth.activations(cfg)
    out = torch.zeros((cfg.M, cfg.N), dtype=torch.bfloat16, device=G.DEV)
    layer.forward(G.dev_x(x), out)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    # the oracle on the product's statistic
    assert oracle.theta_percentile(am, 0.99) == theta
    ptr, src, coef, st = oracle.build_map(am, theta)
    p2, s2, c2 = h.map()
    assert np.array_equal(p2, ptr) and np.array_equal(s2, src) and np.array_equal(c2, coef)
    w = oracle.prepare_weights(W, ptr, src, cfg.w_bits, A, Bm)
    wc, ws, wz, wcs = h.weights()
    assert np.array_equal(wc, oracle.pack4(w["codes"]) if cfg.w_bits == 4 else w["codes"])
    assert np.array_equal(ws, w["scale"]) and np.array_equal(wz, w["zero"]) and np.array_equal(wcs, w["colsum"])
    pc, ps, pz, pr, lanes = layer.workspace_ptrs()

    def from_dev(p, shape, typestr):
        class View:
            __cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(p), False), version=2)
        return torch.as_tensor(View(), device=G.DEV).cpu().numpy().copy()

    codes = from_dev(pc, (cfg.M, cfg.K if lanes == 8 else cfg.K // 2), "|u1")
    if lanes == 4:
        codes = parity.unpack_codes(codes, 4)
    scale, zero, rowsum = from_dev(ps, (cfg.M,), "<f4"), from_dev(pz, (cfg.M,), "<f4"), from_dev(pr, (cfg.M,), "<i4")
    ref_q = oracle.reassemble_quant(x, gamma, beta, cfg.ln_eps, ptr, src, coef, cfg.a_bits, want_pre=True)
    parity.check_activation_codes(codes, scale, zero, rowsum, ref_q, cfg.a_bits)
    acc = oracle.int_matmul(codes, w["codes"])
    ref = oracle.epilogue(acc, cfg.K, scale, zero, rowsum, w["scale"], w["zero"], w["colsum"], None)
    parity.check_output(G.bf16_bits(out.cpu()), ref, "bf16")
    layer.destroy()
