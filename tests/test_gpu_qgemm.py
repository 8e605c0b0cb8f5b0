"""GPU parity of the integer GEMM + dequantizing epilogue against the oracle, given identical codes."""
import numpy as np
import pytest

import oracle
from paper_2310_08041_b200 import synth

import parity

pytestmark = pytest.mark.gpu

# (M, N, K, a_bits, w_bits): tiny, ragged tails, several tiles, decode sizes, byte lanes, mixed widths
SHAPES = [
    (1, 64, 128, 4, 4), (5, 33, 64, 4, 4), (16, 100, 256, 4, 4), (17, 40, 72, 4, 4),
    (8, 22016, 512, 4, 4), (3, 48, 4096, 4, 4), (16, 1000, 4096, 4, 4),
    (64, 512, 256, 4, 4), (130, 272, 384, 4, 4), (300, 528, 1024, 4, 4), (129, 144, 8192, 4, 4),
    (257, 528, 640, 6, 6), (150, 256, 5120, 6, 6), (9, 31, 77, 6, 6), (40, 64, 256, 8, 8),
    (140, 272, 512, 8, 4), (33, 80, 256, 4, 8), (200, 16, 128, 4, 4), (128, 256, 128, 4, 4),
    (8, 136, 512, 6, 6), (12, 520, 1024, 8, 4), (5, 61, 256, 4, 8), (16, 22016, 4096, 4, 4), (1, 8, 128, 4, 4),
    (600, 272, 256, 4, 4), (520, 136, 512, 8, 4), (513, 80, 160, 4, 8),
    # CTA-pair kernel edges: one row past a 128-row block, narrowest output, K that ends inside a stage, 1000^3
    (129, 8, 128, 8, 8), (385, 264, 272, 8, 8), (1000, 1000, 1008, 6, 6),
    # decode kernel edges: K that splits unevenly over a warp pair, a single 64-byte step (one warp of the pair idle),
    # a last task with 8 of 16 channels, 9 tokens (second MMA half empty), two tasks per warp pair
    (9, 40, 384, 4, 4), (16, 17, 128, 4, 4), (7, 2408, 640, 6, 6), (2, 24000, 128, 4, 4),
]


def _operands(seed, M, N, K, a_bits, w_bits):
    qa = synth.random_codes(seed, M, K, a_bits)
    qw = synth.random_codes(seed + 1, N, K, w_bits)
    return qa, qw


@pytest.mark.parametrize("M,N,K,a_bits,w_bits", SHAPES)
def test_accumulators_bit_exact(M, N, K, a_bits, w_bits):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    qa, qw = _operands(M + N + K, M, N, K, a_bits, w_bits)
    ref = oracle.int_matmul(qa, qw)
    guard = G.Guarded((M, N), torch.int32, -12345)       # canaries on both sides of the output
    acc = guard.t
    B.qllm_qgemm_acc(G.dev(G.store_codes(qa, a_bits)), G.dev(G.store_codes(qw, w_bits)), acc, M, N, K, a_bits, w_bits)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    guard.check("accumulators")
    assert np.array_equal(acc.cpu().numpy(), ref)


def _epilogue_inputs(seed, M, N, a_bits, w_bits, qa, qw):
    rng = np.random.default_rng([seed, 7])
    qa_max, qw_max = (1 << a_bits) - 1, (1 << w_bits) - 1
    return dict(a_scale=rng.uniform(0.01, 0.5, M).astype(np.float32),
                a_zero=rng.integers(-2, qa_max + 3, M).astype(np.float32),
                w_scale=rng.uniform(1e-3, 1e-2, N).astype(np.float32),
                w_zero=rng.integers(0, qw_max + 1, N).astype(np.float32),
                bias=rng.standard_normal(N).astype(np.float32),
                a_rowsum=qa.sum(1, dtype=np.int64).astype(np.int32),
                w_colsum=qw.sum(1, dtype=np.int64).astype(np.int32))


@pytest.mark.parametrize("out_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("M,N,K,a_bits,w_bits", [(5, 33, 64, 4, 4), (16, 1000, 4096, 4, 4), (130, 272, 384, 4, 4),
                                                 (257, 528, 640, 6, 6), (9, 31, 77, 6, 6), (140, 272, 512, 8, 4),
                                                 (385, 264, 272, 8, 8), (129, 8, 128, 8, 8)])
def test_epilogue_matches_oracle(M, N, K, a_bits, w_bits, out_dtype):
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    qa, qw = _operands(3 * M + N, M, N, K, a_bits, w_bits)
    e = _epilogue_inputs(M + K, M, N, a_bits, w_bits, qa, qw)
    acc = oracle.int_matmul(qa, qw)
    tdt = torch.float32 if out_dtype == "f32" else torch.bfloat16
    da, dw = G.dev(G.store_codes(qa, a_bits)), G.dev(G.store_codes(qw, w_bits))
    for bias in (e["bias"], None):
        for give_rowsum in (True, False):
            ref = oracle.epilogue(acc, K, e["a_scale"], e["a_zero"], e["a_rowsum"], e["w_scale"], e["w_zero"], e["w_colsum"], bias)
            guard = G.Guarded((M, N), tdt, 0)
            out = guard.t
            B.qllm_qgemm(da, G.dev(e["a_scale"]), G.dev(e["a_zero"]), dw, G.dev(e["w_scale"]), G.dev(e["w_zero"]),
                         G.dev(e["w_colsum"]), None if bias is None else G.dev(bias), out, M, N, K, a_bits, w_bits,
                         a_rowsum=G.dev(e["a_rowsum"]) if give_rowsum else None)
            torch.cuda.synchronize()
            guard.check("out")
            got = out.cpu().numpy() if out_dtype == "f32" else G.bf16_bits(out.contiguous())
            parity.check_output(got, ref, out_dtype)


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_full_size_sampled_entries(name):
    """Benchmark-size launch; accumulators and outputs checked on sampled (m, n) entries."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cfg = synth.CONFIGS[name]
    M, N, K = cfg.M, cfg.N, cfg.K
    qa, qw = _operands(cfg.seed, M, N, K, cfg.a_bits, cfg.w_bits)
    e = _epilogue_inputs(cfg.seed, M, N, cfg.a_bits, cfg.w_bits, qa, qw)
    rng = np.random.default_rng(cfg.seed)
    ms = np.concatenate([rng.integers(0, M, 3000), [0, 0, M - 1, M - 1]]).astype(np.int64)
    ns = np.concatenate([rng.integers(0, N, 3000), [0, N - 1, 0, N - 1]]).astype(np.int32)
    ref_acc = oracle.int_matmul_at(qa, qw, ms, ns)
    da, dw = G.dev(G.store_codes(qa, cfg.a_bits)), G.dev(G.store_codes(qw, cfg.w_bits))
    acc = torch.zeros((M, N), dtype=torch.int32, device=G.DEV)
    B.qllm_qgemm_acc(da, dw, acc, M, N, K, cfg.a_bits, cfg.w_bits)
    torch.cuda.synchronize()
    assert B.qllm_poll_status() == 0
    acc_np = acc.cpu().numpy()
    assert np.array_equal(acc_np[ms, ns], ref_acc)
    # every row and column sum of the accumulators (a property that holds at any size):
    # sum_n acc[m][n] = qa[m] . (sum_n qw[n])
    colvec = qw.astype(np.int64).sum(0)
    assert np.array_equal(acc_np.astype(np.int64).sum(1), qa.astype(np.int64) @ colvec)
    rowvec = qa.astype(np.int64).sum(0)
    assert np.array_equal(acc_np.astype(np.int64).sum(0), qw.astype(np.int64) @ rowvec)
    del acc
    for out_dtype, tdt in (("f32", torch.float32), ("bf16", torch.bfloat16)):
        out = torch.zeros((M, N), dtype=tdt, device=G.DEV)
        B.qllm_qgemm(da, G.dev(e["a_scale"]), G.dev(e["a_zero"]), dw, G.dev(e["w_scale"]), G.dev(e["w_zero"]),
                     G.dev(e["w_colsum"]), G.dev(e["bias"]), out, M, N, K, cfg.a_bits, cfg.w_bits,
                     a_rowsum=G.dev(e["a_rowsum"]))
        torch.cuda.synchronize()
        # oracle epilogue on the sampled entries, one (m, n) at a time
        ref = np.array([oracle.epilogue(np.array([[a]], np.int32), K, e["a_scale"][m:m + 1], e["a_zero"][m:m + 1],
                                        e["a_rowsum"][m:m + 1], e["w_scale"][n:n + 1], e["w_zero"][n:n + 1],
                                        e["w_colsum"][n:n + 1], e["bias"][n:n + 1])[0, 0]
                        for a, m, n in zip(ref_acc[:400], ms[:400], ns[:400])])
        o = out.cpu()
        got = o.numpy()[ms[:400], ns[:400]] if out_dtype == "f32" else G.bf16_bits(o)[ms[:400], ns[:400]]
        parity.check_output(got, ref, out_dtype)
        del out


def test_empty_and_status():
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    n0 = B.qllm_launch_count()
    z = torch.zeros(16, device=G.DEV)
    zi = torch.zeros(16, dtype=torch.int32, device=G.DEV)
    zb = torch.zeros(64, dtype=torch.uint8, device=G.DEV)
    B.qllm_qgemm(zb, z, z, zb, z, z, zi, None, z, 0, 8, 16, 4, 4)
    assert B.qllm_launch_count() == n0
    with pytest.raises(B.QllmError) as e:
        B.qllm_qgemm(zb, z, z, zb, z, z, zi, None, z, 2, 8, 15, 4, 4)
    assert e.value.status == B.QLLM_ERR_SHAPE
    assert B.qllm_poll_status() == 0


def test_bounded_wait_expiry_is_reported_once_and_harmless():
    """A device-side wait that runs out raises the status word and returns; the host reads QLLM_ERR_TIMEOUT once,
    then QLLM_OK, and the next GEMM is bit-exact.  The expiry is produced by a one-warp kernel that waits, under a
    short limit, for a barrier nothing arrives on (the GEMM kernels themselves are not altered for the test)."""
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    assert B.qllm_poll_status() == 0
    gave_up = torch.zeros(1, dtype=torch.int32, device=G.DEV)
    B.qllm_debug_wait_expiry(gave_up)
    torch.cuda.synchronize()                       # the launch returns
    assert int(gave_up.item()) == 1
    assert B.qllm_poll_status() == B.QLLM_ERR_TIMEOUT
    assert B.qllm_poll_status() == 0               # reported once
    M, N, K = 300, 384, 512
    qa, qw = synth.random_codes(3, M, K, 8), synth.random_codes(4, N, K, 8)
    acc = torch.zeros((M, N), dtype=torch.int32, device=G.DEV)
    B.qllm_qgemm_acc(G.dev(qa), G.dev(qw), acc, M, N, K, 8, 8)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), oracle.int_matmul(qa, qw))
    assert B.qllm_poll_status() == 0
