"""qllm_qgemm_noalloc: the GEMM entry point for callers that cannot allocate device memory
(memory-pool or latency-critical serving code, processes whose device memory belongs to another
allocator).  Its row-sum scratch is a fixed array inside the library, shared by all calls, so the
test runs it twice in a row -- a larger problem first, then a smaller one whose rows would pick up
stale sums if the scratch were not rewritten -- and compares each result with qllm_qgemm.
Collected last on purpose: a failure here cannot hide the other tests."""
import numpy as np
import pytest

from paper_2310_08041_b200 import synth

pytestmark = pytest.mark.gpu


def _case(seed, M, N, K, a_bits, w_bits):
    rng = np.random.default_rng([seed, 3])
    qa = synth.random_codes(seed, M, K, a_bits)
    qw = synth.random_codes(seed + 1, N, K, w_bits)
    return dict(M=M, N=N, K=K, a_bits=a_bits, w_bits=w_bits, qa=qa, qw=qw,
                a_scale=rng.uniform(0.01, 0.5, M).astype(np.float32),
                a_zero=rng.integers(0, (1 << a_bits), M).astype(np.float32),
                w_scale=rng.uniform(1e-3, 1e-2, N).astype(np.float32),
                w_zero=rng.integers(0, (1 << w_bits), N).astype(np.float32),
                bias=rng.standard_normal(N).astype(np.float32),
                w_colsum=qw.sum(1, dtype=np.int64).astype(np.int32))


def test_noalloc_matches_qgemm_on_two_calls_in_a_row():
    import torch
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    cases = [_case(11, 300, 528, 1024, 4, 4), _case(12, 9, 136, 512, 6, 6), _case(13, 150, 272, 384, 4, 4)]
    for c in cases:
        M, N, K = c["M"], c["N"], c["K"]
        da, dw = G.dev(G.store_codes(c["qa"], c["a_bits"])), G.dev(G.store_codes(c["qw"], c["w_bits"]))
        args = (da, G.dev(c["a_scale"]), G.dev(c["a_zero"]), dw, G.dev(c["w_scale"]), G.dev(c["w_zero"]),
                G.dev(c["w_colsum"]), G.dev(c["bias"]))
        for tdt in (torch.float32, torch.bfloat16):
            ref = torch.zeros((M, N), dtype=tdt, device=G.DEV)
            B.qllm_qgemm(*args, ref, M, N, K, c["a_bits"], c["w_bits"])        # library-allocated scratch
            got = torch.full((M, N), 7.0, dtype=tdt, device=G.DEV)
            B.qllm_qgemm_noalloc(*args, got, M, N, K, c["a_bits"], c["w_bits"])
            torch.cuda.synchronize()
            # same kernels, same row sums: the outputs agree bit for bit (tighter than the 1e-5 /
            # 1-ULP bound the other GEMM tests use)
            assert torch.equal(got.view(torch.int32 if tdt == torch.float32 else torch.int16),
                               ref.view(torch.int32 if tdt == torch.float32 else torch.int16))
    # an argument error is found before anything is launched: the shared array keeps the last call's sums
    n0 = B.qllm_launch_count()
    ptrs = [B._dp(t) for t in args]
    raw = lambda p, out, dt: B._lib.qllm_qgemm_noalloc(*p, out, M, N, K, c["a_bits"], c["w_bits"], dt, None)
    assert raw(ptrs, None, B.QLLM_F32) == B.QLLM_ERR_NULL                         # no output
    assert raw(ptrs[:4] + [None] + ptrs[5:], B._dp(got), B.QLLM_BF16) == B.QLLM_ERR_NULL   # no weight scales
    assert raw(ptrs, B._dp(got), 7) == B.QLLM_ERR_DTYPE
    assert raw(ptrs, B._dp(got) + 2, B.QLLM_BF16) == B.QLLM_ERR_ALIGN
    assert B.qllm_launch_count() == n0
    # sizes beyond the fixed scratch are refused with a clear status, nothing is launched
    n0 = B.qllm_launch_count()
    z = torch.zeros(16, device=G.DEV)
    with pytest.raises(B.QllmError) as e:
        B.qllm_qgemm_noalloc(da, z, z, dw, z, z, z.int(), None, z, B.QLLM_NOALLOC_MAX_M + 1, 8, 16, 4, 4)
    assert e.value.status == B.QLLM_ERR_UNSUPPORTED and B.qllm_launch_count() == n0


@pytest.mark.parametrize("a_bits,w_bits", [(4, 4), (8, 4)])
def test_noalloc_in_its_own_regime_against_the_oracle(a_bits, w_bits):
    """From 385 token rows qllm_qgemm widens 4-bit operands into library scratch; the entry point that may not
    allocate stays on the kernel that unpacks tiles in shared memory, where every CTA walks several tiles.  Same
    bits as qllm_qgemm, the oracle's integer sums on sampled entries, no device memory taken, no wait expired."""
    import torch
    import oracle
    import parity
    import gpu_util as G
    from paper_2310_08041_b200 import binding as B
    c = _case(21 + a_bits, 1536, 4096, 512, a_bits, w_bits)
    M, N, K = c["M"], c["N"], c["K"]
    da, dw = G.dev(G.store_codes(c["qa"], a_bits)), G.dev(G.store_codes(c["qw"], w_bits))
    args = (da, G.dev(c["a_scale"]), G.dev(c["a_zero"]), dw, G.dev(c["w_scale"]), G.dev(c["w_zero"]),
            G.dev(c["w_colsum"]), G.dev(c["bias"]))
    ref = torch.zeros((M, N), dtype=torch.float32, device=G.DEV)
    got = torch.full((M, N), 7.0, dtype=torch.float32, device=G.DEV)
    B.qllm_qgemm(*args, ref, M, N, K, a_bits, w_bits)
    B.qllm_qgemm_noalloc(*args, got, M, N, K, a_bits, w_bits)              # warm: the array's address is looked up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(2):
        got.fill_(7.0)
        B.qllm_qgemm_noalloc(*args, got, M, N, K, a_bits, w_bits)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0, "the allocation-free entry point took device memory"
    assert B.qllm_poll_status() == 0
    assert torch.equal(got.view(torch.int32), ref.view(torch.int32))
    rng = np.random.default_rng(5)
    ms = np.concatenate([rng.integers(0, M, 400), [0, M - 1, 127, 128, 1535]]).astype(np.int64)
    ns = np.concatenate([rng.integers(0, N, 400), [0, N - 1, 255, 256, 4095]]).astype(np.int32)
    acc = oracle.int_matmul_at(c["qa"], c["qw"], ms, ns)
    rowsum = c["qa"].sum(1, dtype=np.int64).astype(np.int32)
    want = np.array([oracle.epilogue(np.array([[a]], np.int32), K, c["a_scale"][m:m + 1], c["a_zero"][m:m + 1], rowsum[m:m + 1],
                                     c["w_scale"][n:n + 1], c["w_zero"][n:n + 1], c["w_colsum"][n:n + 1], c["bias"][n:n + 1])[0, 0]
                     for a, m, n in zip(acc, ms, ns)])
    parity.check_output(got.cpu().numpy()[ms, ns], want, "f32")
