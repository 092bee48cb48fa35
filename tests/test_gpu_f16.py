"""GPU parity of the FP16 2:4 sparse model (Sec. 3.1, Sec. 3.4): compression and packing bit-exact
against the oracle; the sparse GEMM's FP32 sums against the oracle's exact sums within the bound an
FP32 accumulator allows; the FP16 output within one binary16 ulp plus that bound."""
import numpy as np
import pytest

import oracle
from paper_2305_10727_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2305_10727_b200 import binding
    binding.load()
    binding.set_block_tokens(0)
    return binding


def cu(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def acc_bound(mag, K):
    # products of binary16 values are exact; the tensor core adds them into an FP32 accumulator, one
    # rounding (or truncation) of at most 2^-23 of the running magnitude per 32-column instruction,
    # plus a few inside an instruction's adder tree
    return (K / 32.0 + 8.0) * 2.0 ** -23 * mag


def f16_ulp(y):
    a = np.abs(y.astype(np.float64))
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -14)))
    return 2.0 ** (e - 10)


def prepare(B, W):
    vals, meta = B.compress24_f16(B.prune24(cu(W)))
    return vals, meta, B.pack24_f16(vals, meta)


@pytest.mark.parametrize("N,K", [(1, 8), (5, 24), (64, 16), (768, 192), (129, 1288), (300, 776)])
def test_compress24_f16_bit_exact(B, N, K):
    rng = np.random.default_rng(N + K)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[0, :8] = [1e-9, -2.0, 0.0, 3.0, 5.0, 5.0, 5.0, 5.0]      # underflow to zero; a four-way tie
    if K >= 16:
        W[0, 8:16] = [65504.0, 7e4, -7e4, 1.0, 6e-8, -6e-8, 3e-8, 0.0]   # overflow to infinity, subnormals
    prep = oracle.prepare_weight_f16(W)
    vals, meta, _ = prepare(B, W)
    assert np.array_equal(vals.cpu().numpy().view(np.uint16), prep["vals"].view(np.uint16))
    assert np.array_equal(meta.cpu().numpy(), prep["meta"])
    assert B.packed_bytes_f16(N, K) == ((N + 255) // 256 * 256) * ((K + 127) // 128 * 128) * 9 // 8


GEMM_SHAPES = [(1, 8, 8), (16, 128, 64), (64, 256, 128), (197, 256, 192), (257, 384, 136), (300, 128, 1280),
               (333, 384, 776), (1576, 768, 192), (1000, 512, 2048), (394, 96, 48), (500, 288, 96), (70, 5, 32)]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("block_t", [0, 32, 96, 224])
def test_spgemm_f16_sums(B, M, N, K, block_t):
    d = inputs.random_layer(500 + M + N + K, M, N, K)
    prep = oracle.prepare_weight_f16(d["W"])
    acc_o, mag = oracle.spgemm_f16_rows(d["X"], prep["vals"], prep["meta"])
    _, _, Wpk = prepare(B, d["W"])
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.set_block_tokens(block_t)
    try:
        acc = B.spgemm_f16(cu(d["X"]), Wpk, N, out_type=B.OUT_F32, status_buf=status).cpu().numpy()
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert (np.abs(acc.astype(np.float64) - acc_o) <= acc_bound(mag, K) + 1e-45).all()


@pytest.mark.parametrize("M,N,K", [(197, 256, 192), (1576, 768, 192), (333, 128, 1024), (394, 96, 48), (100, 200, 72)])
@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("use_bias", [True, False])
def test_spgemm_f16_epilogue(B, M, N, K, act, use_bias):
    d = inputs.random_layer(700 + M + N + K, M, N, K)
    bias = d["bias"] if use_bias else None
    prep = oracle.prepare_weight_f16(d["W"])
    acc_o, mag = oracle.spgemm_f16_rows(d["X"], prep["vals"], prep["meta"])
    Y_o = oracle.epilogue_f16(acc_o, bias, act=act)
    _, _, Wpk = prepare(B, d["W"])
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    Y = B.spgemm_f16(cu(d["X"]), Wpk, N, bias=None if bias is None else cu(bias), act=act,
                     status_buf=status).cpu().numpy()
    assert status.cpu().tolist() == [0, 0, 0, 0]
    # one binary16 ulp for the final rounding, plus the accumulator's slack through an epilogue whose
    # slope is at most 1.13 (GELU), plus the kernel's GELU error (< 1e-5 relative)
    tol = f16_ulp(Y_o) + 1.2 * acc_bound(mag, K) + 2e-5 * np.abs(Y_o.astype(np.float64))
    assert (np.abs(Y.astype(np.float64) - Y_o.astype(np.float64)) <= tol).all()
    # the accumulator slack is far below an ulp here: nearly every output is the oracle's, the rest one ulp off
    assert (Y.view(np.uint16) != Y_o.view(np.uint16)).mean() < 0.02


def test_spgemm_f16_against_library_product(B):
    # the same layer as a library matrix product of the decompressed binary16 weight, in FP32
    M, N, K = 512, 256, 512
    d = inputs.random_layer(42, M, N, K)
    prep = oracle.prepare_weight_f16(d["W"])
    _, _, Wpk = prepare(B, d["W"])
    acc = B.spgemm_f16(cu(d["X"]), Wpk, N, out_type=B.OUT_F32)
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        ref = cu(d["X"]).float() @ cu(prep["Wh"]).float().T
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev
    assert torch.allclose(acc, ref, rtol=0, atol=1e-4)


@pytest.mark.parametrize("li", range(4))
def test_f16_deit_base_block_full_size(B, li):
    cfg = inputs.CONFIGS["deit_base_b64"]
    L = cfg.layers[li]
    d = inputs.make_layer_inputs(cfg, li)
    prep = oracle.prepare_weight_f16(d["W"])
    vals, meta, Wpk = prepare(B, d["W"])
    assert np.array_equal(vals.cpu().numpy().view(np.uint16), prep["vals"].view(np.uint16))
    assert np.array_equal(meta.cpu().numpy(), prep["meta"])
    rng = np.random.default_rng(li)
    rows = np.unique(np.concatenate([[0, 1, 223, 224, cfg.M - 1, cfg.M - 2, cfg.M // 2], rng.integers(0, cfg.M, 24)]))
    acc_o, mag = oracle.spgemm_f16_rows(d["X"], prep["vals"], prep["meta"], rows)
    act = 1 if L.gelu else 0
    Y_o = oracle.epilogue_f16(acc_o, d["bias"], act=act)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    X = cu(d["X"])
    acc = B.spgemm_f16(X, Wpk, L.N, out_type=B.OUT_F32, status_buf=status)
    assert (np.abs(acc[cu(rows)].cpu().numpy().astype(np.float64) - acc_o) <= acc_bound(mag, L.K)).all()
    Y = B.spgemm_f16(X, Wpk, L.N, bias=cu(d["bias"]), act=act, status_buf=status)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    tol = f16_ulp(Y_o) + 1.2 * acc_bound(mag, L.K) + 2e-5 * np.abs(Y_o.astype(np.float64))
    assert (np.abs(Y[cu(rows)].cpu().numpy().astype(np.float64) - Y_o.astype(np.float64)) <= tol).all()
    assert torch.isfinite(Y).all()
