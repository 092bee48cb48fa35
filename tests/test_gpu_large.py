"""GPU parity beyond 2^31 elements: byte offsets, element counts and tile counts that no longer fit
32 bits.  The tensors are too large for the oracle as a whole, so they are drawn on the device
(seeded) and checked on sampled rows the oracle computes one by one, plus reductions a library
routine provides (the tensor's maximum) and exact column-sum identities."""
import numpy as np
import pytest

import oracle

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


def f16_ulp_distance(a, b):
    def key(h):
        u = h.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(np.ascontiguousarray(a)) - key(np.ascontiguousarray(b)))


def _rows(M, seed, n=48):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, M - 1, M - 2, M // 2, (1 << 20) - 1, 1 << 20, (1 << 20) + 1]
    return np.unique(np.array([r for r in fixed if 0 <= r < M] + rng.integers(0, M, n).tolist(), np.int64))


def test_quant_act_more_than_2_31_elements(B):
    M, K = 70000, 32768                                   # 2.29e9 elements, 4.6 GB of binary16
    assert M * K > 1 << 31
    gen = torch.Generator(device="cuda").manual_seed(5)
    X = torch.empty((M, K), dtype=torch.float16, device="cuda")
    for i in range(0, M, 10000):                          # drawn in slabs to bound the FP32 temporary
        X[i:i + 10000] = torch.randn((min(10000, M - i), K), generator=gen, device="cuda").half()
    X[M - 1, K - 1] = 9.5                                 # the maximum sits in the very last element
    Xq, xs = B.quant_act(X)
    amax = np.float32(float(X.abs().max().cpu()))
    assert amax == np.float32(9.5)
    want_scale = np.float32(amax / np.float32(127.0))
    assert xs.cpu().numpy()[0] == want_scale
    rows = _rows(M, 1)
    Xq_o, _ = oracle.quant_act(X[cu(rows)].cpu().numpy(), x_scale=want_scale)
    assert np.array_equal(Xq[cu(rows)].cpu().numpy(), Xq_o)
    # the supplied-scale kernel and the static-scratch entry point on the same tensor
    Xq2, _ = B.quant_act(X, x_scale=xs, scale_mode=B.SCALE_GIVEN)
    assert torch.equal(Xq, Xq2)
    del Xq2
    Xq3, xs3 = B.quant_act_static(X)
    assert xs3.cpu().numpy()[0] == want_scale
    assert np.array_equal(Xq3[cu(rows)].cpu().numpy(), Xq_o)           # against the oracle, sampled rows
    assert torch.equal(Xq, Xq3)                                        # and every element against the other kernel


@pytest.mark.parametrize("out", ["i8", "f16", "i32"])
def test_gemm_more_than_2_31_outputs(B, out):
    M, N, K = 1_200_000, 2048, 32                         # 2.46e9 outputs
    assert M * N > 1 << 31
    rng = np.random.default_rng(11)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    prep = oracle.prepare_weight(W)
    gen = torch.Generator(device="cuda").manual_seed(6)
    Xq = torch.randint(-127, 128, (M, K), generator=gen, device="cuda", dtype=torch.int8)
    xs = np.float32(0.031)
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    rows = _rows(M, 2)
    acc_o = oracle.spgemm_acc_rows(Xq[cu(rows)].cpu().numpy(), prep["vals"], prep["meta"],
                                   np.arange(rows.size, dtype=np.int64))
    args = dict(w_scale=cu(prep["w_scale"]), x_scale=cu(np.array([xs], np.float32)), bias=cu(bias),
                status_buf=status)
    if out == "i32":
        Y = B.spgemm_i8(Xq, Wpk, N, out_type=B.OUT_I32, status_buf=status)
        assert np.array_equal(Y[cu(rows)].cpu().numpy(), acc_o)
        # sum_m acc[m, n] = Wq[n, :] . sum_m Xq[m, :], exact in 64-bit integers, over every output
        col = torch.zeros(N, dtype=torch.int64, device="cuda")
        for i in range(0, M, 200_000):
            col += Y[i:i + 200_000].sum(dim=0, dtype=torch.int64)
        xsum = torch.zeros(K, dtype=torch.int64, device="cuda")
        for i in range(0, M, 200_000):
            xsum += Xq[i:i + 200_000].sum(dim=0, dtype=torch.int64)
        want = prep["Wq"].astype(np.int64) @ xsum.cpu().numpy()
        assert np.array_equal(col.cpu().numpy(), want)
    elif out == "f16":
        Y = B.spgemm_i8(Xq, Wpk, N, out_type=B.OUT_F16, **args)
        Y_o = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=0, out_type=0)
        assert f16_ulp_distance(Y[cu(rows)].cpu().numpy(), Y_o).max() == 0
    else:
        y = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=0, out_type=0).astype(np.float32)
        out_scale = np.float32(np.abs(y).max() / 127.0)
        Y = B.spgemm_i8(Xq, Wpk, N, out_type=B.OUT_I8, out_scale=cu(np.array([out_scale], np.float32)), **args)
        Q_o = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=0, out_type=1, out_scale=out_scale)
        assert np.array_equal(Y[cu(rows)].cpu().numpy(), Q_o)
    assert status.cpu().tolist() == [0, 0, 0, 0]
