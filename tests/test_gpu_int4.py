"""GPU parity of the INT4 model (Sec. 3.1: pair-wise 4:8 sparsity) against the oracle: every stage of
the weight preparation bit for bit in the paper's 4-bit storage format, the 4-bit activation codes,
and the sums of the sparse GEMM, which the library computes on the INT8 2:4 path with regrouped
columns (there is no 4-bit tensor-core kind on this GPU) and which must equal the oracle's
decompress-then-multiply sums exactly."""
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


def f16_ulp_distance(a, b):
    def key(h):
        u = h.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(np.ascontiguousarray(a)) - key(np.ascontiguousarray(b)))


def regroup(K):
    """new column k holds old column regroup(K)[k]: inside every eight, first elements of the sub-chunks, then the second."""
    k = np.arange(K)
    return 8 * (k // 8) + 2 * (k % 4) + (k % 8) // 4


@pytest.mark.parametrize("N,K", [(1, 16), (96, 48), (768, 192), (200, 1280), (3072, 768)])
def test_weight_preparation_bit_exact(B, N, K):
    W = inputs.random_layer(N + K, 4, N, K)["W"]
    W[0, :8] = [1, 1, -1, -1, 2, 0, 0, 2]                  # all four sub-chunks weigh the same: lower indices win
    if N > 1:
        W[1, :16] = 0.0                                    # all-zero chunks: two sub-chunks are still "kept"
    prep = oracle.prepare_weight4(W)
    Wp, mask = B.prune48(cu(W), want_mask=True)
    Wq, ws = B.quant_weight4(Wp)
    vals4, meta4 = B.compress48(Wq)
    assert np.array_equal(Wp.cpu().numpy(), prep["Wp"])
    assert np.array_equal(mask.cpu().numpy(), prep["mask"])
    assert np.array_equal(Wq.cpu().numpy(), prep["Wq"])
    assert np.array_equal(ws.cpu().numpy(), prep["w_scale"])
    assert np.array_equal(vals4.cpu().numpy(), prep["vals"])
    assert np.array_equal(meta4.cpu().numpy(), prep["meta"])
    assert vals4.numel() + meta4.numel() == N * K * 5 // 16          # 0.3125 bytes per weight (Sec. 3.1: 37.5 % saved)
    # expansion: the same matrix with regrouped columns, as a well-formed 2:4 INT8 operand
    vals, meta = B.expand48(vals4, meta4)
    Wr = oracle.decompress24(vals.cpu().numpy(), meta.cpu().numpy())
    assert np.array_equal(Wr, prep["Wq"][:, regroup(K)])
    assert np.array_equal(B.decompress24(vals, meta).cpu().numpy(), Wr)
    # in place
    Win = cu(W)
    B.load().gpusq_prune48(Win.data_ptr(), Win.data_ptr(), None, N, K, torch.cuda.current_stream().cuda_stream)
    assert np.array_equal(Win.cpu().numpy(), prep["Wp"])


@pytest.mark.parametrize("M,K,dist", [(1, 16, "normal"), (197, 192, "normal"), (1576, 768, "normal"),
                                      (333, 1280, "student_t4")])
def test_activation_codes(B, M, K, dist):
    X = inputs.random_layer(3 * M + K, M, 8, K, x_dist=dist)["X"]
    Xq_o, s_o = oracle.quant_act4(X)
    Xq, s = B.quant_act4(cu(X))
    assert s.cpu().numpy()[0] == s_o
    assert np.array_equal(Xq.cpu().numpy(), Xq_o[:, regroup(K)])
    given = np.float32(0.4 * float(s_o))                   # a supplied scale: values beyond 7 * scale clamp
    Xq_o2, _ = oracle.quant_act4(X, x_scale=given)
    Xq2, _ = B.quant_act4(cu(X), x_scale=cu(np.array([given], np.float32)), scale_mode=B.SCALE_GIVEN)
    assert np.array_equal(Xq2.cpu().numpy(), Xq_o2[:, regroup(K)])
    assert (np.abs(X.astype(np.float32)) > 7.5 * given).any() and (np.abs(Xq_o2) == 7).any()      # some values do clamp


@pytest.mark.parametrize("M,N,K", [(16, 128, 16), (197, 256, 192), (1000, 96, 48), (1576, 768, 192), (333, 384, 1280)])
@pytest.mark.parametrize("act", [0, 1])
def test_layer_sums_and_output(B, M, N, K, act):
    d = inputs.random_layer(11 * M + N + K, M, N, K)
    prep = oracle.prepare_weight4(d["W"])
    ref = oracle.layer_forward4(d["X"], prep, d["bias"], act=act, threads=oracle.host_cores())
    Wq, ws = B.quant_weight4(B.prune48(cu(d["W"])))
    Wpk = B.pack24(*B.expand48(*B.compress48(Wq)))
    Xq, xs = B.quant_act4(cu(d["X"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    acc = B.spgemm_i8(Xq, Wpk, N, out_type=B.OUT_I32, status_buf=status)
    Y = B.spgemm_i8(Xq, Wpk, N, ws, xs, cu(d["bias"]), act=act, out_type=B.OUT_F16, status_buf=status)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])   # the 4-bit model's sums, exactly
    dist = f16_ulp_distance(Y.cpu().numpy(), ref["Y"])
    assert dist.max() <= (1 if act else 0)


def test_deit_base_fc1_full_size(B):
    # the benchmark's largest-output layer in the 4-bit model, every output element against the oracle
    cfg = inputs.CONFIGS["deit_base_b64"]
    d = inputs.make_layer_inputs(cfg, 2)
    L = cfg.layers[2]
    prep = oracle.prepare_weight4(d["W"])
    ref = oracle.layer_forward4(d["X"], prep, d["bias"], act=1, threads=oracle.host_cores())
    Wq, ws = B.quant_weight4(B.prune48(cu(d["W"])))
    Wpk = B.pack24(*B.expand48(*B.compress48(Wq)))
    Xq, xs = B.quant_act4(cu(d["X"]))
    acc = B.spgemm_i8(Xq, Wpk, L.N, out_type=B.OUT_I32)
    Y = B.spgemm_i8(Xq, Wpk, L.N, ws, xs, cu(d["bias"]), act=B.ACT_GELU, out_type=B.OUT_F16)
    assert xs.item() == ref["x_scale"]
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert f16_ulp_distance(Y.cpu().numpy(), ref["Y"]).max() <= 1
