"""GPU parity of the patch-embedding path (Sec. 3.3): gpusq_patch_quant against the oracle's image
codes and patch rows (bit-exact), then the sparse GEMM on those rows against the oracle's strided
convolution (INT32 bit-exact) and its epilogue (FP16 within 1 ulp, exact without activation)."""
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


# B, C, H, W, P, D: the three vector widths of the kernel (P % 8, P % 4, P % 2), padded and unpadded
# reduction lengths, one patch per image, non-square images, widths below a feature tile
SMALL = [
    (2, 3, 32, 32, 16, 128), (3, 3, 28, 28, 14, 40), (2, 3, 16, 24, 4, 96), (1, 3, 8, 8, 8, 8),
    (5, 1, 12, 20, 2, 16), (2, 4, 64, 32, 32, 24), (4, 3, 42, 14, 14, 1280), (1, 8, 6, 6, 6, 8),
    # more items than one pass of the grid, and the narrower vector widths on wider images
    (2, 3, 28, 56, 14, 16), (1, 2, 4, 16, 2, 8), (3, 3, 12, 40, 4, 48), (1300, 1, 16, 16, 16, 8),
]


@pytest.mark.parametrize("Bn,C,H,W,P,D", SMALL)
@pytest.mark.parametrize("given", [False, True])
def test_patch_quant_and_embedding_small(B, Bn, C, H, W, P, D, given):
    d = inputs.random_patch(Bn + C + H + P, Bn, C, H, W, P, D)
    K = C * P * P
    Kp = (K + 15) // 16 * 16
    prep = oracle.patch_embed_weight(d["W4"], Kp)
    x_scale = np.float32(0.011) if given else None        # a supplied scale below max/127: some codes clamp
    r = oracle.patch_embed_forward(d["img"], prep, P, d["bias"], x_scale=x_scale)

    if given:
        Xq, xs = B.patch_quant(cu(d["img"]), P, Kp, x_scale=cu(np.array([x_scale], np.float32)),
                               scale_mode=B.SCALE_GIVEN)
        assert (np.abs(r["imgq"]) == 127).any()
    else:
        Xq, xs = B.patch_quant(cu(d["img"]), P, Kp)
    assert xs.cpu().numpy()[0] == r["x_scale"]
    assert np.array_equal(Xq.cpu().numpy(), r["Xq"])

    # offline weight steps on the flattened, zero-padded conv weight
    Wf = B.flatten_conv_weight(cu(d["W4"]), Kp)
    Wq, ws = B.quant_weight(B.prune24(Wf))
    assert np.array_equal(Wq.cpu().numpy(), prep["Wq"])
    vals, meta = B.compress24(Wq)
    Wpk = B.pack24(vals, meta)

    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    acc = B.spgemm_i8(Xq, Wpk, D, out_type=B.OUT_I32, status_buf=status).cpu().numpy()
    conv, macs = oracle.patch_conv_acc(r["imgq"], prep["Wq"][:, :K].reshape(D, C, P, P))
    assert np.array_equal(acc, conv)                      # the GEMM on patch rows is the convolution
    assert macs == Bn * C * H * W * D
    Y = B.spgemm_i8(Xq, Wpk, D, ws, xs, cu(d["bias"]), out_type=B.OUT_F16, status_buf=status).cpu().numpy()
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert f16_ulp_distance(Y, r["Y"]).max() == 0


def test_patch_quant_reuses_the_quant_act_workspace(B):
    # one zero-filled workspace serves gpusq_quant_act and gpusq_patch_quant in any order
    d = inputs.random_patch(7, 2, 3, 32, 32, 16, 128)
    ws = torch.zeros((B.quant_act_workspace(8, 768),), dtype=torch.uint8, device="cuda")
    X = cu(d["img"].reshape(8, -1))
    a1, s1 = B.quant_act(X, workspace=ws)
    p1, t1 = B.patch_quant(cu(d["img"]), 16, workspace=ws)
    a2, s2 = B.quant_act(X, workspace=ws)
    p2, t2 = B.patch_quant(cu(d["img"]), 16, workspace=ws)
    assert torch.equal(a1, a2) and torch.equal(p1, p2) and torch.equal(s1, s2) and torch.equal(t1, s1) and torch.equal(t2, s1)
    imgq, xs = oracle.quant_act(d["img"].reshape(1, -1))
    assert np.array_equal(a1.cpu().numpy().reshape(-1), imgq.reshape(-1)) and s1.cpu().numpy()[0] == xs
    assert np.array_equal(p1.cpu().numpy(), oracle.patch_rows(imgq.reshape(d["img"].shape), 16))


@pytest.mark.parametrize("name", list(inputs.PATCH_CONFIGS))
def test_patch_config_full_size(B, name):
    cfg = inputs.PATCH_CONFIGS[name]
    d = inputs.make_patch_inputs(cfg)
    prep = oracle.patch_embed_weight(d["W4"], cfg.Kp)
    rng = np.random.default_rng(cfg.cid)
    T = cfg.tokens
    rows = np.unique(np.concatenate([[0, 1, T - 1, T - 2, T // 2, 195, 196, 197],
                                     rng.integers(0, T, 24)]).astype(np.int64))
    rows = rows[rows < T]
    r = oracle.patch_embed_forward(d["img"], prep, cfg.P, d["bias"], rows=rows)

    Xq, xs = B.patch_quant(cu(d["img"]), cfg.P, cfg.Kp)
    assert xs.cpu().numpy()[0] == r["x_scale"]
    assert np.array_equal(Xq.cpu().numpy(), r["Xq"])      # every code of every patch row

    Wf = B.flatten_conv_weight(cu(d["W4"]), cfg.Kp)
    Wq, ws = B.quant_weight(B.prune24(Wf))
    assert np.array_equal(Wq.cpu().numpy(), prep["Wq"])
    vals, meta = B.compress24(Wq)
    Wpk = B.pack24(vals, meta)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    acc = B.spgemm_i8(Xq, Wpk, cfg.D, out_type=B.OUT_I32, status_buf=status)
    assert np.array_equal(acc[cu(rows)].cpu().numpy(), r["acc"])
    # column sums tie every accumulator to the image codes: sum_t acc[t, d] = Wq[d, :] . sum_t Xq[t, :]
    col = acc.sum(dim=0, dtype=torch.int64).cpu().numpy()
    want = prep["Wq"].astype(np.int64) @ r["Xq"].astype(np.int64).sum(0)
    assert np.array_equal(col, want)
    Y = B.spgemm_i8(Xq, Wpk, cfg.D, ws, xs, cu(d["bias"]), out_type=B.OUT_F16, status_buf=status)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert f16_ulp_distance(Y[cu(rows)].cpu().numpy(), r["Y"]).max() == 0
    assert torch.isfinite(Y).all()
