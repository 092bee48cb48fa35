"""Chained layers (Sec. 2.2: quantise / de-quantise nodes through the whole deployed model): the
epilogue that reports the largest magnitude it wrote, the one-pass quantise node that uses it, and a
whole transformer block's linears chained on the device against the oracle chained the same way.
What lies between the linears of a real block (attention, LayerNorm, residuals: not sparsified,
Sec. 3.2) is stood in for by exact data movement, so that every link can be compared to the bit."""
import numpy as np
import pytest

import oracle
from paper_2305_10727_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F16_ULP_TOL = 1


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


@pytest.mark.parametrize("M,N,K,tiling", [
    (197, 256, 192, None), (1576, 768, 192, None), (333, 384, 128, None), (1000, 96, 48, None),
    (1001, 512, 256, (96, 3)), (130, 8, 16, None), (12608, 768, 256, None)])
@pytest.mark.parametrize("act", [0, 1])
def test_absmax_epilogue(B, M, N, K, tiling, act):
    d = inputs.random_layer(31 * M + N + K, M, N, K)
    prep = oracle.prepare_weight(d["W"])
    ref = oracle.layer_forward(d["X"], prep, d["bias"], act=act, threads=oracle.host_cores())
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    Xq, xs = cu(ref["Xq"]), cu(np.array([ref["x_scale"]], np.float32))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    if tiling:
        B.set_tile_mix(*tiling)
    try:
        Y0 = B.spgemm_i8(Xq, Wpk, N, cu(prep["w_scale"]), xs, cu(d["bias"]), act=act, status_buf=status)
        Y, amax = B.spgemm_i8_absmax(Xq, Wpk, N, cu(prep["w_scale"]), xs, cu(d["bias"]), act=act, status_buf=status)
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    Yh = Y.cpu().numpy()
    assert np.array_equal(Yh.view(np.uint16), Y0.cpu().numpy().view(np.uint16))      # the same output, bit for bit
    assert f16_ulp_distance(Yh, ref["Y"]).max() <= (F16_ULP_TOL if act else 0)
    # the number reported is the largest magnitude of what was written (rows past M and features past N
    # of the last tiles do not count) ...
    got = np.float32(amax.cpu().numpy()[0])
    assert got == np.abs(Yh.astype(np.float32)).max()
    # ... which without GELU is the oracle's own maximum, to the bit
    if act == 0:
        assert got == np.abs(ref["Y"].astype(np.float32)).max()
    # merged, not overwritten: a larger value already there stays
    big = torch.full((1,), 1.0e4, dtype=torch.float32, device="cuda")
    B.spgemm_i8_absmax(Xq, Wpk, N, cu(prep["w_scale"]), xs, cu(d["bias"]), act=act, y_absmax=big)
    assert big.item() == 1.0e4


@pytest.mark.parametrize("M,K", [(1, 8), (197, 192), (1576, 768), (333, 1288)])
def test_quant_act_absmax_equals_computed_scale(B, M, K):
    X = inputs.random_layer(5 * M + K, M, 8, K)["X"]
    Xq_o, s_o = oracle.quant_act(X)
    amax = np.abs(X.astype(np.float32)).max()
    Xq, s = B.quant_act_absmax(cu(X), cu(np.array([amax], np.float32)))
    assert s.cpu().numpy()[0] == s_o
    assert np.array_equal(Xq.cpu().numpy(), Xq_o)
    # an all-zero tensor: scale 1, codes 0
    Z = np.zeros((4, 16), np.float16)
    Zq, zs = B.quant_act_absmax(cu(Z), cu(np.zeros(1, np.float32)))
    assert zs.item() == 1.0 and not Zq.cpu().numpy().any()


def test_chained_block(B):
    # qkv -> [attention stand-in: the first H columns, copied] -> proj (reports max |y|) ->
    # [residual / LayerNorm stand-in: identity] -> one-pass quantise from that maximum -> fc1 + GELU writing
    # INT8 with a calibrated scale -> fc2.  Every tensor that crosses a link is compared with the oracle's.
    M, H, F = 777, 128, 512
    cfgs = [inputs.random_layer(100 + i, M, n, k) for i, (n, k) in enumerate([(3 * H, H), (H, H), (F, H), (H, F)])]
    preps = [oracle.prepare_weight(c["W"]) for c in cfgs]
    T = oracle.host_cores()

    # ---- the oracle's chain
    o_qkv = oracle.layer_forward(cfgs[0]["X"], preps[0], cfgs[0]["bias"], act=0, threads=T)
    o_att = np.ascontiguousarray(o_qkv["Y"][:, :H])
    o_proj = oracle.layer_forward(o_att, preps[1], cfgs[1]["bias"], act=0, threads=T)
    o_fc1 = oracle.layer_forward(o_proj["Y"], preps[2], cfgs[2]["bias"], act=1, threads=T)
    y_scale = np.float32(np.abs(o_fc1["Y"].astype(np.float32)).max() / 127.0)         # calibration
    o_q1 = oracle.epilogue(o_fc1["acc"], preps[2]["w_scale"], o_fc1["x_scale"], cfgs[2]["bias"], act=1, out_type=1,
                           out_scale=y_scale)
    o_acc2 = oracle.spgemm_acc(o_q1, preps[3]["vals"], preps[3]["meta"], threads=T)
    o_y2 = oracle.epilogue(o_acc2, preps[3]["w_scale"], y_scale, cfgs[3]["bias"], act=0, out_type=0)

    # ---- the device's chain
    dev = [dict(Wpk=B.pack24(cu(p["vals"]), cu(p["meta"])), ws=cu(p["w_scale"]), bias=cu(c["bias"]))
           for p, c in zip(preps, cfgs)]
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    Xq0, xs0 = B.quant_act(cu(cfgs[0]["X"]))
    Yqkv = B.spgemm_i8(Xq0, dev[0]["Wpk"], 3 * H, dev[0]["ws"], xs0, dev[0]["bias"], status_buf=status)
    att = Yqkv[:, :H].contiguous()
    Xq1, xs1 = B.quant_act(att)
    Yproj, amax = B.spgemm_i8_absmax(Xq1, dev[1]["Wpk"], H, dev[1]["ws"], xs1, dev[1]["bias"], status_buf=status)
    Xq2, xs2 = B.quant_act_absmax(Yproj, amax)
    ys = cu(np.array([y_scale], np.float32))
    Q1 = B.spgemm_i8(Xq2, dev[2]["Wpk"], F, dev[2]["ws"], xs2, dev[2]["bias"], act=B.ACT_GELU, out_type=B.OUT_I8,
                     out_scale=ys, status_buf=status)
    Y2 = B.spgemm_i8(Q1, dev[3]["Wpk"], H, dev[3]["ws"], ys, dev[3]["bias"], status_buf=status)
    assert status.cpu().tolist() == [0, 0, 0, 0]

    # ---- link by link: everything up to fc1's input is a fixed IEEE sequence, hence equal to the bit
    assert np.array_equal(Xq0.cpu().numpy(), o_qkv["Xq"]) and xs0.item() == o_qkv["x_scale"]
    assert np.array_equal(Yqkv.cpu().numpy().view(np.uint16), o_qkv["Y"].view(np.uint16))
    assert np.array_equal(Xq1.cpu().numpy(), o_proj["Xq"]) and xs1.item() == o_proj["x_scale"]
    assert np.array_equal(Yproj.cpu().numpy().view(np.uint16), o_proj["Y"].view(np.uint16))
    assert amax.item() == np.abs(o_proj["Y"].astype(np.float32)).max()
    assert np.array_equal(Xq2.cpu().numpy(), o_fc1["Xq"]) and xs2.item() == o_fc1["x_scale"]
    # fc1's codes: the kernel's GELU may move a code at a rounding tie
    steps = np.abs(Q1.cpu().numpy().astype(np.int32) - o_q1.astype(np.int32))
    assert steps.max() <= 1 and (steps != 0).mean() < 1e-3
    # fc2: rows whose input codes all agree are the oracle's to the bit; the others are off by at most the
    # moved codes times the largest de-quantised weight, plus the binary16 rounding
    y2, y2_o = Y2.cpu().numpy().astype(np.float32), o_y2.astype(np.float32)
    same = steps.sum(axis=1) == 0
    assert same.any() and np.array_equal(y2[same], y2_o[same])
    w_max = float((np.abs(preps[3]["Wq"]).max(axis=1) * preps[3]["w_scale"]).max())
    bound = steps.sum(axis=1, keepdims=True) * w_max * float(y_scale) + np.abs(y2_o) * 2.0 ** -10 + 2.0 ** -24
    assert (np.abs(y2 - y2_o) <= bound).all()
