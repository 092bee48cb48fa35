"""GPU parity: every kernel of libgpusq against the CPU oracle, element by element,
through the C-ABI (ctypes binding), on seeded inputs that span several tiles
and ragged tails.  Integer stages must be bit-exact; the FP16 epilogue must be
within 1 binary16 ulp of the oracle's FP32 epilogue rounded to binary16."""
import numpy as np
import pytest

import oracle
from paper_2305_10727_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F16_ULP_TOL = 1      # spec tolerance: max-abs-diff <= 1 FP16 ulp


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


# ------------------------------------------------------------------ elementwise
@pytest.mark.parametrize("N,K", [(1, 4), (3, 8), (5, 24), (96, 64), (768, 192), (257, 1280)])
def test_prune24(B, N, K):
    W = inputs.random_layer(N + K, 4, N, K)["W"]
    W[0, :4] = [1.0, -1.0, 1.0, 1.0]                     # ties: the lower indices win
    if K >= 8:
        W[0, 4:8] = 0.0                                  # all-zero group keeps positions 0, 1
    Wp_o, mask_o = oracle.prune24(W, return_mask=True)
    Wp, mask = B.prune24(cu(W), want_mask=True)
    assert np.array_equal(mask.cpu().numpy(), mask_o)
    assert np.array_equal(Wp.cpu().numpy().view(np.uint32), Wp_o.view(np.uint32))
    Win = cu(W)                                          # in place, no mask
    B.prune24(Win, Wp=Win)
    assert np.array_equal(Win.cpu().numpy().view(np.uint32), Wp_o.view(np.uint32))


@pytest.mark.parametrize("N,K", [(1, 4), (7, 8), (33, 24), (768, 192), (130, 5120)])
def test_quant_weight(B, N, K):
    W = oracle.prune24(inputs.random_layer(2 * N + K, 4, N, K)["W"])
    if N > 2:
        W[1] = 0.0                                       # zero row: scale 1
        W[2, :4] = [127.0, 0.5, 1.5, -2.5]               # exact ties when the scale is 1
        W[2, 4:] = 0.0
    Wq_o, s_o = oracle.quant_weight(W)
    Wq, s = B.quant_weight(cu(W))
    assert np.array_equal(s.cpu().numpy(), s_o)
    assert np.array_equal(Wq.cpu().numpy(), Wq_o)


@pytest.mark.parametrize("N,K", [(1, 8), (5, 24), (64, 16), (768, 192), (129, 1288)])
def test_compress_decompress_pack(B, N, K):
    Wq, _ = oracle.quant_weight(oracle.prune24(inputs.random_layer(N + 3 * K, 4, N, K)["W"]))
    vals_o, meta_o = oracle.compress24(Wq)
    vals, meta = B.compress24(cu(Wq))
    assert np.array_equal(vals.cpu().numpy(), vals_o)
    assert np.array_equal(meta.cpu().numpy(), meta_o)
    assert np.array_equal(B.decompress24(vals, meta).cpu().numpy(), Wq)
    # packed blob: zero-padded values, then metadata blocks [N/128][K/128][128][16]
    blob = B.pack24(vals, meta).cpu().numpy()
    Np, Kp = -(-N // 256) * 256, -(-K // 128) * 128     # rows padded to a CTA pair's 256 features
    assert blob.size == B.packed_bytes(N, K) == Np * Kp * 5 // 8
    pv = blob[:Np * Kp // 2].view(np.int8).reshape(Np, Kp // 2)
    assert np.array_equal(pv[:N, :K // 2], vals_o) and not pv[N:].any() and not pv[:, K // 2:].any()
    pm = blob[Np * Kp // 2:].reshape(Np // 128, Kp // 128, 128, 16)
    full = np.full((Np, Kp // 8), 0x44, np.uint8)
    full[:N, :K // 8] = meta_o
    want = full.reshape(Np // 128, 128, Kp // 128, 16).transpose(0, 2, 1, 3)
    assert np.array_equal(pm, want)


@pytest.mark.parametrize("M,K,dist", [(1, 8, "normal"), (197, 192, "normal"), (1576, 768, "normal"),
                                      (333, 1288, "student_t4")])
def test_quant_act(B, M, K, dist):
    X = inputs.random_layer(M + K, M, 8, K, x_dist=dist)["X"]
    Xq_o, s_o = oracle.quant_act(X)
    Xq, s = B.quant_act(cu(X))
    assert s.cpu().numpy()[0] == s_o
    assert np.array_equal(Xq.cpu().numpy(), Xq_o)
    # supplied scale (e.g. learned in training): values beyond 127 * scale clamp
    given = np.float32(0.5 * float(s_o))
    Xq_o2, _ = oracle.quant_act(X, x_scale=given)
    Xq2, s2 = B.quant_act(cu(X), x_scale=cu(np.array([given], np.float32)), scale_mode=B.SCALE_GIVEN)
    assert s2.cpu().numpy()[0] == given
    assert np.array_equal(Xq2.cpu().numpy(), Xq_o2)


def test_quant_act_zero_tensor_and_reused_workspace(B):
    # one zero-filled workspace serves calls of different sizes, back to back
    ws = torch.zeros((B.quant_act_workspace(4096, 4096),), dtype=torch.uint8, device="cuda")
    X = np.zeros((16, 64), np.float16)
    Xq, s = B.quant_act(cu(X), workspace=ws)
    assert s.cpu().numpy()[0] == 1.0 and not Xq.cpu().numpy().any()
    for M, K in [(3000, 1024), (1, 8), (700, 3072), (3000, 1024)]:
        X = inputs.random_layer(M * 7 + K, M, 8, K)["X"]
        Xq_o, s_o = oracle.quant_act(X)
        Xq, s = B.quant_act(cu(X), workspace=ws)
        assert s.cpu().numpy()[0] == s_o
        assert np.array_equal(Xq.cpu().numpy(), Xq_o)
    # the control words and the slots of the grid-wide barrier (everything behind the 2048 words other
    # entry points use for partial maxima) are zero again after every call
    assert not ws.cpu().numpy()[2048 * 4:].any()
    assert B.quant_act_status(ws) == 0


@pytest.mark.parametrize("given", [1e-3, 0.5, 3.0, 1e-30, 1e30])
def test_quant_act_given_scale_extremes(B, given):
    # supplied scales far from the data: saturation to +-127, underflow to 0, reciprocal overflow
    X = inputs.random_layer(77, 257, 8, 264)["X"]
    X[0, :8] = [0.0, -0.0, 65504.0, -65504.0, 6e-8, -6e-8, 1.0, -1.0]
    g = np.float32(given)
    Xq_o, _ = oracle.quant_act(X, x_scale=g)
    Xq, _ = B.quant_act(cu(X), x_scale=cu(np.array([g], np.float32)), scale_mode=B.SCALE_GIVEN)
    assert np.array_equal(Xq.cpu().numpy(), Xq_o)


def test_quant_act_wait_that_runs_out_is_reported(B):
    # A planted failure in an allowed form: the last CTA never publishes its maximum, so the bounded
    # wait of every CTA runs out (5 ms here) and the kernel returns.  Expected: status word
    # GPUSQ_ERR_TIMEOUT, a NaN scale (the real one is written only after every CTA came through),
    # and, after the workspace has been zero-filled again, a correct result from the same buffers.
    X = inputs.random_layer(77, 1576, 8, 768)["X"]
    Xq_o, xs_o = oracle.quant_act(X)
    Xd = cu(X)
    ws = torch.zeros((B.quant_act_workspace(*X.shape),), dtype=torch.uint8, device="cuda")
    Xq = torch.zeros(X.shape, dtype=torch.int8, device="cuda")
    xs = torch.zeros((1,), dtype=torch.float32, device="cuda")
    B.set_quant_act_wait(5_000_000, withhold_last_cta=True)
    try:
        B.quant_act(Xd, Xq=Xq, x_scale=xs, workspace=ws)
        torch.cuda.synchronize()
    finally:
        B.set_quant_act_wait(2_000_000_000, withhold_last_cta=False)
    assert B.quant_act_status(ws) == 7 and "TIMEOUT" in B.status_string(7)
    assert torch.isnan(xs).all()
    ws.zero_()
    B.quant_act(Xd, Xq=Xq, x_scale=xs, workspace=ws)
    assert B.quant_act_status(ws) == 0
    assert xs.cpu().numpy()[0] == xs_o and np.array_equal(Xq.cpu().numpy(), Xq_o)
    # and the workspace serves further calls without being touched by the caller
    B.quant_act(Xd, Xq=Xq, x_scale=xs, workspace=ws)
    assert B.quant_act_status(ws) == 0 and np.array_equal(Xq.cpu().numpy(), Xq_o)


# ------------------------------------------------------------------------- GEMM
def _prep(seed, M, N, K, dist="normal"):
    d = inputs.random_layer(seed, M, N, K, x_dist=dist)
    prep = oracle.prepare_weight(d["W"])
    Xq, xs = oracle.quant_act(d["X"])
    return d, prep, Xq, xs


GEMM_SHAPES = [
    (1, 128, 16), (16, 128, 64), (197, 256, 192), (257, 384, 128), (300, 128, 1280),
    (1576, 768, 192), (1000, 512, 2048),
    # output widths that do not fill the last 128-feature tile (DeiT-Tiny 192 / 576, Swin-Tiny 96 / 288), K < 128
    (394, 96, 48), (197, 192, 192), (500, 288, 96), (333, 576, 192), (70, 8, 16), (129, 200, 64), (65, 5, 32),
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("block_t", [0, 32, 96, 224])
def test_spgemm_int32_bit_exact(B, M, N, K, block_t):
    d, prep, Xq, xs = _prep(M + N + K, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.set_block_tokens(block_t)
    try:
        Y = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_I32, status_buf=status)
        Yd = B.gemm_i8_dense(cu(Xq), cu(prep["Wq"]), out_type=B.OUT_I32, status_buf=status)
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(Y.cpu().numpy(), acc_o)
    assert np.array_equal(Yd.cpu().numpy(), acc_o)       # same C as the dense GEMM (Fig. 1)


@pytest.mark.parametrize("M,N,K,block_t,n_big", [
    (1000, 512, 256, 96, 3), (1576, 768, 192, 224, 2), (700, 256, 128, 64, 0), (2000, 384, 320, 160, 5),
    (333, 576, 192, 128, 1), (900, 1024, 64, 192, 100), (12608, 768, 256, 192, 24), (5000, 96, 48, 128, 7)])
def test_mixed_tile_heights(B, M, N, K, block_t, n_big):
    # token tiles of two heights in one launch (the first n_big of block_t tokens, the rest 32 lower):
    # accumulators bit-exact, FP16 + GELU within one ulp, INT8 exact, sparse and dense instruction
    d, prep, Xq, xs = _prep(7 * M + N + K, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"], threads=oracle.host_cores())
    Y_o = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=1, out_type=0, threads=oracle.host_cores())
    yf = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=0, out_type=0).astype(np.float32)
    out_scale = np.float32(np.abs(yf).max() / 127.0)
    Q_o = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=0, out_type=1, out_scale=out_scale)
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    common = dict(w_scale=cu(prep["w_scale"]), x_scale=cu(np.array([xs], np.float32)), bias=cu(d["bias"]),
                  status_buf=status)
    B.set_tile_mix(block_t, n_big)
    try:
        acc = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_I32, status_buf=status).cpu().numpy()
        accd = B.gemm_i8_dense(cu(Xq), cu(prep["Wq"]), out_type=B.OUT_I32, status_buf=status).cpu().numpy()
        Y = B.spgemm_i8(cu(Xq), Wpk, N, act=B.ACT_GELU, out_type=B.OUT_F16, **common).cpu().numpy()
        Q = B.spgemm_i8(cu(Xq), Wpk, N, act=B.ACT_NONE, out_type=B.OUT_I8,
                        out_scale=cu(np.array([out_scale], np.float32)), **common).cpu().numpy()
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(acc, acc_o)
    assert np.array_equal(accd, acc_o)
    assert f16_ulp_distance(Y, Y_o).max() <= F16_ULP_TOL
    assert np.array_equal(Q, Q_o)


@pytest.mark.parametrize("pairs", [1, 3, 20])
def test_fewer_cta_pairs_same_result(B, pairs):
    # the measurement hook that holds a launch to a few CTA pairs changes who computes a tile, never the tile:
    # accumulators and FP16 + GELU output against the oracle, with many tiles per pair and a ragged end
    M, N, K = 1576, 768, 192
    d, prep, Xq, xs = _prep(5 * M + N + K + pairs, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"], threads=oracle.host_cores())
    Y_o = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=1, out_type=0, threads=oracle.host_cores())
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.set_max_clusters(pairs)
    try:
        acc = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_I32, status_buf=status).cpu().numpy()
        Y = B.spgemm_i8(cu(Xq), Wpk, N, cu(prep["w_scale"]), cu(np.array([xs], np.float32)), cu(d["bias"]),
                        act=B.ACT_GELU, out_type=B.OUT_F16, status_buf=status).cpu().numpy()
    finally:
        B.set_max_clusters(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(acc, acc_o)
    assert f16_ulp_distance(Y, Y_o).max() <= F16_ULP_TOL


def test_gemm_wait_that_runs_out_is_reported(B):
    # A planted failure in an allowed form: the first CTA pair's loads for the last k block of its first tile
    # are never issued, so the MMA issuer's bounded wait (5 ms here) runs out.  Expected: status_buf =
    # {GPUSQ_ERR_TIMEOUT, tile 0, role 1 (MMA issuer), stage}, the kernel returns, and the next call on
    # the same buffers is correct (the context is intact, tensor memory was released).
    M, N, K = 1576, 768, 192
    d, prep, Xq, xs = _prep(123, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    Xd = cu(Xq)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.set_gemm_wait(5000, withhold_loads=True)
    try:
        B.spgemm_i8(Xd, Wpk, N, out_type=B.OUT_I32, status_buf=status)
        torch.cuda.synchronize()
    finally:
        B.set_gemm_wait(2_000_000, withhold_loads=False)
    st = status.cpu().tolist()
    assert st[0] == 7 and st[1] == 0 and st[2] == 1, st
    status.zero_()
    Y = B.spgemm_i8(Xd, Wpk, N, out_type=B.OUT_I32, status_buf=status)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(Y.cpu().numpy(), acc_o)


def test_spgemm_extreme_codes_do_not_overflow(B):
    # every kept code and every activation at +-127, K = 5120: |acc| = 127^2 * K / 2
    M, N, K = 40, 128, 5120
    Wq = np.zeros((N, K), np.int8)
    Wq[:, 0::4] = 127
    Wq[:, 3::4] = -127
    Xq = np.zeros((M, K), np.int8)
    Xq[:, 0::4] = 127
    Xq[:, 3::4] = -127
    vals, meta = oracle.compress24(Wq)
    acc_o = oracle.spgemm_acc(Xq, vals, meta)
    assert acc_o.max() == 127 * 127 * K // 2
    Y = B.spgemm_i8(cu(Xq), B.pack24(cu(vals), cu(meta)), N, out_type=B.OUT_I32)
    assert np.array_equal(Y.cpu().numpy(), acc_o)


@pytest.mark.parametrize("M,N,K", [(197, 256, 192), (1576, 768, 192), (333, 128, 1024), (394, 96, 48),
                                   (591, 576, 192), (100, 200, 64), (77, 8, 16)])
@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("use_bias", [True, False])
def test_epilogue_f16(B, M, N, K, act, use_bias):
    d, prep, Xq, xs = _prep(11 + M + N + K, M, N, K)
    bias = d["bias"] if use_bias else None
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    Y_o = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=act, out_type=0)
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    args = dict(w_scale=cu(prep["w_scale"]), x_scale=cu(np.array([xs], np.float32)),
                bias=None if bias is None else cu(bias), act=act, out_type=B.OUT_F16)
    Y = B.spgemm_i8(cu(Xq), Wpk, N, **args).cpu().numpy()
    Yd = B.gemm_i8_dense(cu(Xq), cu(prep["Wq"]), **args).cpu().numpy()
    dist = f16_ulp_distance(Y, Y_o)
    assert dist.max() <= F16_ULP_TOL
    if act == 0:
        assert dist.max() == 0                           # fixed IEEE sequence: reproducible to the bit
    assert np.array_equal(Y.view(np.uint16), Yd.view(np.uint16))


def test_epilogue_gelu_wide_range(B):
    # drive y across [-12, 12] so the negative tail and the subnormal results are covered
    M, N, K = 256, 128, 64
    d, prep, Xq, xs = _prep(99, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    w_scale = np.full(N, 12.0 / np.abs(acc_o).max(), np.float32)
    Y_o = oracle.epilogue(acc_o, w_scale, np.float32(1.0), None, act=1, out_type=0)
    assert (Y_o.astype(np.float32) < -0.1).any() and (np.abs(Y_o.astype(np.float32)) < 6e-5).any()
    Y = B.spgemm_i8(cu(Xq), B.pack24(cu(prep["vals"]), cu(prep["meta"])), N, w_scale=cu(w_scale),
                    x_scale=cu(np.ones(1, np.float32)), act=B.ACT_GELU, out_type=B.OUT_F16).cpu().numpy()
    assert f16_ulp_distance(Y, Y_o).max() <= F16_ULP_TOL


@pytest.mark.parametrize("M,N,K,block_t", [(514, 256, 1280, 0), (197, 128, 192, 0), (1000, 384, 256, 96),
                                           (33, 128, 64, 32), (1576, 768, 192, 224), (394, 96, 48, 0),
                                           (500, 288, 96, 64), (333, 576, 192, 0), (70, 16, 16, 0)])
@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("shrink", [1.0, 0.3])           # 0.3: a third of the range saturates at +-127
def test_epilogue_int8_requantised(B, act, M, N, K, block_t, shrink):
    d, prep, Xq, xs = _prep(5, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    yf = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=act, out_type=0).astype(np.float32)
    out_scale = np.float32(shrink * np.abs(yf).max() / 127.0)
    Q_o = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=act, out_type=1, out_scale=out_scale)
    assert shrink == 1.0 or (np.abs(Q_o) == 127).mean() > 1e-3
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.set_block_tokens(block_t)
    try:
        Q = B.spgemm_i8(cu(Xq), B.pack24(cu(prep["vals"]), cu(prep["meta"])), N, w_scale=cu(prep["w_scale"]),
                        x_scale=cu(np.array([xs], np.float32)), bias=cu(d["bias"]), act=act, out_type=B.OUT_I8,
                        out_scale=cu(np.array([out_scale], np.float32)), status_buf=status).cpu().numpy()
        Qd = B.gemm_i8_dense(cu(Xq), cu(prep["Wq"]), w_scale=cu(prep["w_scale"]),
                             x_scale=cu(np.array([xs], np.float32)), bias=cu(d["bias"]), act=act,
                             out_type=B.OUT_I8, out_scale=cu(np.array([out_scale], np.float32)),
                             status_buf=status).cpu().numpy()
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(Q, Qd)                         # the dense variant runs the same epilogue
    diff = np.abs(Q.astype(np.int32) - Q_o.astype(np.int32))
    if act == 0:
        assert diff.max() == 0                           # integer decision taken in the same FP32 sequence
    else:
        # GELU differs from the oracle's by < 1 FP32-level rounding: a code may flip only at a tie
        assert diff.max() <= 1 and (diff != 0).mean() < 1e-3


@pytest.mark.parametrize("out_scale", [1e-30, 1e-17, 1e-3, 3e6, 1e9, 1e30])
def test_epilogue_int8_extreme_output_scales(B, out_scale):
    # supplied output scales far from the data: everything saturates, or everything rounds to zero, or the
    # squares the kernel's range test works with leave the binary32 range; no GELU, so exact
    M, N, K = 300, 256, 128
    d, prep, Xq, xs = _prep(17, M, N, K)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    Q_o = oracle.epilogue(acc_o, prep["w_scale"], xs, d["bias"], act=0, out_type=1, out_scale=np.float32(out_scale))
    Q = B.spgemm_i8(cu(Xq), B.pack24(cu(prep["vals"]), cu(prep["meta"])), N, w_scale=cu(prep["w_scale"]),
                    x_scale=cu(np.array([xs], np.float32)), bias=cu(d["bias"]), act=0, out_type=B.OUT_I8,
                    out_scale=cu(np.array([out_scale], np.float32))).cpu().numpy()
    assert np.array_equal(Q, Q_o)


def test_int8_chained_mlp(B):
    # fc1 (GELU) writes requantised INT8 codes that fc2 reads with the same scale: the deployed model's
    # quantise / de-quantise chain (Sec. 2.2).  fc1's codes may differ from the oracle's by one code at
    # rounding ties of the GELU (< 0.1 % of them); fc2's output may then differ by at most that many
    # code steps times the largest de-quantised weight, per row, plus the FP16 rounding.
    M, H, F = 333, 128, 512
    d1 = inputs.random_layer(21, M, F, H)
    d2 = inputs.random_layer(22, M, H, F)
    p1, p2 = oracle.prepare_weight(d1["W"]), oracle.prepare_weight(d2["W"])
    r1 = oracle.layer_forward(d1["X"], p1, d1["bias"], act=1)
    y_scale = np.float32(np.abs(r1["Y"].astype(np.float32)).max() / 127.0)
    q1_o = oracle.epilogue(r1["acc"], p1["w_scale"], r1["x_scale"], d1["bias"], act=1, out_type=1, out_scale=y_scale)
    acc2_o = oracle.spgemm_acc(q1_o, p2["vals"], p2["meta"])
    y2_o = oracle.epilogue(acc2_o, p2["w_scale"], y_scale, d2["bias"], act=0, out_type=0).astype(np.float32)

    Xq, xs = B.quant_act(cu(d1["X"]))
    ys = cu(np.array([y_scale], np.float32))
    q1 = B.spgemm_i8(Xq, B.pack24(cu(p1["vals"]), cu(p1["meta"])), F, cu(p1["w_scale"]), xs, cu(d1["bias"]),
                     act=B.ACT_GELU, out_type=B.OUT_I8, out_scale=ys)
    y2 = B.spgemm_i8(q1, B.pack24(cu(p2["vals"]), cu(p2["meta"])), H, cu(p2["w_scale"]), ys, cu(d2["bias"]),
                     act=B.ACT_NONE, out_type=B.OUT_F16).cpu().numpy().astype(np.float32)
    steps = np.abs(q1.cpu().numpy().astype(np.int32) - q1_o.astype(np.int32))
    assert steps.max() <= 1 and (steps != 0).mean() < 1e-3
    w_max = float((np.abs(p2["Wq"]).max(axis=1) * p2["w_scale"]).max())
    bound = steps.sum(axis=1, keepdims=True) * w_max * float(y_scale) + np.abs(y2_o) * 2.0 ** -10 + 2.0 ** -24
    assert (np.abs(y2 - y2_o) <= bound).all()
    # rows whose codes all agree are reproduced to the bit
    same = steps.sum(axis=1) == 0
    assert same.any() and np.array_equal(y2[same], y2_o[same])


def test_whole_path_on_device_matches_oracle(B):
    # every step of the path on the GPU, chained, against the oracle chained the same way
    cfg = inputs.CONFIGS["deit_tiny_fc1"]
    d = inputs.make_layer_inputs(cfg, 0)
    L = cfg.layers[0]
    prep = oracle.prepare_weight(d["W"])
    ref = oracle.layer_forward(d["X"], prep, d["bias"], act=1)
    Wp, mask = B.prune24(cu(d["W"]), want_mask=True)
    Wq, ws = B.quant_weight(Wp)
    vals, meta = B.compress24(Wq)
    Wpk = B.pack24(vals, meta)
    Xq, xs = B.quant_act(cu(d["X"]))
    acc = B.spgemm_i8(Xq, Wpk, L.N, out_type=B.OUT_I32)
    Y = B.spgemm_i8(Xq, Wpk, L.N, ws, xs, cu(d["bias"]), act=B.ACT_GELU)
    assert np.array_equal(mask.cpu().numpy(), prep["mask"])
    assert np.array_equal(Wq.cpu().numpy(), prep["Wq"])
    assert np.array_equal(ws.cpu().numpy(), prep["w_scale"])
    assert np.array_equal(vals.cpu().numpy(), prep["vals"])
    assert np.array_equal(meta.cpu().numpy(), prep["meta"])
    assert np.array_equal(Xq.cpu().numpy(), ref["Xq"])
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert f16_ulp_distance(Y.cpu().numpy(), ref["Y"]).max() <= F16_ULP_TOL


def test_non_default_stream(B):
    d, prep, Xq, xs = _prep(3, 300, 128, 256)
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
        Y = B.spgemm_i8(cu(Xq), Wpk, 128, out_type=B.OUT_I32)
    s.synchronize()
    assert np.array_equal(Y.cpu().numpy(), acc_o)


def _random_gemm_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        M = int(rng.integers(1, 700))
        N = int(rng.integers(1, 88)) * 8
        K = int(rng.integers(1, 38)) * 16
        block_t = int(rng.choice([0, 32, 64, 128, 160, 192, 224]))
        cases.append((i, M, N, K, block_t, int(rng.integers(0, 2)), bool(rng.integers(0, 2))))
    return cases


@pytest.mark.parametrize("i,M,N,K,block_t,act,use_bias", _random_gemm_cases(40, 2024))
def test_layer_random_shapes(B, i, M, N, K, block_t, act, use_bias):
    # seeded random shapes within the documented limits (N % 8, K % 16), random tile height:
    # accumulators bit-exact, FP16 output within one ulp, INT8 output (when N % 16 == 0) within one code
    d, prep, Xq, xs = _prep(3000 + i, M, N, K)
    bias = d["bias"] if use_bias else None
    acc_o = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    Y_o = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=act, out_type=0)
    Wpk = B.pack24(cu(prep["vals"]), cu(prep["meta"]))
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    common = dict(w_scale=cu(prep["w_scale"]), x_scale=cu(np.array([xs], np.float32)),
                  bias=None if bias is None else cu(bias), act=act, status_buf=status)
    B.set_block_tokens(block_t)
    try:
        acc = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_I32, status_buf=status).cpu().numpy()
        Y = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_F16, **common).cpu().numpy()
        Q = Q_o = None
        if N % 16 == 0:
            out_scale = np.float32(0.7 * np.abs(Y_o.astype(np.float32)).max() / 127.0 + 1e-6)
            Q_o = oracle.epilogue(acc_o, prep["w_scale"], xs, bias, act=act, out_type=1, out_scale=out_scale)
            Q = B.spgemm_i8(cu(Xq), Wpk, N, out_type=B.OUT_I8, out_scale=cu(np.array([out_scale], np.float32)),
                            **common).cpu().numpy()
    finally:
        B.set_block_tokens(0)
    assert status.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(acc, acc_o)
    dist = f16_ulp_distance(Y, Y_o)
    assert dist.max() <= (F16_ULP_TOL if act else 0)
    if Q is not None:
        diff = np.abs(Q.astype(np.int32) - Q_o.astype(np.int32))
        assert diff.max() <= (1 if act else 0)
        # with GELU a code may flip only at a rounding tie: fewer than one in a thousand (at least
        # one element is always allowed, so that tiny outputs are not held to a stricter bar)
        assert (diff != 0).sum() <= max(1, int(1e-3 * diff.size))
