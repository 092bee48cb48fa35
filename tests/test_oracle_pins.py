"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these tests calls the CUDA library.  Each pin checks the oracle against
something other than its own formula: numbers printed in the paper, a
hand-worked example, brute force over a complete small domain, invariants,
closed forms, or an independent library routine (numpy / scipy).
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2305_10727_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = vals
    return out


# --------------------------------------------------------------------------- O1
def test_prune24_at_most_two_nonzeros_per_group():
    # Sec. 1: two values from every four contiguous elements on rows must be zero
    W = inputs.random_layer(3, 4, 96, 64)["W"]
    Wp = oracle.prune24(W)
    nz = (Wp.reshape(96, 16, 4) != 0).sum(-1)
    assert nz.max() <= 2
    kept = Wp != 0
    assert np.array_equal(Wp[kept], W[kept])          # kept values are unchanged


def test_prune24_exhaustive_small_domain_matches_sorted_top2():
    # every 4-vector over {0, +-1, +-2}: 625 cases, all tie patterns included
    vals = [0.0, 1.0, -1.0, 2.0, -2.0]
    groups = np.array(list(itertools.product(vals, repeat=4)), np.float32)   # [625, 4]
    Wp, mask = oracle.prune24(groups, return_mask=True)
    for g, p, mk in zip(groups, Wp, mask[:, 0]):
        order = np.argsort(-np.abs(g), kind="stable")     # magnitude desc, index asc
        keep = sorted(order[:2].tolist())
        expect = np.zeros(4, np.float32)
        expect[keep] = g[keep]
        assert np.array_equal(p, expect), (g, p)
        assert mk == (1 << keep[0]) | (1 << keep[1])


def test_prune24_keeps_largest_magnitudes_random():
    W = inputs.random_layer(5, 4, 64, 128)["W"]
    Wp, mask = oracle.prune24(W, return_mask=True)
    a = np.abs(W).reshape(64, 32, 4)
    bits = ((mask[..., None] >> np.arange(4)) & 1).astype(bool)
    assert (bits.sum(-1) == 2).all()
    kept_min = np.where(bits, a, np.inf).min(-1)
    dropped_max = np.where(~bits, a, -np.inf).max(-1)
    assert (kept_min >= dropped_max).all()


# ----------------------------------------------------------------------- O2 / O4
def test_quant_weight_error_bound_range_and_absmax():
    W = oracle.prune24(inputs.random_layer(7, 4, 48, 256)["W"])
    Wq, s = oracle.quant_weight(W)
    assert Wq.min() >= -127 and Wq.max() <= 127
    err = np.abs(W.astype(np.float64) - s.astype(np.float64)[:, None] * Wq)
    assert (err <= s.astype(np.float64)[:, None] / 2 * (1 + 1e-6)).all()
    # the largest magnitude of each row maps to +-127; scale is that magnitude / 127
    assert (np.abs(Wq).max(1) == 127).all()
    assert np.allclose(s, np.abs(W).max(1) / 127.0, rtol=1e-7)
    # per output channel: rescaling one row changes only that row's scale, not its codes
    W2 = W.copy()
    W2[3] *= 4.0
    Wq2, s2 = oracle.quant_weight(W2)
    assert np.array_equal(Wq2, Wq) and s2[3] == 4 * s[3] and np.array_equal(np.delete(s2, 3), np.delete(s, 3))


def test_quant_round_half_even_and_clamp():
    # scale is exactly 1 when the row maximum is 127
    row = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 126.5, -126.5, 0.49, -127.0]], np.float32)
    Wq, s = oracle.quant_weight(row)
    assert s[0] == 1.0
    assert Wq[0].tolist() == [127, 0, 2, 2, 0, -2, -2, 4, 126, -126, 0, -127]
    # zero row: scale 1, codes 0
    Wq0, s0 = oracle.quant_weight(np.zeros((1, 8), np.float32))
    assert s0[0] == 1.0 and not Wq0.any()


def test_quant_act_supplied_scale_clamps_to_127():
    X = np.array([[300.0, -300.0, 127.4, -128.6, 1.0, 0.0, 2.5, -2.5]], np.float16)
    Xq, s = oracle.quant_act(X, x_scale=1.0)
    assert s == 1.0
    assert Xq[0].tolist() == [127, -127, 127, -127, 1, 0, 2, -2]


def test_quant_act_per_tensor_scale_and_bound():
    X = inputs.random_layer(11, 37, 8, 64)["X"]
    Xq, s = oracle.quant_act(X)
    xf = X.astype(np.float64)
    assert np.isclose(float(s), np.abs(xf).max() / 127.0, rtol=1e-7)      # one scale for the tensor
    assert np.abs(Xq).max() == 127
    assert (np.abs(xf - float(s) * Xq) <= float(s) / 2 * (1 + 1e-6)).all()
    Xz, sz = oracle.quant_act(np.zeros((2, 8), np.float16))
    assert sz == 1.0 and not Xz.any()


def test_f16_conversions_match_numpy():
    lib_bits = np.arange(65536, dtype=np.uint16)
    as_f32 = lib_bits.view(np.float16).astype(np.float32)
    mine = np.array([oracle.f16_bits_to_f32(int(b)) for b in lib_bits], np.float32)
    same = (mine == as_f32) | (np.isnan(mine) & np.isnan(as_f32))
    assert same.all()
    rng = np.random.default_rng(0)
    xs = np.concatenate([
        rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 6, 4000).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 65536.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25,
                  1.5 * 2.0 ** -25, 3 * 2.0 ** -25, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -25, 1084.5, 1085.5,
                  np.inf, -np.inf], np.float32),
        # every tie between two neighbouring binary16 values in [1, 2)
        (1.0 + (np.arange(1024, dtype=np.float64) + 0.5) / 1024.0).astype(np.float32),
    ])
    with np.errstate(over="ignore"):
        want = xs.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f32_to_f16_bits(float(x)) for x in xs], np.uint16)
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------- O3
def test_compress_roundtrip_bytes_and_nibbles():
    W = inputs.random_layer(13, 4, 40, 192)["W"]
    Wq, _ = oracle.quant_weight(oracle.prune24(W))
    vals, meta = oracle.compress24(Wq)
    assert vals.shape == (40, 96) and meta.shape == (40, 24)       # K/2 values, 2 bits per kept value
    assert np.array_equal(oracle.decompress24(vals, meta), Wq)
    nibs = np.concatenate([(meta & 0xF).ravel(), (meta >> 4).ravel()])
    assert set(np.unique(nibs).tolist()) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}   # i0 < i1
    # nibble of group g is the low nibble of byte g/2 for even g: check by brute force on row 0
    for g in range(48):
        byte = meta[0, g // 2]
        nib = (byte >> (4 * (g & 1))) & 0xF
        i0, i1 = nib & 3, nib >> 2
        grp = Wq[0, 4 * g:4 * g + 4]
        assert grp[i0] == vals[0, 2 * g] and grp[i1] == vals[0, 2 * g + 1]
        assert np.count_nonzero(grp) == np.count_nonzero([grp[i0], grp[i1]])


def test_storage_saving_matches_paper():
    g = _read_golden("paper_storage_saving.txt")
    N, K = 64, 256
    Wq, _ = oracle.quant_weight(oracle.prune24(inputs.random_layer(1, 4, N, K)["W"]))
    vals, meta = oracle.compress24(Wq)
    # INT8: bytes(values) + bytes(metadata) against the dense INT8 matrix
    saved_i8 = 100.0 * (1 - (vals.nbytes + meta.nbytes) / (N * K))
    assert saved_i8 == float(g["int8"][1])
    # FP16 with the same metadata: 2 bytes per kept value
    saved_f16 = 100.0 * (1 - (2 * vals.size + meta.nbytes) / (2 * N * K))
    assert saved_f16 == float(g["fp16"][1])
    assert (4 * N * K) / (vals.nbytes + meta.nbytes) == float(g["fp32_over_int8_sparse"][0])


# ----------------------------------------------------------------- hand-worked
def test_hand_worked_example():
    g = _read_golden("hand_worked_2x8.txt")
    f = lambda k, dt, shape: np.array([float(v) for v in g[k]], np.float64).astype(dt).reshape(shape)
    W = f("W", np.float32, (2, 8))
    Wp, mask = oracle.prune24(W, return_mask=True)
    assert np.array_equal(Wp, f("Wp", np.float32, (2, 8)))
    assert mask.ravel().tolist() == [int(v) for v in g["mask"]]
    Wq, ws = oracle.quant_weight(Wp)
    assert ws[0] == float(g["w_scale_row0"][0])
    assert np.array_equal(Wq, f("Wq", np.int8, (2, 8)))
    vals, meta = oracle.compress24(Wq)
    assert np.array_equal(vals, f("vals", np.int8, (2, 4)))
    assert meta.ravel().tolist() == [int(v) for v in g["meta"]]
    X = f("X", np.float16, (2, 8))
    Xq, xs = oracle.quant_act(X)
    assert xs == float(g["x_scale"][0])
    assert np.array_equal(Xq, f("Xq", np.int8, (2, 8)))
    acc = oracle.spgemm_acc(Xq, vals, meta)
    assert np.array_equal(acc, f("acc", np.int32, (2, 2)))           # [M, N]
    bias = f("bias", np.float32, (2,))
    Y = oracle.epilogue(acc, ws, xs, bias)
    assert Y[:, 0].astype(np.float64).tolist() == [float(v) for v in g["Y_f16_channel0"]]
    Y32 = oracle.epilogue(acc, ws, xs, bias, out_type=2)
    assert np.array_equal(Y32, acc)


# --------------------------------------------------------------------------- O5
@pytest.mark.parametrize("M,N,K", [(1, 1, 8), (3, 2, 8), (5, 7, 64), (33, 20, 192)])
def test_spgemm_equals_dense_gemm_of_pruned_matrix(M, N, K):
    # Fig. 1 / Sec. 3.1: the sparse GEMM computes the same result matrix as the dense one
    d = inputs.random_layer(17 + M, M, N, K)
    Wq, _ = oracle.quant_weight(oracle.prune24(d["W"]))
    vals, meta = oracle.compress24(Wq)
    Xq, _ = oracle.quant_act(d["X"])
    acc = oracle.spgemm_acc(Xq, vals, meta)
    dense = np.zeros((M, N), np.int64)
    for m in range(M):                  # brute force, no library matmul
        for n in range(N):
            dense[m, n] = sum(int(Wq[n, k]) * int(Xq[m, k]) for k in range(K))
    assert acc.shape == (M, N) and np.array_equal(acc, dense)
    assert np.array_equal(acc, Xq.astype(np.int64) @ Wq.astype(np.int64).T)   # library cross-check


def test_spgemm_single_group_by_hand():
    # K = 8 is the smallest compressible row: two groups, one metadata byte
    vals = np.array([[3, -5, 7, 0]], np.int8)
    meta = np.array([[0xE | (0x4 << 4)]], np.uint8)   # group 0 -> (2, 3); group 1 -> (0, 1)
    Xq = np.array([[1, 2, 3, 4, 5, 6, 7, 8]], np.int8)
    acc = oracle.spgemm_acc(Xq, vals, meta)
    assert acc.tolist() == [[3 * 3 + (-5) * 4 + 7 * 5 + 0 * 6]]


def test_spgemm_rows_subset_and_extremes():
    d = inputs.random_layer(23, 50, 24, 128)
    prep = oracle.prepare_weight(d["W"])
    Xq, _ = oracle.quant_act(d["X"])
    full = oracle.spgemm_acc(Xq, prep["vals"], prep["meta"])
    rows = np.array([49, 0, 7, 7, 31])
    assert np.array_equal(oracle.spgemm_acc_rows(Xq, prep["vals"], prep["meta"], rows), full[rows])
    # largest possible magnitude: all kept codes and all activations at +-127, K = 5120
    K = 5120
    Wq = np.zeros((1, K), np.int8)
    Wq[0, 0::4] = 127
    Wq[0, 1::4] = -127
    vals, meta = oracle.compress24(Wq)
    X = np.zeros((1, K), np.int8)
    X[0, 0::4] = 127
    X[0, 1::4] = -127
    assert oracle.spgemm_acc(X, vals, meta)[0, 0] == 127 * 127 * K // 2


# --------------------------------------------------------------------------- O6
def test_epilogue_linear_part_single_rounding():
    rng = np.random.default_rng(3)
    acc = rng.integers(-40_000_000, 40_000_000, size=(64, 16)).astype(np.int32)
    acc[0, :4] = [0, 16777217, -16777219, 33554434 + 2]     # float(acc) must round, ties to even
    ws = (rng.random(16).astype(np.float32) + np.float32(0.5)) * np.float32(1e-4)
    xs = np.float32(0.0371)
    bias = rng.standard_normal(16).astype(np.float32) * np.float32(0.01)
    Y = oracle.epilogue(acc, ws, xs, bias)
    # independent: exact rational arithmetic with one rounding per stated step
    for m in range(0, 64, 7):
        for n in range(16):
            t = np.float32(int(acc[m, n]))                          # numpy: int -> binary32, nearest-even
            s = np.float32(ws[n] * xs)
            exact = Fraction(float(t)) * Fraction(float(s)) + Fraction(float(bias[n]))
            y32 = np.float32(float(exact)) if abs(exact) < 2 ** 60 else None
            # float(Fraction) rounds once to binary64; binary32 of that can double-round only on a
            # 2^-29 relative tie, which the random values do not hit
            assert Y[m, n] == np.float16(y32)
    # acc == 0 => y = bias
    Y0 = oracle.epilogue(np.zeros((1, 16), np.int32), ws, xs, bias)
    assert np.array_equal(Y0[0], bias.astype(np.float16))
    # no bias pointer == zero bias
    assert np.array_equal(oracle.epilogue(acc, ws, xs, None), oracle.epilogue(acc, ws, xs, np.zeros(16, np.float32)))


def _ulp_distance_f16(a, b):
    def key(h):
        u = h.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(a) - key(b))


def test_epilogue_gelu_against_scipy_erf_and_closed_forms():
    from scipy.special import erf
    # choose acc, scale so that y = acc * 2^-12 exactly (bias 0): a fine sweep of [-8, 8]
    acc = np.arange(-32768, 32769, 5, dtype=np.int32)[None, :].repeat(1, 0).reshape(-1, 1)
    ws = np.array([2.0 ** -12], np.float32)
    Y = oracle.epilogue(acc, ws, np.float32(1.0), None, act=1)
    y = acc.astype(np.float64) * 2.0 ** -12
    ref = (0.5 * y * (1.0 + erf(y / np.sqrt(2.0)))).astype(np.float32)   # the 1+erf form, scipy
    # the two forms differ by cancellation only where the result is far below binary16's spacing
    with np.errstate(over="ignore"):
        ref16 = ref.astype(np.float16)
    assert _ulp_distance_f16(Y.ravel(), ref16.ravel()).max() <= 1
    zero = oracle.epilogue(np.zeros((1, 1), np.int32), ws, np.float32(1.0), None, act=1)
    assert zero[0, 0] == 0.0
    big = oracle.epilogue(np.array([[40000]], np.int32), ws, np.float32(1.0), None, act=1)
    assert big[0, 0] == np.float16(40000 * 2.0 ** -12)                  # GELU(y) -> y
    neg = oracle.epilogue(np.array([[-60000]], np.int32), ws, np.float32(1.0), None, act=1)
    assert neg[0, 0] == 0.0 and np.signbit(neg[0, 0])                   # -> -0
    # GELU(y) - GELU(-y) = y
    Yf = oracle.epilogue(acc, ws, np.float32(1.0), None, act=1).astype(np.float64).ravel()
    assert np.allclose(Yf - Yf[::-1], y.ravel(), atol=2e-3, rtol=2e-3)
    # minimum of GELU is about -0.17 near y = -0.7518
    assert abs(Yf.min() + 0.16997) < 2e-4 and abs(y.ravel()[Yf.argmin()] + 0.7518) < 5e-2   # binary16 plateau


def test_epilogue_int8_requantised_output():
    rng = np.random.default_rng(5)
    acc = rng.integers(-200000, 200000, size=(32, 8)).astype(np.int32)
    ws = np.full(8, 1e-4, np.float32)
    bias = rng.standard_normal(8).astype(np.float32)
    yf = oracle.epilogue(acc, ws, np.float32(0.05), bias, out_type=0).astype(np.float64)
    out_scale = np.float32(np.abs(yf).max() / 127.0)
    q = oracle.epilogue(acc, ws, np.float32(0.05), bias, out_type=1, out_scale=out_scale)
    assert q.dtype == np.int8 and q.min() >= -127 and q.max() <= 127
    y64 = acc.astype(np.float64) * (1e-4 * 0.05) + bias.astype(np.float64)
    inside = np.abs(y64) < 126.5 * float(out_scale)      # values the clamp cannot touch
    assert (np.abs(y64 - float(out_scale) * q)[inside] <= float(out_scale) * (0.5 + 1e-3)).all()


def test_layer_forward_composition_and_sqnr():
    cfg = inputs.CONFIGS["deit_tiny_fc1"]
    d = inputs.make_layer_inputs(cfg, 0, M=64)
    prep = oracle.prepare_weight(d["W"])
    out = oracle.layer_forward(d["X"], prep, d["bias"], act=0)
    # information only ("parity unpinned"): quantised layer vs the FP32 layer on the pruned weight
    ref = d["X"].astype(np.float32) @ prep["Wp"].T + d["bias"]
    assert oracle.sqnr_db(ref, out["Y"].astype(np.float32)) > 25.0
    rows = np.array([3, 60])
    sub = oracle.layer_forward(d["X"], prep, d["bias"], act=0, rows=rows)
    assert np.array_equal(sub["Y"], out["Y"][rows])


def test_sqnr_hand_value():
    # ref = [1, 1], test = [1, 0.9]: signal 2, noise 0.01 -> 10 log10(200) dB; equal scaling of both leaves it alone
    want = 10.0 * np.log10(200.0)
    got = oracle.sqnr_db(np.array([1.0, 1.0], np.float32), np.array([1.0, 0.9], np.float32))
    assert abs(got - want) < 1e-5                        # 0.9 is not exact in binary32
    assert abs(oracle.sqnr_db(np.array([4.0, 4.0], np.float32), np.array([4.0, 3.5], np.float32))
               - 10.0 * np.log10(32.0 / 0.25)) < 1e-12   # exact inputs: 21.07 dB


def test_row_parallel_driver_equals_single_thread():
    # the several-thread driver only splits the token rows over plain calls of the same C routines:
    # on the whole of the small workload config its results equal the single-threaded ones bit for bit
    cfg = inputs.CONFIGS["deit_tiny_fc1"]
    d = inputs.make_layer_inputs(cfg, 0)
    prep = oracle.prepare_weight(d["W"])
    one = oracle.layer_forward(d["X"], prep, d["bias"], act=1)
    for threads in (2, 3, 7):
        many = oracle.layer_forward(d["X"], prep, d["bias"], act=1, threads=threads)
        assert np.array_equal(one["acc"], many["acc"])
        assert np.array_equal(one["Y"].view(np.uint16), many["Y"].view(np.uint16))
    q1 = oracle.epilogue(one["acc"], prep["w_scale"], one["x_scale"], d["bias"], act=1, out_type=1, out_scale=0.01)
    q4 = oracle.epilogue(one["acc"], prep["w_scale"], one["x_scale"], d["bias"], act=1, out_type=1, out_scale=0.01,
                         threads=4)
    assert np.array_equal(q1, q4)
    assert oracle.host_cores() >= 1


# ---------------------------------------------------------------- patch embedding (Sec. 3.3)

PATCH_SHAPES = [(2, 3, 8, 8, 4, 5), (1, 3, 28, 42, 14, 7), (3, 2, 32, 16, 16, 4), (2, 1, 6, 4, 2, 3)]


def _patch_case(seed, B, C, H, W, P, D):
    rng = np.random.default_rng(seed)
    imgq = rng.integers(-127, 128, (B, C, H, W)).astype(np.int8)
    Wq4 = rng.integers(-127, 128, (D, C, P, P)).astype(np.int8)
    return imgq, Wq4


@pytest.mark.parametrize("B,C,H,W,P,D", PATCH_SHAPES)
def test_patch_conv_matches_library_convolution_and_paper_flop_count(B, C, H, W, P, D):
    torch = pytest.importorskip("torch")
    imgq, Wq4 = _patch_case(1, B, C, H, W, P, D)
    acc, macs = oracle.patch_conv_acc(imgq, Wq4)
    # the strided convolution of a library (exact in float64 on these integers), flattened the usual way
    ref = torch.nn.functional.conv2d(torch.from_numpy(imgq.astype(np.float64)),
                                     torch.from_numpy(Wq4.astype(np.float64)), stride=P)
    ref = ref.flatten(2).transpose(1, 2).reshape(-1, D).numpy()
    assert np.array_equal(acc.astype(np.float64), ref)
    # Sec. 3.3: FLOPs of the patch embedding = 2 * N * C * H * W * D_embed
    assert 2 * macs == 2 * B * C * H * W * D


@pytest.mark.parametrize("B,C,H,W,P,D", PATCH_SHAPES)
def test_patch_rows_times_flat_weight_is_the_convolution(B, C, H, W, P, D):
    imgq, Wq4 = _patch_case(2, B, C, H, W, P, D)
    K = C * P * P
    Kp = (K + 15) // 16 * 16
    X = oracle.patch_rows(imgq, P, Kp)
    assert X.shape == (B * (H // P) * (W // P), Kp)      # one token per patch
    assert not X[:, K:].any()
    # the same rearrangement written with array axes instead of loops
    alt = imgq.reshape(B, C, H // P, P, W // P, P).transpose(0, 2, 4, 1, 3, 5).reshape(-1, K)
    assert np.array_equal(X[:, :K], alt)
    acc, _ = oracle.patch_conv_acc(imgq, Wq4)
    assert np.array_equal(X[:, :K].astype(np.int64) @ Wq4.reshape(D, K).astype(np.int64).T, acc)


def test_patch_rows_by_hand():
    # one 1-channel 4x4 image, 2x2 patches: tokens in reading order, each patch in reading order
    imgq = np.arange(16, dtype=np.int8).reshape(1, 1, 4, 4)
    X = oracle.patch_rows(imgq, 2)
    assert X.tolist() == [[0, 1, 4, 5], [2, 3, 6, 7], [8, 9, 12, 13], [10, 11, 14, 15]]
    # two channels: a token's row is channel 0's patch, then channel 1's
    img2 = np.stack([imgq[0, 0], -imgq[0, 0]])[None]
    assert oracle.patch_rows(img2, 2)[1].tolist() == [2, 3, 6, 7, -2, -3, -6, -7]


def test_patch_embed_forward_is_the_sparse_layer_on_patch_rows():
    d = inputs.random_patch(3, 2, 3, 28, 28, 14, 16)     # K = 588, padded to 592
    prep = oracle.patch_embed_weight(d["W4"], 592)
    assert prep["Wq"].shape == (16, 592) and not prep["Wq"][:, 588:].any()
    # padding the reduction axis changes neither the kept positions nor the codes (groups of four stay aligned)
    Wp_plain = oracle.prune24(d["W4"].reshape(16, 588))
    assert np.array_equal(prep["Wp"][:, :588], Wp_plain)
    assert np.array_equal(prep["Wq"][:, :588], oracle.quant_weight(Wp_plain)[0])
    r = oracle.patch_embed_forward(d["img"], prep, 14, d["bias"])
    # one scale for the whole image tensor, from its largest magnitude
    assert r["x_scale"] == np.float32(np.abs(d["img"].astype(np.float32)).max() / np.float32(127.0))
    # the accumulators are those of the convolution of the pruned, quantised weight over the image codes
    Wq4 = prep["Wq"][:, :588].reshape(16, 3, 14, 14)
    acc, _ = oracle.patch_conv_acc(r["imgq"], Wq4)
    assert np.array_equal(r["acc"], acc)
    # de-quantised output tracks the FP32 convolution of the pruned weight
    Wp4 = prep["Wp"][:, :588].reshape(16, 3, 14, 14).astype(np.float64)
    X = d["img"].astype(np.float64).reshape(2, 3, 2, 14, 2, 14).transpose(0, 2, 4, 1, 3, 5).reshape(-1, 588)
    ref = X @ Wp4.reshape(16, 588).T + d["bias"].astype(np.float64)
    err = np.abs(r["Y"].astype(np.float64) - ref)
    assert err.max() < 0.05 * np.abs(ref).max()


# ---------------------------------------------------------------- FP16 2:4 sparse model (M_SF)

def test_f16_storage_saving_matches_paper():
    # Sec. 3.1: the compressed FP16 operand is 43.75 % smaller than the dense FP16 one
    W = np.random.default_rng(0).standard_normal((64, 256)).astype(np.float32)
    prep = oracle.prepare_weight_f16(W)
    dense_bytes = W.size * 2
    assert Fraction(prep["vals"].nbytes + prep["meta"].nbytes, dense_bytes) == 1 - Fraction(4375, 10000)


def test_f16_compress_roundtrip_and_positions():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((33, 64)).astype(np.float32)
    W[0, :8] = [1e-9, -2.0, 0.0, 3.0, 5.0, 5.0, 5.0, 5.0]      # underflow to zero; a four-way tie
    prep = oracle.prepare_weight_f16(W)
    Wh = prep["Wh"]
    assert np.array_equal(Wh, prep["Wp"].astype(np.float16))    # numpy's RNE narrowing
    assert np.array_equal(oracle.decompress24_f16(prep["vals"], prep["meta"]), Wh)
    # group 0 keeps positions 1 and 3, group 1 (all equal) the two lowest: nibbles 1|3<<2 and 0|1<<2
    assert prep["meta"][0, 0] == (1 | (3 << 2)) | ((0 | (1 << 2)) << 4)
    assert prep["vals"][0, :4].tolist() == [-2.0, 3.0, 5.0, 5.0]
    # the kept positions are those of the pruning mask wherever both kept values stay non-zero in binary16
    mask = prep["mask"]
    for n in range(1, 33):
        for g in range(16):
            nib = (prep["meta"][n, g // 2] >> (4 * (g & 1))) & 0xF
            assert (1 << (nib & 3)) | (1 << (nib >> 2)) == mask[n, g]


@pytest.mark.parametrize("M,N,K", [(5, 7, 16), (9, 12, 64), (3, 4, 200)])
def test_f16_spgemm_is_the_dense_product_of_the_pruned_matrix(M, N, K):
    rng = np.random.default_rng(M + N + K)
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    X = rng.standard_normal((M, K)).astype(np.float16)
    prep = oracle.prepare_weight_f16(W)
    acc, mag = oracle.spgemm_f16_rows(X, prep["vals"], prep["meta"])
    # exact rational arithmetic on the binary16 values
    Wh = prep["Wh"]
    for m in range(M):
        for n in range(N):
            exact = sum(Fraction(float(Wh[n, k])) * Fraction(float(X[m, k])) for k in range(K))
            assert abs(Fraction(acc[m, n]) - exact) <= Fraction(mag[m, n]) * Fraction(1, 2 ** 48)
    assert np.allclose(mag, np.abs(X.astype(np.float64)) @ np.abs(Wh.astype(np.float64)).T, rtol=1e-12)
    # a row subset returns those rows
    sub, _ = oracle.spgemm_f16_rows(X, prep["vals"], prep["meta"], np.array([M - 1, 0]))
    assert np.array_equal(sub, acc[[M - 1, 0]])


def test_f16_epilogue_roundings():
    acc = np.array([[1.0 + 2.0 ** -30, -3.0, 0.1, 1e-9]], np.float64)
    bias = np.array([2.0 ** -12, 0.5, 0.0, 0.0], np.float32)
    Y = oracle.epilogue_f16(acc, bias, act=0)
    # (float)acc drops the 2^-30; binary16 spacing at 1 is 2^-10, so 1 + 2^-12 rounds down to 1.0
    assert Y[0].tolist() == [1.0, -2.5, np.float16(np.float32(0.1)), np.float16(np.float32(1e-9))]
    G = oracle.epilogue_f16(np.array([[0.0, 1.0, -1.0, 10.0]], np.float64), None, act=1).astype(np.float64)
    from math import erf, sqrt
    want = [0.5 * v * (1 + erf(v / sqrt(2))) for v in (0.0, 1.0, -1.0, 10.0)]
    assert np.allclose(G[0], want, rtol=2 ** -11, atol=0)
