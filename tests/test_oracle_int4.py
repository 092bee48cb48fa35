"""Pins for the oracle's INT4 model (Sec. 3.1: pair-wise structured sparsity at a granularity of 4:8).
No CUDA here.  Each pin checks the oracle against something other than its own formula: the numbers
the paper prints, a hand-worked chunk, brute force over a complete small domain, invariants, and an
independent library routine."""
import itertools

import numpy as np

import oracle
from paper_2305_10727_b200 import inputs


def test_storage_saving_matches_the_paper():
    # Sec. 3.1: the sparse INT4 format saves 37.5 % of the dense INT4 storage; Table 1 prints the INT4
    # models as 12.7x smaller than FP32 -- the compressed linear layers alone are 4 / 0.3125 = 12.8x, the
    # whole model a little less because not every parameter is a compressed linear weight
    N, K = 48, 256
    Wq, _ = oracle.quant_weight4(oracle.prune48(inputs.random_layer(1, 4, N, K)["W"]))
    vals, meta = oracle.compress48(Wq)
    stored = vals.nbytes + meta.nbytes
    assert stored == N * K * 5 // 16                       # 4 of 8 values at 4 bits + 4 bits of indices per chunk
    assert 1.0 - stored / (N * K * 0.5) == 0.375
    assert N * K * 4 / stored == 12.8 and 12.7 <= 12.8


def test_hand_worked_chunk():
    # one row of two chunks, worked by hand from the format's description:
    # chunk 0: sub-chunks (1,-1) (0.5,0) (-3,2) (0,0.25) -> weights 2, 0.5, 5, 0.25 -> keep 0 and 2
    # chunk 1: sub-chunks (1,1) (-1,-1) (2,0) (0,2)     -> weights 2, 2, 2, 2     -> tie: keep 0 and 1
    W = np.array([[1, -1, 0.5, 0, -3, 2, 0, 0.25, 1, 1, -1, -1, 2, 0, 0, 2]], np.float32)
    Wp, mask = oracle.prune48(W, return_mask=True)
    assert np.array_equal(Wp, np.array([[1, -1, 0, 0, -3, 2, 0, 0, 1, 1, -1, -1, 0, 0, 0, 0]], np.float32))
    assert mask.tolist() == [[0b0101, 0b0011]]
    Wq, s = oracle.quant_weight4(Wp)                       # max 3 -> scale 3/7; codes round(w * 7 / 3)
    assert s[0] == np.float32(3.0) / np.float32(7.0)
    assert Wq.tolist() == [[2, -2, 0, 0, -7, 5, 0, 0, 2, 2, -2, -2, 0, 0, 0, 0]]
    vals, meta = oracle.compress48(Wq)
    # kept codes 2,-2,-7,5 | 2,2,-2,-2 as nibbles (two's complement), first code in the low nibble
    assert vals.tolist() == [[0x2 | 0xE << 4, 0x9 | 0x5 << 4, 0x2 | 0x2 << 4, 0xE | 0xE << 4]]
    # indices (0,2) -> 0 | 2<<2 = 8 in the low nibble, (0,1) -> 0 | 1<<2 = 4 in the high nibble
    assert meta.tolist() == [[0x8 | 0x4 << 4]]
    assert np.array_equal(oracle.decompress48(vals, meta), Wq)


def test_prune48_exhaustive_small_domain():
    # every chunk whose four sub-chunks have weights from {0, 1, 2, 3}: all tie patterns
    rows = []
    for w in itertools.product([0.0, 1.0, 2.0, 3.0], repeat=4):
        rows.append([v for pw in w for v in (pw - 0.25 if pw else 0.0, 0.25 if pw else 0.0)])
    W = np.array(rows, np.float32)                         # sub-chunk weight |a| + |b| = pw exactly
    Wp, mask = oracle.prune48(W, return_mask=True)
    for w, p, mk in zip(W, Wp, mask[:, 0]):
        weight = np.abs(w).reshape(4, 2).sum(1)
        order = np.argsort(-weight, kind="stable")          # weight descending, index ascending
        keep = sorted(order[:2].tolist())
        expect = np.zeros(8, np.float32)
        for q in keep:
            expect[2 * q:2 * q + 2] = w[2 * q:2 * q + 2]
        assert np.array_equal(p, expect), (w, p)
        assert mk == (1 << keep[0]) | (1 << keep[1])


def test_pattern_invariants_random():
    W = inputs.random_layer(9, 4, 64, 128)["W"]
    Wp, mask = oracle.prune48(W, return_mask=True)
    pairs = Wp.reshape(64, 16, 4, 2)
    nz = (pairs != 0).any(-1).sum(-1)
    assert nz.max() <= 2                                    # at most two sub-chunks of a chunk are not all zero
    kept = Wp != 0
    assert np.array_equal(Wp[kept], W[kept])
    bits = ((mask[..., None] >> np.arange(4)) & 1).astype(bool)
    assert (bits.sum(-1) == 2).all()
    weight = np.abs(W).reshape(64, 16, 4, 2).sum(-1)
    assert (np.where(bits, weight, np.inf).min(-1) >= np.where(~bits, weight, -np.inf).max(-1)).all()


def test_quantiser_range_and_error_bound():
    W = oracle.prune48(inputs.random_layer(11, 4, 32, 256)["W"])
    Wq, s = oracle.quant_weight4(W)
    assert Wq.min() >= -7 and Wq.max() <= 7 and (np.abs(Wq).max(1) == 7).all()
    err = np.abs(W.astype(np.float64) - s.astype(np.float64)[:, None] * Wq)
    assert (err <= s.astype(np.float64)[:, None] / 2 * (1 + 1e-6)).all()
    X = inputs.random_layer(12, 50, 8, 64)["X"]
    Xq, xs = oracle.quant_act4(X)
    assert np.abs(Xq).max() == 7 and xs == np.float32(np.abs(X.astype(np.float32)).max()) / np.float32(7.0)
    assert (np.abs(X.astype(np.float64) - float(xs) * Xq) <= float(xs) / 2 * (1 + 1e-6)).all()
    # ties at a scale of exactly 1 round to even; beyond +-7 clamps
    ties = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, 6.5, 7.0, -7.0]], np.float16)
    q, _ = oracle.quant_act4(ties, x_scale=np.float32(1.0))
    assert q.tolist() == [[0, 2, 2, 0, -2, 6, 7, -7]]
    q, _ = oracle.quant_act4(np.array([[9.0, -30.0, 7.4, 7.6, 0, 0, 0, 0]], np.float16), x_scale=np.float32(1.0))
    assert q.tolist() == [[7, -7, 7, 7, 0, 0, 0, 0]]


def test_round_trip_and_gemm_equals_brute_force():
    d = inputs.random_layer(13, 9, 24, 48)
    prep = oracle.prepare_weight4(d["W"])
    assert np.array_equal(oracle.decompress48(prep["vals"], prep["meta"]), prep["Wq"])
    Xq, _ = oracle.quant_act4(d["X"])
    acc = oracle.spgemm48_acc(Xq, prep["vals"], prep["meta"])
    # Fig. 1: the sparse GEMM returns the dense GEMM's result; pure-Python sums and a library product
    brute = [[sum(int(prep["Wq"][n, k]) * int(Xq[m, k]) for k in range(48)) for n in range(24)] for m in range(9)]
    assert acc.tolist() == brute
    assert np.array_equal(acc, Xq.astype(np.int64) @ prep["Wq"].astype(np.int64).T)
    assert np.array_equal(oracle.spgemm48_acc(Xq, prep["vals"], prep["meta"], threads=3), acc)


def test_column_regrouping_turns_the_pattern_into_2_4():
    # Taking, inside every chunk of eight, the first elements of the four sub-chunks and then the second
    # ones (e -> (e % 2) * 4 + e // 2) makes a pair-wise 4:8 matrix a 2:4 matrix, and a GEMM does not change
    # when weight and activation columns are permuted alike: the INT8 2:4 path computes the 4-bit
    # model's sums exactly.
    d = inputs.random_layer(14, 17, 40, 64)
    prep = oracle.prepare_weight4(d["W"])
    Xq, _ = oracle.quant_act4(d["X"])
    perm = np.array([8 * (k // 8) + 2 * (k % 4) + (k % 8) // 4 for k in range(64)])      # new column k holds old column perm[k]
    Wr, Xr = prep["Wq"][:, perm], Xq[:, perm]
    assert ((Wr.reshape(40, 16, 4) != 0).sum(-1) <= 2).all()
    vals, meta = oracle.compress24(Wr)
    assert np.array_equal(oracle.decompress24(vals, meta), Wr)
    assert np.array_equal(oracle.spgemm_acc(Xr, vals, meta), oracle.spgemm48_acc(Xq, prep["vals"], prep["meta"]))
