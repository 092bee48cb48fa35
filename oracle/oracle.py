"""ctypes front for the plain C oracle -- TEST INFRASTRUCTURE, not product code.

Argument marshalling only: every arithmetic step is in ``gpusq_oracle.c``.
Arrays are numpy, C-contiguous; binary16 tensors travel as ``numpy.float16``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gpusq_oracle.c")
_HDR = os.path.join(_HERE, "gpusq_oracle.h")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "libgpusq_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction)."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (
        force
        or not os.path.exists(_OUT)
        or os.path.getmtime(_OUT) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    )
    if stale:
        tmp = _OUT + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
               "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _OUT)
    return _OUT


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
            lib.o_prune24.argtypes = [vp, vp, vp, i32, i32]
            lib.o_quant_weight.argtypes = [vp, vp, vp, i32, i32]
            lib.o_compress24.argtypes = [vp, vp, vp, i32, i32]
            lib.o_decompress24.argtypes = [vp, vp, vp, i32, i32]
            lib.o_quant_act.argtypes = [vp, vp, vp, i32, i64, i32]
            lib.o_spgemm_acc.argtypes = [vp, vp, vp, vp, i64, i32, i32]
            lib.o_spgemm_acc.restype = i64
            lib.o_spgemm_acc_rows.argtypes = [vp, vp, vp, vp, i64, vp, i32, i32]
            lib.o_spgemm_acc_rows.restype = i64
            lib.o_patch_rows.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32]
            lib.o_patch_rows.restype = None
            lib.o_patch_conv_acc.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32]
            lib.o_patch_conv_acc.restype = i64
            lib.o_to_f16.argtypes = [vp, vp, i64]
            lib.o_compress24_f16.argtypes = [vp, vp, vp, i32, i32]
            lib.o_decompress24_f16.argtypes = [vp, vp, vp, i32, i32]
            lib.o_spgemm_f16_rows.argtypes = [vp, vp, vp, vp, i64, vp, vp, i32, i32]
            lib.o_epilogue_f16.argtypes = [vp, vp, i32, vp, i64, i32]
            for name in ("o_to_f16", "o_compress24_f16", "o_decompress24_f16", "o_spgemm_f16_rows",
                         "o_epilogue_f16"):
                getattr(lib, name).restype = None
            lib.o_epilogue.argtypes = [vp, vp, f32, vp, i32, i32, f32, vp, i64, i32]
            lib.o_f32_to_f16.argtypes = [f32]
            lib.o_f32_to_f16.restype = ctypes.c_uint16
            lib.o_f16_to_f32.argtypes = [ctypes.c_uint16]
            lib.o_f16_to_f32.restype = f32
            lib.o_prune48.argtypes = [vp, vp, vp, i32, i32]
            lib.o_quant_weight4.argtypes = [vp, vp, vp, i32, i32]
            lib.o_compress48.argtypes = [vp, vp, vp, i32, i32]
            lib.o_decompress48.argtypes = [vp, vp, vp, i32, i32]
            lib.o_quant_act4.argtypes = [vp, vp, vp, i32, i64, i32]
            lib.o_spgemm48_acc.argtypes = [vp, vp, vp, vp, i64, i32, i32]
            lib.o_spgemm48_acc.restype = i64
            for name in ("o_prune48", "o_quant_weight4", "o_compress48", "o_decompress48", "o_quant_act4"):
                getattr(lib, name).restype = None
            lib.o_sqnr_db.argtypes = [vp, vp, i64]
            lib.o_sqnr_db.restype = ctypes.c_double
            for name in ("o_prune24", "o_quant_weight", "o_compress24", "o_decompress24",
                         "o_quant_act", "o_epilogue"):
                getattr(lib, name).restype = None
            _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def host_cores() -> int:
    """Cores this process may run on."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _row_blocks(n_rows: int, threads: int):
    """Contiguous row ranges, a few per thread so that uneven speeds even out."""
    parts = max(1, min(n_rows, 4 * threads))
    edges = [n_rows * i // parts for i in range(parts + 1)]
    return [(a, b) for a, b in zip(edges[:-1], edges[1:]) if b > a]


def _over_row_blocks(n_rows: int, threads, fn):
    """Run fn(lo, hi) over row blocks: output rows are independent of one another, so the plain
    single-threaded C routine is simply called once per block, from several Python threads when
    threads > 1 (ctypes releases the interpreter lock during the call).  The arithmetic is the C
    file's in either case; only which call computes which rows differs."""
    if not threads or threads <= 1 or n_rows < 2:
        fn(0, n_rows)
        return
    with ThreadPoolExecutor(max_workers=threads) as pool:
        for f in [pool.submit(fn, lo, hi) for lo, hi in _row_blocks(n_rows, threads)]:
            f.result()


def prune24(W, return_mask=False):
    W = _c(W, np.float32)
    N, K = W.shape
    assert K % 4 == 0
    Wp = np.empty_like(W)
    mask = np.empty((N, K // 4), np.uint8)
    _load().o_prune24(_p(W), _p(Wp), _p(mask), N, K)
    return (Wp, mask) if return_mask else Wp


def quant_weight(Wp):
    Wp = _c(Wp, np.float32)
    N, K = Wp.shape
    Wq = np.empty((N, K), np.int8)
    s = np.empty((N,), np.float32)
    _load().o_quant_weight(_p(Wp), _p(Wq), _p(s), N, K)
    return Wq, s


def compress24(Wq):
    Wq = _c(Wq, np.int8)
    N, K = Wq.shape
    assert K % 8 == 0
    vals = np.empty((N, K // 2), np.int8)
    meta = np.empty((N, K // 8), np.uint8)
    _load().o_compress24(_p(Wq), _p(vals), _p(meta), N, K)
    return vals, meta


def decompress24(vals, meta):
    vals = _c(vals, np.int8)
    meta = _c(meta, np.uint8)
    N, K = vals.shape[0], vals.shape[1] * 2
    assert meta.shape == (N, K // 8)
    Wq = np.empty((N, K), np.int8)
    _load().o_decompress24(_p(vals), _p(meta), _p(Wq), N, K)
    return Wq


def quant_act(X, x_scale=None):
    """X float16 [M, K]; x_scale None => computed (mode 0), else supplied (mode 1)."""
    X = _c(X, np.float16)
    M, K = X.shape
    Xq = np.empty((M, K), np.int8)
    s = np.zeros((1,), np.float32)
    mode = 0
    if x_scale is not None:
        s[0] = x_scale
        mode = 1
    _load().o_quant_act(_p(X.view(np.uint16)), _p(Xq), _p(s), mode, M, K)
    return Xq, np.float32(s[0])


def spgemm_acc(Xq, vals, meta, threads=None):
    """threads > 1: the token rows are split into blocks, one plain o_spgemm_acc call per block."""
    Xq, vals, meta = _c(Xq, np.int8), _c(vals, np.int8), _c(meta, np.uint8)
    M, K = Xq.shape
    N = vals.shape[0]
    assert vals.shape == (N, K // 2) and meta.shape == (N, K // 8)
    acc = np.empty((M, N), np.int32)
    lib = _load()
    overflow = []

    def block(lo, hi):
        overflow.append(lib.o_spgemm_acc(_p(Xq[lo:hi]), _p(vals), _p(meta), _p(acc[lo:hi]), hi - lo, N, K))

    _over_row_blocks(M, threads, block)
    assert sum(overflow) == 0, "INT32 overflow in %d sums" % sum(overflow)
    return acc


def spgemm_acc_rows(Xq, vals, meta, rows):
    Xq, vals, meta = _c(Xq, np.int8), _c(vals, np.int8), _c(meta, np.uint8)
    rows = _c(rows, np.int64)
    M, K = Xq.shape
    N = vals.shape[0]
    assert rows.min() >= 0 and rows.max() < M
    acc = np.empty((rows.size, N), np.int32)
    ovf = _load().o_spgemm_acc_rows(_p(Xq), _p(vals), _p(meta), _p(rows), rows.size,
                                    _p(acc), N, K)
    assert ovf == 0
    return acc


def patch_rows(imgq, P, Kp=None):
    """INT8 image codes [B, C, H, W] -> activation matrix [B*(H/P)*(W/P), Kp] of the patch-embedding GEMM."""
    imgq = _c(imgq, np.int8)
    B, C, H, W = imgq.shape
    assert H % P == 0 and W % P == 0
    K = C * P * P
    Kp = K if Kp is None else Kp
    assert Kp >= K
    X = np.empty((B * (H // P) * (W // P), Kp), np.int8)
    _load().o_patch_rows(_p(imgq), _p(X), B, C, H, W, P, Kp)
    return X


def patch_conv_acc(imgq, Wq4):
    """The strided convolution on INT8 codes, as its definition; returns (acc [tokens, D], multiply-adds)."""
    imgq, Wq4 = _c(imgq, np.int8), _c(Wq4, np.int8)
    B, C, H, W = imgq.shape
    D, C2, P, P2 = Wq4.shape
    assert C2 == C and P2 == P and H % P == 0 and W % P == 0
    acc = np.empty((B * (H // P) * (W // P), D), np.int32)
    macs = _load().o_patch_conv_acc(_p(imgq), _p(Wq4), _p(acc), B, C, H, W, P, D)
    return acc, int(macs)


_OUT_DTYPES = {0: np.float16, 1: np.int8, 2: np.int32}


def epilogue(acc, w_scale, x_scale, bias=None, act=0, out_type=0, out_scale=1.0, threads=None):
    """threads > 1: one plain o_epilogue call per block of whole rows."""
    acc = _c(acc, np.int32)
    w_scale = _c(w_scale, np.float32)
    if bias is not None:
        bias = _c(bias, np.float32)
    N = acc.shape[-1]
    Y = np.empty(acc.shape, _OUT_DTYPES[out_type])
    lib = _load()
    acc2, Y2 = acc.reshape(-1, N), Y.reshape(-1, N)

    def block(lo, hi):
        lib.o_epilogue(_p(acc2[lo:hi]), _p(w_scale), float(x_scale), _p(bias), act, out_type,
                       float(out_scale), _p(Y2[lo:hi]), (hi - lo) * N, N)

    _over_row_blocks(acc2.shape[0], threads, block)
    return Y


def f32_to_f16_bits(x: float) -> int:
    return int(_load().o_f32_to_f16(float(np.float32(x))))


def f16_bits_to_f32(h: int) -> float:
    return float(_load().o_f16_to_f32(int(h)))


def sqnr_db(ref, test) -> float:
    ref, test = _c(ref, np.float32), _c(test, np.float32)
    return float(_load().o_sqnr_db(_p(ref), _p(test), ref.size))


# ---- the two call stacks of the path, as compositions of the steps above ----

def prepare_weight(W):
    """Offline weight preparation: prune -> quantise -> compress."""
    Wp, mask = prune24(W, return_mask=True)
    Wq, w_scale = quant_weight(Wp)
    vals, meta = compress24(Wq)
    return {"Wp": Wp, "mask": mask, "Wq": Wq, "w_scale": w_scale, "vals": vals, "meta": meta}


def layer_forward(X, prep, bias=None, act=0, out_type=0, out_scale=1.0, x_scale=None,
                  rows=None, threads=None):
    """Per-inference call: quantise activations -> sparse GEMM -> epilogue.

    rows: optional token-row subset (the activation scale still comes from all of X).
    threads: GEMM and epilogue over row blocks on that many host threads (see _over_row_blocks);
    the activation quantisation, whose scale needs the whole tensor, stays one call.
    """
    Xq, xs = quant_act(X, x_scale)
    if rows is None:
        acc = spgemm_acc(Xq, prep["vals"], prep["meta"], threads=threads)
    else:
        acc = spgemm_acc_rows(Xq, prep["vals"], prep["meta"], rows)
    Y = epilogue(acc, prep["w_scale"], xs, bias, act, out_type, out_scale, threads=threads)
    return {"Xq": Xq, "x_scale": xs, "acc": acc, "Y": Y}


# ---- FP16 2:4 sparse model (M_SF) ----

def to_f16(W):
    W = _c(W, np.float32)
    Wh = np.empty(W.shape, np.uint16)
    _load().o_to_f16(_p(W), _p(Wh), W.size)
    return Wh.view(np.float16)


def compress24_f16(Wh):
    Wh = _c(Wh, np.float16)
    N, K = Wh.shape
    assert K % 8 == 0
    vals = np.empty((N, K // 2), np.float16)
    meta = np.empty((N, K // 8), np.uint8)
    _load().o_compress24_f16(_p(Wh.view(np.uint16)), _p(vals.view(np.uint16)), _p(meta), N, K)
    return vals, meta


def decompress24_f16(vals, meta):
    vals, meta = _c(vals, np.float16), _c(meta, np.uint8)
    N, K = vals.shape[0], vals.shape[1] * 2
    Wh = np.empty((N, K), np.float16)
    _load().o_decompress24_f16(_p(vals.view(np.uint16)), _p(meta), _p(Wh.view(np.uint16)), N, K)
    return Wh


def spgemm_f16_rows(X, vals, meta, rows=None):
    """Exact sums (binary64) of the FP16 sparse layer for the given token rows, and sum |products|."""
    X, vals, meta = _c(X, np.float16), _c(vals, np.float16), _c(meta, np.uint8)
    M, K = X.shape
    N = vals.shape[0]
    assert vals.shape == (N, K // 2) and meta.shape == (N, K // 8)
    rows = np.arange(M, dtype=np.int64) if rows is None else _c(rows, np.int64)
    acc = np.empty((rows.size, N), np.float64)
    mag = np.empty((rows.size, N), np.float64)
    _load().o_spgemm_f16_rows(_p(X.view(np.uint16)), _p(vals.view(np.uint16)), _p(meta), _p(rows), rows.size,
                              _p(acc), _p(mag), N, K)
    return acc, mag


def epilogue_f16(acc, bias=None, act=0):
    acc = _c(acc, np.float64)
    if bias is not None:
        bias = _c(bias, np.float32)
    Y = np.empty(acc.shape, np.float16)
    _load().o_epilogue_f16(_p(acc), _p(bias), act, _p(Y.view(np.uint16)), acc.size, acc.shape[-1])
    return Y


def prepare_weight_f16(W):
    """Offline steps of the FP16 sparse model: prune -> round to binary16 -> compress."""
    Wp, mask = prune24(W, return_mask=True)
    Wh = to_f16(Wp)
    vals, meta = compress24_f16(Wh)
    return {"Wp": Wp, "mask": mask, "Wh": Wh, "vals": vals, "meta": meta}


def patch_embed_weight(W4, Kp=None):
    """Conv weight [D, C, P, P] -> flattened [D, Kp] (zero columns beyond C*P*P), then the offline steps."""
    W4 = _c(W4, np.float32)
    D = W4.shape[0]
    K = W4[0].size
    Kp = K if Kp is None else Kp
    Wf = np.zeros((D, Kp), np.float32)
    Wf[:, :K] = W4.reshape(D, K)
    return prepare_weight(Wf)


def patch_embed_forward(img, prep, P, bias=None, out_type=0, out_scale=1.0, x_scale=None, rows=None):
    """Patch embedding (Sec. 3.3): quantise the image, cut it into patch rows, sparse GEMM, epilogue."""
    img = _c(img, np.float16)
    Kp = prep["Wq"].shape[1]
    imgq, xs = quant_act(img.reshape(1, -1), x_scale)
    imgq = imgq.reshape(img.shape)
    Xq = patch_rows(imgq, P, Kp)
    if rows is None:
        acc = spgemm_acc(Xq, prep["vals"], prep["meta"])
    else:
        acc = spgemm_acc_rows(Xq, prep["vals"], prep["meta"], rows)
    Y = epilogue(acc, prep["w_scale"], xs, bias, 0, out_type, out_scale)
    return {"imgq": imgq, "Xq": Xq, "x_scale": xs, "acc": acc, "Y": Y}


# ---- INT4 model: pair-wise 4:8 sparsity (Sec. 3.1) ----

def prune48(W, return_mask=False):
    W = _c(W, np.float32)
    N, K = W.shape
    assert K % 8 == 0
    Wp = np.empty_like(W)
    mask = np.empty((N, K // 8), np.uint8)
    _load().o_prune48(_p(W), _p(Wp), _p(mask), N, K)
    return (Wp, mask) if return_mask else Wp


def quant_weight4(Wp):
    Wp = _c(Wp, np.float32)
    N, K = Wp.shape
    Wq = np.empty((N, K), np.int8)
    s = np.empty((N,), np.float32)
    _load().o_quant_weight4(_p(Wp), _p(Wq), _p(s), N, K)
    return Wq, s


def compress48(Wq):
    Wq = _c(Wq, np.int8)
    N, K = Wq.shape
    assert K % 16 == 0
    vals = np.empty((N, K // 4), np.uint8)
    meta = np.empty((N, K // 16), np.uint8)
    _load().o_compress48(_p(Wq), _p(vals), _p(meta), N, K)
    return vals, meta


def decompress48(vals, meta):
    vals, meta = _c(vals, np.uint8), _c(meta, np.uint8)
    N, K = vals.shape[0], vals.shape[1] * 4
    assert meta.shape == (N, K // 16)
    Wq = np.empty((N, K), np.int8)
    _load().o_decompress48(_p(vals), _p(meta), _p(Wq), N, K)
    return Wq


def quant_act4(X, x_scale=None):
    X = _c(X, np.float16)
    M, K = X.shape
    Xq = np.empty((M, K), np.int8)
    s = np.zeros((1,), np.float32)
    mode = 0
    if x_scale is not None:
        s[0] = x_scale
        mode = 1
    _load().o_quant_act4(_p(X.view(np.uint16)), _p(Xq), _p(s), mode, M, K)
    return Xq, np.float32(s[0])


def spgemm48_acc(Xq, vals, meta, threads=None):
    Xq, vals, meta = _c(Xq, np.int8), _c(vals, np.uint8), _c(meta, np.uint8)
    M, K = Xq.shape
    N = vals.shape[0]
    assert vals.shape == (N, K // 4) and meta.shape == (N, K // 16)
    acc = np.empty((M, N), np.int32)
    lib = _load()
    overflow = []

    def block(lo, hi):
        overflow.append(lib.o_spgemm48_acc(_p(Xq[lo:hi]), _p(vals), _p(meta), _p(acc[lo:hi]), hi - lo, N, K))

    _over_row_blocks(M, threads, block)
    assert sum(overflow) == 0
    return acc


def prepare_weight4(W):
    """Offline steps of the INT4 model: pair-wise 4:8 prune -> 4-bit quantise -> compress."""
    Wp, mask = prune48(W, return_mask=True)
    Wq, w_scale = quant_weight4(Wp)
    vals, meta = compress48(Wq)
    return {"Wp": Wp, "mask": mask, "Wq": Wq, "w_scale": w_scale, "vals": vals, "meta": meta}


def layer_forward4(X, prep, bias=None, act=0, threads=None):
    """Per-inference call of the INT4 model: 4-bit activation codes -> sparse GEMM -> the usual epilogue (FP16 out)."""
    Xq, xs = quant_act4(X)
    acc = spgemm48_acc(Xq, prep["vals"], prep["meta"], threads=threads)
    Y = epilogue(acc, prep["w_scale"], xs, bias, act, 0, 1.0, threads=threads)
    return {"Xq": Xq, "x_scale": xs, "acc": acc, "Y": Y}
