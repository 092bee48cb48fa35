"""Thin Python binding of libgpusq.so: argument marshalling only.

Every function has the name of the C entry point it calls (without the
``gpusq_`` prefix), takes CUDA ``torch`` tensors, allocates the outputs with
torch when the caller does not pass them, enqueues on torch's current stream
and returns without synchronising.  All arithmetic runs in the CUDA kernels.
A missing library or a non-zero status raises; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgpusq.so")

ACT_NONE, ACT_GELU = 0, 1
OUT_F16, OUT_I8, OUT_I32 = 0, 1, 2
SCALE_COMPUTE, SCALE_GIVEN = 0, 1

EXPORTS = (
    "gpusq_status_string", "gpusq_prune24", "gpusq_quant_weight", "gpusq_compress24",
    "gpusq_decompress24", "gpusq_packed_bytes", "gpusq_pack24", "gpusq_quant_act_workspace",
    "gpusq_quant_act", "gpusq_quant_act_static", "gpusq_patch_quant", "gpusq_spgemm_i8", "gpusq_gemm_i8_dense", "gpusq_set_block_tokens", "gpusq_set_tile_mix", "gpusq_set_quant_act_wait", "gpusq_set_gemm_wait", "gpusq_set_max_clusters",
    "gpusq_spgemm_i8_absmax", "gpusq_quant_act_absmax",
    "gpusq_prune48", "gpusq_quant_weight4", "gpusq_compress48", "gpusq_expand48", "gpusq_quant_act4",
    "gpusq_compress24_f16", "gpusq_packed_bytes_f16", "gpusq_pack24_f16", "gpusq_spgemm_f16",
)

_lib = None


class GpusqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, status_string(status)))


def load() -> ctypes.CDLL:
    """Load libgpusq.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libgpusq.so not found at %s: build it with `python -m paper_2305_10727_b200.build` "
            "(there is no CPU fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.gpusq_status_string.argtypes = [i32]
    lib.gpusq_status_string.restype = ctypes.c_char_p
    lib.gpusq_prune24.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_quant_weight.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_compress24.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_decompress24.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_packed_bytes.argtypes = [i32, i32]
    lib.gpusq_packed_bytes.restype = sz
    lib.gpusq_pack24.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_quant_act_workspace.argtypes = [i64, i32]
    lib.gpusq_quant_act_workspace.restype = sz
    lib.gpusq_quant_act.argtypes = [vp, vp, vp, i32, i64, i32, vp, sz, vp]
    lib.gpusq_quant_act_static.argtypes = [vp, vp, vp, i32, i64, i32, vp]
    lib.gpusq_patch_quant.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, sz, vp]
    gemm_args = [vp, vp, vp, vp, vp, i32, i32, vp, vp, i64, i32, i32, vp, vp]
    lib.gpusq_spgemm_i8.argtypes = gemm_args
    lib.gpusq_gemm_i8_dense.argtypes = gemm_args
    lib.gpusq_spgemm_i8_absmax.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, i64, i32, i32, vp, vp]
    lib.gpusq_quant_act_absmax.argtypes = [vp, vp, vp, vp, i64, i32, vp]
    lib.gpusq_prune48.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_quant_weight4.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_compress48.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_expand48.argtypes = [vp, vp, vp, vp, i32, i32, vp]
    lib.gpusq_quant_act4.argtypes = [vp, vp, vp, i32, i64, i32, vp, sz, vp]
    lib.gpusq_set_block_tokens.argtypes = [i32]
    lib.gpusq_set_tile_mix.argtypes = [i32, i32]
    lib.gpusq_set_quant_act_wait.argtypes = [ctypes.c_ulonglong, i32]
    lib.gpusq_set_gemm_wait.argtypes = [ctypes.c_uint, i32]
    lib.gpusq_set_max_clusters.argtypes = [i32]
    lib.gpusq_compress24_f16.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_packed_bytes_f16.argtypes = [i32, i32]
    lib.gpusq_packed_bytes_f16.restype = sz
    lib.gpusq_pack24_f16.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.gpusq_spgemm_f16.argtypes = [vp, vp, vp, i32, i32, vp, i64, i32, i32, vp, vp]
    for name in EXPORTS:
        if name not in ("gpusq_status_string", "gpusq_packed_bytes", "gpusq_packed_bytes_f16",
                        "gpusq_quant_act_workspace"):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().gpusq_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise GpusqError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return t


def prune24(W: torch.Tensor, Wp: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None,
            want_mask: bool = False):
    _dev(W, torch.float32, "W")
    N, K = W.shape
    if Wp is None:
        Wp = torch.empty_like(W)
    if mask is None and want_mask:
        mask = torch.empty((N, K // 4), dtype=torch.uint8, device=W.device)
    _check(load().gpusq_prune24(_ptr(W), _ptr(Wp), _ptr(mask), N, K, _stream()), "gpusq_prune24")
    return (Wp, mask) if want_mask else Wp


def quant_weight(Wp: torch.Tensor, Wq: Optional[torch.Tensor] = None, w_scale: Optional[torch.Tensor] = None):
    _dev(Wp, torch.float32, "Wp")
    N, K = Wp.shape
    if Wq is None:
        Wq = torch.empty((N, K), dtype=torch.int8, device=Wp.device)
    if w_scale is None:
        w_scale = torch.empty((N,), dtype=torch.float32, device=Wp.device)
    _check(load().gpusq_quant_weight(_ptr(Wp), _ptr(Wq), _ptr(w_scale), N, K, _stream()), "gpusq_quant_weight")
    return Wq, w_scale


def compress24(Wq: torch.Tensor, vals: Optional[torch.Tensor] = None, meta: Optional[torch.Tensor] = None):
    _dev(Wq, torch.int8, "Wq")
    N, K = Wq.shape
    if vals is None:
        vals = torch.empty((N, K // 2), dtype=torch.int8, device=Wq.device)
    if meta is None:
        meta = torch.empty((N, K // 8), dtype=torch.uint8, device=Wq.device)
    _check(load().gpusq_compress24(_ptr(Wq), _ptr(vals), _ptr(meta), N, K, _stream()), "gpusq_compress24")
    return vals, meta


def decompress24(vals: torch.Tensor, meta: torch.Tensor, Wq: Optional[torch.Tensor] = None):
    _dev(vals, torch.int8, "vals")
    _dev(meta, torch.uint8, "meta")
    N, K = vals.shape[0], vals.shape[1] * 2
    if Wq is None:
        Wq = torch.empty((N, K), dtype=torch.int8, device=vals.device)
    _check(load().gpusq_decompress24(_ptr(vals), _ptr(meta), _ptr(Wq), N, K, _stream()), "gpusq_decompress24")
    return Wq


def packed_bytes(N: int, K: int) -> int:
    return int(load().gpusq_packed_bytes(N, K))


def pack24(vals: torch.Tensor, meta: torch.Tensor, Wpacked: Optional[torch.Tensor] = None):
    _dev(vals, torch.int8, "vals")
    _dev(meta, torch.uint8, "meta")
    N, K = vals.shape[0], vals.shape[1] * 2
    if Wpacked is None:
        Wpacked = torch.empty((packed_bytes(N, K),), dtype=torch.uint8, device=vals.device)
    _check(load().gpusq_pack24(_ptr(vals), _ptr(meta), _ptr(Wpacked), N, K, _stream()), "gpusq_pack24")
    return Wpacked


def quant_act_workspace(M: int, K: int) -> int:
    return int(load().gpusq_quant_act_workspace(M, K))


def quant_act(X: torch.Tensor, Xq: Optional[torch.Tensor] = None, x_scale: Optional[torch.Tensor] = None,
              scale_mode: int = SCALE_COMPUTE, workspace: Optional[torch.Tensor] = None):
    _dev(X, torch.float16, "X")
    M, K = X.shape
    if Xq is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    if x_scale is None:
        if scale_mode == SCALE_GIVEN:
            raise ValueError("scale_mode GIVEN needs x_scale")
        x_scale = torch.empty((1,), dtype=torch.float32, device=X.device)
    if workspace is None and scale_mode == SCALE_COMPUTE:
        workspace = torch.zeros((quant_act_workspace(M, K),), dtype=torch.uint8, device=X.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().gpusq_quant_act(_ptr(X), _ptr(Xq), _ptr(x_scale), scale_mode, M, K, _ptr(workspace),
                                  ws_bytes, _stream()), "gpusq_quant_act")
    return Xq, x_scale


QUANT_ACT_STATUS_OFFSET = 8196       # GPUSQ_QUANT_ACT_STATUS_OFFSET of gpusq.h


def quant_act_status(workspace: torch.Tensor) -> int:
    """The status word gpusq_quant_act keeps in its workspace (0, or 7 = a bounded wait expired).  Synchronises."""
    word = workspace.view(torch.uint8)[QUANT_ACT_STATUS_OFFSET:QUANT_ACT_STATUS_OFFSET + 4].view(torch.int32)
    return int(word.cpu().item())


def set_quant_act_wait(limit_ns: int, withhold_last_cta: bool = False) -> None:
    """Test hook (gpusq_testing.h): bound of the one-launch kernel's waits; optionally plant an arrival that never comes."""
    _check(load().gpusq_set_quant_act_wait(int(limit_ns), 1 if withhold_last_cta else 0), "gpusq_set_quant_act_wait")


def set_gemm_wait(limit_us: int, withhold_loads: bool = False) -> None:
    """Test hook (gpusq_testing.h): bound of the GEMM kernels' waits; optionally plant loads that never come."""
    _check(load().gpusq_set_gemm_wait(int(limit_us), 1 if withhold_loads else 0), "gpusq_set_gemm_wait")


def quant_act_static(X: torch.Tensor, Xq: Optional[torch.Tensor] = None, x_scale: Optional[torch.Tensor] = None,
                     scale_mode: int = SCALE_COMPUTE):
    """gpusq_quant_act_static: no workspace argument; the library's own fixed scratch is used."""
    _dev(X, torch.float16, "X")
    M, K = X.shape
    if Xq is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    if x_scale is None:
        if scale_mode == SCALE_GIVEN:
            raise ValueError("scale_mode GIVEN needs x_scale")
        x_scale = torch.empty((1,), dtype=torch.float32, device=X.device)
    _check(load().gpusq_quant_act_static(_ptr(X), _ptr(Xq), _ptr(x_scale), scale_mode, M, K, _stream()),
           "gpusq_quant_act_static")
    return Xq, x_scale


def patch_quant(img: torch.Tensor, P: int, Kp: Optional[int] = None, Xq: Optional[torch.Tensor] = None,
                x_scale: Optional[torch.Tensor] = None, scale_mode: int = SCALE_COMPUTE,
                workspace: Optional[torch.Tensor] = None):
    """gpusq_patch_quant: img f16 [B, C, H, W] -> (Xq i8 [B*(H/P)*(W/P), Kp], x_scale)."""
    _dev(img, torch.float16, "img")
    B, C, H, W = img.shape
    if Kp is None:
        Kp = (C * P * P + 15) // 16 * 16
    tokens = B * (H // P) * (W // P)
    if Xq is None:
        Xq = torch.empty((tokens, Kp), dtype=torch.int8, device=img.device)
    if x_scale is None:
        if scale_mode == SCALE_GIVEN:
            raise ValueError("scale_mode GIVEN needs x_scale")
        x_scale = torch.empty((1,), dtype=torch.float32, device=img.device)
    if workspace is None and scale_mode == SCALE_COMPUTE:
        workspace = torch.zeros((quant_act_workspace(tokens, Kp),), dtype=torch.uint8, device=img.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().gpusq_patch_quant(_ptr(img), _ptr(Xq), _ptr(x_scale), scale_mode, B, C, H, W, P, Kp,
                                    _ptr(workspace), ws_bytes, _stream()), "gpusq_patch_quant")
    return Xq, x_scale


def flatten_conv_weight(W4: torch.Tensor, Kp: Optional[int] = None) -> torch.Tensor:
    """Conv weight [D, C, P, P] -> [D, Kp] f32 row-major, zero columns beyond C*P*P (a copy, no arithmetic)."""
    D = W4.shape[0]
    K = W4[0].numel()
    if Kp is None:
        Kp = (K + 15) // 16 * 16
    Wf = torch.zeros((D, Kp), dtype=torch.float32, device=W4.device)
    Wf[:, :K] = W4.reshape(D, K)
    return Wf


_OUT_DTYPE = {OUT_F16: torch.float16, OUT_I8: torch.int8, OUT_I32: torch.int32}


def _gemm(fn_name, Xq, Wop, w_scale, x_scale, bias, act, out_type, out_scale, Y, N, status_buf):
    _dev(Xq, torch.int8, "Xq")
    M, K = Xq.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=_OUT_DTYPE[out_type], device=Xq.device)
    fn = getattr(load(), fn_name)
    _check(fn(_ptr(Xq), _ptr(Wop), _ptr(w_scale), _ptr(x_scale), _ptr(bias), act, out_type, _ptr(out_scale),
              _ptr(Y), M, N, K, _ptr(status_buf), _stream()), fn_name)
    return Y


def spgemm_i8(Xq: torch.Tensor, Wpacked: torch.Tensor, N: int, w_scale=None, x_scale=None, bias=None,
              act: int = ACT_NONE, out_type: int = OUT_F16, out_scale=None, Y=None, status_buf=None):
    return _gemm("gpusq_spgemm_i8", Xq, Wpacked, w_scale, x_scale, bias, act, out_type, out_scale, Y, N,
                 status_buf)


def spgemm_i8_absmax(Xq: torch.Tensor, Wpacked: torch.Tensor, N: int, w_scale, x_scale, bias=None,
                     act: int = ACT_NONE, Y=None, y_absmax=None, status_buf=None):
    """gpusq_spgemm_i8_absmax: FP16 output plus max |Y| merged into y_absmax (float32[1], zeroed here if not given)."""
    _dev(Xq, torch.int8, "Xq")
    M, K = Xq.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    if y_absmax is None:
        y_absmax = torch.zeros((1,), dtype=torch.float32, device=Xq.device)
    _check(load().gpusq_spgemm_i8_absmax(_ptr(Xq), _ptr(Wpacked), _ptr(w_scale), _ptr(x_scale), _ptr(bias), act,
                                         _ptr(Y), _ptr(y_absmax), M, N, K, _ptr(status_buf), _stream()),
           "gpusq_spgemm_i8_absmax")
    return Y, y_absmax


def quant_act_absmax(X: torch.Tensor, absmax: torch.Tensor, Xq: Optional[torch.Tensor] = None,
                     x_scale: Optional[torch.Tensor] = None):
    """gpusq_quant_act_absmax: one-pass quantisation with the scale derived from a known max |X|."""
    _dev(X, torch.float16, "X")
    M, K = X.shape
    if Xq is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    if x_scale is None:
        x_scale = torch.empty((1,), dtype=torch.float32, device=X.device)
    _check(load().gpusq_quant_act_absmax(_ptr(X), _ptr(Xq), _ptr(x_scale), _ptr(absmax), M, K, _stream()),
           "gpusq_quant_act_absmax")
    return Xq, x_scale


def gemm_i8_dense(Xq: torch.Tensor, Wq: torch.Tensor, w_scale=None, x_scale=None, bias=None,
                  act: int = ACT_NONE, out_type: int = OUT_F16, out_scale=None, Y=None, status_buf=None):
    _dev(Wq, torch.int8, "Wq")
    return _gemm("gpusq_gemm_i8_dense", Xq, Wq, w_scale, x_scale, bias, act, out_type, out_scale, Y,
                 Wq.shape[0], status_buf)


def set_block_tokens(block_t: int) -> None:
    """Test hook (gpusq_testing.h): force the GEMM tile height; 0 = automatic."""
    _check(load().gpusq_set_block_tokens(block_t), "gpusq_set_block_tokens")


def set_max_clusters(clusters: int) -> None:
    """Measurement hook (gpusq_testing.h): the GEMM launches use at most that many CTA pairs (0 = all)."""
    _check(load().gpusq_set_max_clusters(int(clusters)), "gpusq_set_max_clusters")


def set_tile_mix(block_t: int, n_big: int) -> None:
    """Test hook (gpusq_testing.h): n_big token tiles of block_t tokens, the rest 32 tokens lower."""
    _check(load().gpusq_set_tile_mix(block_t, n_big), "gpusq_set_tile_mix")


# ---- FP16 2:4 sparse model ----
OUT_F32 = 2


def compress24_f16(Wp: torch.Tensor):
    _dev(Wp, torch.float32, "Wp")
    N, K = Wp.shape
    vals = torch.empty((N, K // 2), dtype=torch.float16, device=Wp.device)
    meta = torch.empty((N, K // 8), dtype=torch.uint8, device=Wp.device)
    _check(load().gpusq_compress24_f16(_ptr(Wp), _ptr(vals), _ptr(meta), N, K, _stream()), "gpusq_compress24_f16")
    return vals, meta


def packed_bytes_f16(N: int, K: int) -> int:
    return int(load().gpusq_packed_bytes_f16(N, K))


def pack24_f16(vals: torch.Tensor, meta: torch.Tensor, Wpacked: Optional[torch.Tensor] = None):
    _dev(vals, torch.float16, "vals")
    _dev(meta, torch.uint8, "meta")
    N, K = vals.shape[0], vals.shape[1] * 2
    if Wpacked is None:
        Wpacked = torch.empty((packed_bytes_f16(N, K),), dtype=torch.uint8, device=vals.device)
    _check(load().gpusq_pack24_f16(_ptr(vals), _ptr(meta), _ptr(Wpacked), N, K, _stream()), "gpusq_pack24_f16")
    return Wpacked


def spgemm_f16(X: torch.Tensor, Wpacked: torch.Tensor, N: int, bias=None, act: int = ACT_NONE,
               out_type: int = OUT_F16, Y=None, status_buf=None):
    _dev(X, torch.float16, "X")
    M, K = X.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16 if out_type == OUT_F16 else torch.float32, device=X.device)
    _check(load().gpusq_spgemm_f16(_ptr(X), _ptr(Wpacked), _ptr(bias), act, out_type, _ptr(Y), M, N, K,
                                   _ptr(status_buf), _stream()), "gpusq_spgemm_f16")
    return Y


# ---- INT4 model (pair-wise 4:8 sparsity) ----

def prune48(W: torch.Tensor, want_mask: bool = False):
    _dev(W, torch.float32, "W")
    N, K = W.shape
    Wp = torch.empty_like(W)
    mask = torch.empty((N, K // 8), dtype=torch.uint8, device=W.device) if want_mask else None
    _check(load().gpusq_prune48(_ptr(W), _ptr(Wp), _ptr(mask), N, K, _stream()), "gpusq_prune48")
    return (Wp, mask) if want_mask else Wp


def quant_weight4(Wp: torch.Tensor):
    _dev(Wp, torch.float32, "Wp")
    N, K = Wp.shape
    Wq = torch.empty((N, K), dtype=torch.int8, device=Wp.device)
    w_scale = torch.empty((N,), dtype=torch.float32, device=Wp.device)
    _check(load().gpusq_quant_weight4(_ptr(Wp), _ptr(Wq), _ptr(w_scale), N, K, _stream()), "gpusq_quant_weight4")
    return Wq, w_scale


def compress48(Wq: torch.Tensor):
    _dev(Wq, torch.int8, "Wq")
    N, K = Wq.shape
    vals4 = torch.empty((N, K // 4), dtype=torch.uint8, device=Wq.device)
    meta4 = torch.empty((N, K // 16), dtype=torch.uint8, device=Wq.device)
    _check(load().gpusq_compress48(_ptr(Wq), _ptr(vals4), _ptr(meta4), N, K, _stream()), "gpusq_compress48")
    return vals4, meta4


def expand48(vals4: torch.Tensor, meta4: torch.Tensor):
    """(vals4, meta4) of the 4-bit format -> (vals, meta) of the 2:4 INT8 format, columns regrouped."""
    _dev(vals4, torch.uint8, "vals4")
    _dev(meta4, torch.uint8, "meta4")
    N, K = vals4.shape[0], vals4.shape[1] * 4
    vals = torch.empty((N, K // 2), dtype=torch.int8, device=vals4.device)
    meta = torch.empty((N, K // 8), dtype=torch.uint8, device=vals4.device)
    _check(load().gpusq_expand48(_ptr(vals4), _ptr(meta4), _ptr(vals), _ptr(meta), N, K, _stream()), "gpusq_expand48")
    return vals, meta


def quant_act4(X: torch.Tensor, Xq: Optional[torch.Tensor] = None, x_scale: Optional[torch.Tensor] = None,
               scale_mode: int = SCALE_COMPUTE, workspace: Optional[torch.Tensor] = None):
    """gpusq_quant_act4: 4-bit activation codes (INT8 containers) in the regrouped column order."""
    _dev(X, torch.float16, "X")
    M, K = X.shape
    if Xq is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
    if x_scale is None:
        if scale_mode == SCALE_GIVEN:
            raise ValueError("scale_mode GIVEN needs x_scale")
        x_scale = torch.empty((1,), dtype=torch.float32, device=X.device)
    if workspace is None and scale_mode == SCALE_COMPUTE:
        workspace = torch.zeros((quant_act_workspace(M, K),), dtype=torch.uint8, device=X.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load().gpusq_quant_act4(_ptr(X), _ptr(Xq), _ptr(x_scale), scale_mode, M, K, _ptr(workspace), ws_bytes,
                                   _stream()), "gpusq_quant_act4")
    return Xq, x_scale
