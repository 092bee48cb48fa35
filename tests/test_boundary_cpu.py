"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2305_10727_b200 import binding as B
from paper_2305_10727_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return B.load()


def test_every_declared_symbol_is_exported(lib):
    import glob
    declared = set()
    for path in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):      # the interface and the test hooks
        declared |= set(re.findall(r"\b(gpusq_[a-z0-9_]+)\s*\(", open(path).read()))
    declared -= {"gpusq_status"}
    # the test hooks are declared apart from the library's interface
    iface = open(os.path.join(ROOT, "include", "gpusq.h")).read()
    assert "gpusq_set_block_tokens" not in iface and "gpusq_set_tile_mix" not in iface
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_status_strings(lib):
    assert B.status_string(0) == "GPUSQ_OK"
    for code in range(1, 10):
        assert B.status_string(code).startswith("GPUSQ_ERR_")
    assert "unknown" in B.status_string(99)


def test_size_queries(lib):
    # values K/2 bytes + metadata K/8 bytes per row, both padded to 128 x 128 blocks
    assert B.packed_bytes(768, 768) == 768 * 768 * 5 // 8
    assert B.packed_bytes(768, 192) == 768 * 256 * 5 // 8
    assert B.packed_bytes(100, 64) == 256 * 128 * 5 // 8
    assert B.packed_bytes(0, 64) == 0
    assert B.quant_act_workspace(12608, 768) >= 16


def test_argument_errors_are_reported_before_any_cuda_call(lib):
    buf = (ctypes.c_uint8 * 4096)()
    a = ctypes.addressof(buf)
    a16 = (a + 255) // 256 * 256
    p = ctypes.c_void_p
    NULL, SHAPE, ALIGN, WS, ARG = 1, 2, 3, 4, 8
    assert lib.gpusq_prune24(None, p(a16), None, 4, 8, None) == NULL
    assert lib.gpusq_prune24(p(a16), p(a16), None, 4, 6, None) == SHAPE
    assert lib.gpusq_prune24(p(a16), p(a16), None, 0, 8, None) == SHAPE
    assert lib.gpusq_prune24(p(a16 + 4), p(a16), None, 4, 8, None) == ALIGN
    assert lib.gpusq_quant_weight(p(a16), None, p(a16), 4, 8, None) == NULL
    assert lib.gpusq_quant_weight(p(a16), p(a16), p(a16), 4, 7, None) == SHAPE
    assert lib.gpusq_compress24(p(a16), p(a16), None, 4, 8, None) == NULL
    assert lib.gpusq_compress24(p(a16), p(a16), p(a16), 4, 12, None) == SHAPE
    assert lib.gpusq_decompress24(p(a16), p(a16), p(a16), -1, 8, None) == SHAPE
    assert lib.gpusq_pack24(p(a16), p(a16), p(a16 + 16), 4, 8, None) == ALIGN
    assert lib.gpusq_quant_act(p(a16), p(a16), None, 0, 4, 8, None, 0, None) == NULL
    assert lib.gpusq_quant_act(p(a16), p(a16), p(a16), 0, 4, 8, None, 0, None) == WS
    assert lib.gpusq_quant_act(p(a16), p(a16), p(a16), 0, 4, 8, p(a16), 8, None) == WS
    assert lib.gpusq_quant_act(p(a16), p(a16), p(a16), 2, 4, 8, p(a16), 1 << 20, None) == ARG
    assert lib.gpusq_quant_act(p(a16), p(a16), p(a16), 1, 4, 12, None, 0, None) == SHAPE
    TOO_LARGE = 9
    assert lib.gpusq_quant_act_static(p(a16), p(a16), None, 0, 4, 8, None) == NULL
    assert lib.gpusq_quant_act_static(p(a16), p(a16), p(a16), 0, 4, 12, None) == SHAPE
    assert lib.gpusq_quant_act_static(p(a16), p(a16), p(a16), 5, 4, 8, None) == ARG
    assert lib.gpusq_quant_act_static(p(a16), p(a16), p(a16), 0, (1 << 29) + 1, 8, None) == TOO_LARGE
    assert lib.gpusq_quant_act_static(p(a16 + 8), p(a16), p(a16), 0, 4, 8, None) == ALIGN
    pq = lib.gpusq_patch_quant
    assert pq(p(a16), p(a16), None, 1, 1, 3, 32, 32, 16, 768, None, 0, None) == NULL
    assert pq(p(a16), p(a16), p(a16), 1, 1, 3, 32, 30, 16, 768, None, 0, None) == SHAPE      # W % P
    assert pq(p(a16), p(a16), p(a16), 1, 1, 3, 32, 32, 16, 752, None, 0, None) == SHAPE      # Kp < C P P
    assert pq(p(a16), p(a16), p(a16), 1, 1, 3, 28, 28, 14, 588, None, 0, None) == SHAPE      # Kp % 16
    assert pq(p(a16), p(a16), p(a16), 1, 1, 3, 21, 21, 7, 160, None, 0, None) == SHAPE       # odd P
    assert pq(p(a16), p(a16), p(a16), 3, 1, 3, 32, 32, 16, 768, None, 0, None) == ARG
    assert pq(p(a16), p(a16), p(a16), 0, 1, 3, 32, 32, 16, 768, None, 0, None) == WS
    assert pq(p(a16 + 8), p(a16), p(a16), 1, 1, 3, 32, 32, 16, 768, None, 0, None) == ALIGN
    assert pq(p(a16), p(a16), p(a16), 1, 1 << 20, 3, 224, 224, 2, 1 << 20, None, 0, None) == TOO_LARGE
    for fn in (lib.gpusq_spgemm_i8, lib.gpusq_gemm_i8_dense):
        ok = [p(a16), p(a16), p(a16), p(a16), None, 0, 0, None, p(a16), 8, 128, 64, None, None]
        bad = list(ok); bad[0] = None
        assert fn(*bad) == NULL
        bad = list(ok); bad[10] = 100
        assert fn(*bad) == SHAPE                  # FP16 rows of Y: N % 8
        bad = list(ok); bad[10] = 104; bad[6] = 1; bad[7] = p(a16)
        assert fn(*bad) == SHAPE                  # INT8 rows of Y: N % 16
        bad = list(ok); bad[11] = 40
        assert fn(*bad) == SHAPE                  # K % 16
        bad = list(ok); bad[9] = 0
        assert fn(*bad) == SHAPE
        bad = list(ok); bad[6] = 3
        assert fn(*bad) == ARG
        bad = list(ok); bad[5] = 7
        assert fn(*bad) == ARG
        bad = list(ok); bad[6] = 1
        assert fn(*bad) == NULL                   # INT8 output needs out_scale
        bad = list(ok); bad[2] = None
        assert fn(*bad) == NULL                   # FP16 output needs w_scale
        bad = list(ok); bad[8] = p(a16 + 8)
        assert fn(*bad) == ALIGN
    f16 = lib.gpusq_spgemm_f16
    ok = [p(a16), p(a16), None, 0, 0, p(a16), 8, 128, 64, None, None]
    bad = list(ok); bad[1] = None
    assert f16(*bad) == NULL
    bad = list(ok); bad[4] = 1
    assert f16(*bad) == ARG                       # no INT8 output in the FP16 model
    bad = list(ok); bad[8] = 60
    assert f16(*bad) == SHAPE                     # K % 8
    bad = list(ok); bad[7] = 100
    assert f16(*bad) == SHAPE                     # FP16 rows of Y: N % 8
    bad = list(ok); bad[0] = p(a16 + 8)
    assert f16(*bad) == ALIGN
    assert lib.gpusq_compress24_f16(p(a16), p(a16), None, 4, 8, None) == NULL
    assert lib.gpusq_compress24_f16(p(a16), p(a16), p(a16), 4, 12, None) == SHAPE
    assert lib.gpusq_pack24_f16(p(a16), p(a16), p(a16 + 16), 4, 8, None) == ALIGN
    assert B.packed_bytes_f16(768, 768) == 768 * 768 * 9 // 8
    assert B.packed_bytes_f16(100, 64) == 256 * 128 * 9 // 8
    assert lib.gpusq_set_block_tokens(17) == ARG
    assert lib.gpusq_set_block_tokens(256) == ARG
    assert lib.gpusq_set_block_tokens(0) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.load()
