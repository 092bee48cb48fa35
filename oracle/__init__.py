"""gpusq oracle -- TEST INFRASTRUCTURE, not product code.

A thin numpy/ctypes front for the plain C oracle in ``gpusq_oracle.c``.  Only
the tests, the smoke check and the CPU-baseline leg of the benchmark import
this package; the CUDA library never does, and nothing here touches the GPU
or imports the product package.
"""
from .oracle import (  # noqa: F401
    build,
    host_cores,
    prune24,
    quant_weight,
    compress24,
    decompress24,
    quant_act,
    spgemm_acc,
    spgemm_acc_rows,
    epilogue,
    f32_to_f16_bits,
    f16_bits_to_f32,
    sqnr_db,
    layer_forward,
    prepare_weight,
    patch_rows,
    patch_conv_acc,
    patch_embed_weight,
    patch_embed_forward,
    to_f16,
    compress24_f16,
    decompress24_f16,
    spgemm_f16_rows,
    epilogue_f16,
    prepare_weight_f16,
    prune48,
    quant_weight4,
    compress48,
    decompress48,
    quant_act4,
    spgemm48_acc,
    prepare_weight4,
    layer_forward4,
)
