"""Seeded synthetic inputs for the ViT-shaped linear layers.

This module holds no arithmetic of the method (no pruning, quantisation,
compression or GEMM): it only draws the random tensors that both the CUDA
library and the CPU oracle are given, and names the layer shapes.

Shapes follow the models the paper compresses (DeiT / Swin; Sec. 4) and the
larger ViT-L/H used for scaling: 197 = 14*14+1 tokens per 224x224 image with
16x16 patches, 196 tokens per image in 7x7 windows for Swin stage 3 and
3136 = 56*56 in stage 1 (4x4 patches), 257 = 16*16+1 for ViT-H/14.  Distributions: trained ViT weights are close to a zero-mean
normal with sigma ~0.02 (the usual truncated-normal initialisation keeps that
scale), biases are small, LayerNorm outputs are roughly unit normal; the
heavy-tailed case (Student-t, 4 degrees of freedom, scaled to unit variance)
stands for activations with outliers, where a per-tensor absmax scale wastes
range.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np


@dataclass(frozen=True)
class Layer:
    name: str
    K: int          # input features (the 2:4 axis)
    N: int          # output features
    gelu: bool = False


@dataclass(frozen=True)
class Config:
    cid: int
    name: str
    M: int                      # tokens = batch * tokens per image
    layers: tuple
    x_dist: str = "normal"      # "normal" | "student_t4"
    int8_out: bool = False      # also exercise the requantised-INT8 output


def _block(h: int, mlp: int) -> tuple:
    return (
        Layer("qkv", h, 3 * h),
        Layer("proj", h, h),
        Layer("fc1", h, mlp, gelu=True),
        Layer("fc2", mlp, h),
    )


CONFIGS: Dict[str, Config] = {
    "deit_tiny_fc1": Config(0, "DeiT-Tiny fc1, batch 8", 8 * 197,
                            (Layer("fc1", 192, 768, gelu=True),)),
    "deit_base_b64": Config(1, "DeiT-Base block, batch 64", 64 * 197, _block(768, 3072)),
    "vit_large_b128": Config(2, "ViT-Large/16 block, batch 128", 128 * 197, _block(1024, 4096)),
    "swin_base_s3_b256": Config(3, "Swin-Base stage 3 block, batch 256", 256 * 196,
                                _block(512, 2048), x_dist="student_t4"),
    "vit_huge_b1": Config(4, "ViT-Huge/14 block, batch 1", 1 * 257, _block(1280, 5120), int8_out=True),
    "vit_huge_b8": Config(4, "ViT-Huge/14 block, batch 8", 8 * 257, _block(1280, 5120), int8_out=True),
    "vit_huge_b64": Config(4, "ViT-Huge/14 block, batch 64", 64 * 257, _block(1280, 5120), int8_out=True),
    "vit_huge_b256": Config(4, "ViT-Huge/14 block, batch 256", 256 * 257, _block(1280, 5120),
                            int8_out=True),
    # the paper's smallest models: output widths that are not multiples of the 128-feature tile
    "deit_tiny_b64": Config(5, "DeiT-Tiny block, batch 64", 64 * 197, _block(192, 768), int8_out=True),
    "swin_tiny_s1_b32": Config(6, "Swin-Tiny stage 1 block, batch 32", 32 * 3136, _block(96, 384),
                               x_dist="student_t4", int8_out=True),
}

_TENSOR_ID = {"W": 0, "bias": 1, "X": 2}


def _rng(seed: int, cid: int, layer_idx: int, tensor: str) -> np.random.Generator:
    ss = np.random.SeedSequence([seed, cid, layer_idx, _TENSOR_ID[tensor]])
    return np.random.Generator(np.random.PCG64(ss))


def make_weight(cfg: Config, layer_idx: int, seed: int = 0) -> np.ndarray:
    L = cfg.layers[layer_idx]
    g = _rng(seed, cfg.cid, layer_idx, "W")
    return (g.standard_normal((L.N, L.K), dtype=np.float32) * np.float32(0.02)).astype(np.float32)


def make_bias(cfg: Config, layer_idx: int, seed: int = 0) -> np.ndarray:
    L = cfg.layers[layer_idx]
    g = _rng(seed, cfg.cid, layer_idx, "bias")
    return (g.standard_normal((L.N,), dtype=np.float32) * np.float32(0.01)).astype(np.float32)


def make_activation(cfg: Config, layer_idx: int, seed: int = 0, M: Optional[int] = None,
                    x_dist: Optional[str] = None) -> np.ndarray:
    """binary16 activations [M, K]; M defaults to the config's token count."""
    L = cfg.layers[layer_idx]
    rows = cfg.M if M is None else M
    dist = cfg.x_dist if x_dist is None else x_dist
    g = _rng(seed, cfg.cid, layer_idx, "X")
    if dist == "normal":
        x = g.standard_normal((rows, L.K), dtype=np.float32)
    elif dist == "student_t4":
        x = (g.standard_t(4.0, size=(rows, L.K)) / np.sqrt(2.0)).astype(np.float32)
    else:
        raise ValueError("unknown activation distribution %r" % dist)
    return x.astype(np.float16)


def make_layer_inputs(cfg: Config, layer_idx: int, seed: int = 0, M: Optional[int] = None) -> dict:
    return {
        "W": make_weight(cfg, layer_idx, seed),
        "bias": make_bias(cfg, layer_idx, seed),
        "X": make_activation(cfg, layer_idx, seed, M),
    }


def random_layer(seed: int, M: int, N: int, K: int, x_dist: str = "normal") -> dict:
    """Free-form shapes for tile-tail and edge-case tests."""
    cfg = Config(1000 + (seed % 1000), "adhoc", M, (Layer("adhoc", K, N),), x_dist=x_dist)
    return make_layer_inputs(cfg, 0, seed)


def config_names() -> List[str]:
    return list(CONFIGS.keys())


# ---- patch embedding (Sec. 3.3): an image batch and a convolution weight with kernel = stride = P ----

@dataclass(frozen=True)
class PatchConfig:
    cid: int
    name: str
    B: int          # images
    C: int          # input channels
    H: int
    W: int
    P: int          # patch size
    D: int          # embedding width

    @property
    def K(self) -> int:
        return self.C * self.P * self.P

    @property
    def Kp(self) -> int:
        """Reduction length padded to the 16 codes the GEMM's row pitch needs."""
        return (self.K + 15) // 16 * 16

    @property
    def tokens(self) -> int:
        return self.B * (self.H // self.P) * (self.W // self.P)


PATCH_CONFIGS: Dict[str, PatchConfig] = {
    "patch16_deit_base_b64": PatchConfig(20, "DeiT-Base patch embedding 16x16, batch 64", 64, 3, 224, 224, 16, 768),
    "patch4_swin_tiny_b32": PatchConfig(21, "Swin-Tiny patch embedding 4x4, batch 32", 32, 3, 224, 224, 4, 96),
    "patch4_swin_base_b32": PatchConfig(22, "Swin-Base patch embedding 4x4, batch 32", 32, 3, 224, 224, 4, 128),
    "patch14_vit_huge_b8": PatchConfig(23, "ViT-Huge patch embedding 14x14, batch 8", 8, 3, 224, 224, 14, 1280),
}

# per-channel mean and standard deviation of the usual ImageNet input normalisation
_PIXEL_MEAN = np.array([0.485, 0.456, 0.406], np.float32)
_PIXEL_STD = np.array([0.229, 0.224, 0.225], np.float32)


def make_patch_inputs(cfg: PatchConfig, seed: int = 0, B: Optional[int] = None) -> dict:
    """img f16 [B, C, H, W] (uniform pixels in [0, 1), normalised per channel), W4 f32 [D, C, P, P], bias f32 [D]."""
    nb = cfg.B if B is None else B
    g = _rng(seed, cfg.cid, 0, "X")
    pix = g.random((nb, cfg.C, cfg.H, cfg.W), dtype=np.float32)
    ch = np.arange(cfg.C) % 3
    img = (pix - _PIXEL_MEAN[ch][None, :, None, None]) / _PIXEL_STD[ch][None, :, None, None]
    gw = _rng(seed, cfg.cid, 0, "W")
    W4 = (gw.standard_normal((cfg.D, cfg.C, cfg.P, cfg.P), dtype=np.float32) * np.float32(0.02)).astype(np.float32)
    gb = _rng(seed, cfg.cid, 0, "bias")
    bias = (gb.standard_normal((cfg.D,), dtype=np.float32) * np.float32(0.01)).astype(np.float32)
    return {"img": img.astype(np.float16), "W4": W4, "bias": bias}


def random_patch(seed: int, B: int, C: int, H: int, W: int, P: int, D: int) -> dict:
    """Free-form patch-embedding shapes for edge-case tests."""
    return make_patch_inputs(PatchConfig(2000 + (seed % 1000), "adhoc", B, C, H, W, P, D), seed)
