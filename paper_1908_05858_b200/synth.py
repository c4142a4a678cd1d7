"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method (no sign, no packing, no convolution, no BN
fold): it only draws random tensors, so that the CUDA library and the CPU oracle can be fed
identical host arrays without sharing any code of their own.

The paper measures single binary convolutions and Bi-Real Net 18 on ImageNet-sized images
(Section 2.2, Fig. 5; Table 2).  ImageNet and trained weights are not available, so seeded
N(0,1) tensors of the same shapes stand in for them: the ResNet-18 / Bi-Real-18 stage shapes
(C = 64/128/256/512 at 56/28/14/7 pixels) for the convolutions, 3x224x224 images for the network.

Every tensor has its own stream: seed = 190805858*1000 + 10*config_id + tensor_id.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 190805858 * 1000

# (C, HW) of the four ResNet-18 stages; C_in = C_out, 3x3, stride 1, pad 1, pad value -1
SWEEP_SHAPES = ((64, 56), (128, 28), (256, 14), (512, 7))
STAGE_C = (64, 128, 256, 512)
STAGE_HW = (56, 28, 14, 7)


def rng(config_id: int, tensor_id: int) -> np.random.Generator:
    return np.random.default_rng(BASE_SEED + 10 * config_id + tensor_id)


def normal(config_id: int, tensor_id: int, shape) -> np.ndarray:
    return rng(config_id, tensor_id).standard_normal(size=shape, dtype=np.float32)


def conv_case(config_id: int, N: int, C: int, H: int, W: int, O: int, kh: int, kw: int, salt: int = 0):
    """fp32 N(0,1) activations (NCHW) and weights (OIHW) for one binary convolution."""
    x = normal(config_id, 0 + 2 * salt, (N, C, H, W))
    w = normal(config_id, 1 + 2 * salt, (O, C, kh, kw))
    return x, w


def pack_case(N: int = 128, C: int = 256, H: int = 56, W: int = 56, zero_frac: float = 0.01, config_id: int = 3):
    """fp32 NCHW N(0,1) tensor with about 1 % of the entries set to exact +0.0."""
    g = rng(config_id, 0)
    x = g.standard_normal(size=(N, C, H, W), dtype=np.float32)
    # mask drawn in slabs to keep the peak host memory low
    for n in range(N):
        m = g.random(size=(C, H, W), dtype=np.float32) < zero_frac
        x[n][m] = 0.0
    return x


def bn_params(g: np.random.Generator, O: int):
    """gamma ~ U(0.5,1.5), beta ~ N(0,0.1), running mean ~ N(0,0.1), running var ~ U(0.5,1.5)."""
    gamma = g.uniform(0.5, 1.5, size=O).astype(np.float32)
    beta = (0.1 * g.standard_normal(size=O)).astype(np.float32)
    mean = (0.1 * g.standard_normal(size=O)).astype(np.float32)
    var = g.uniform(0.5, 1.5, size=O).astype(np.float32)
    return gamma, beta, mean, var


def bireal18_params(config_id: int = 4) -> dict:
    """Random-init Bi-Real Net 18 parameters (fp32 numpy arrays)."""
    g = rng(config_id, 1)
    p = {"bn_eps": 1e-5}
    p["stem_w"] = (g.standard_normal(size=(64, 3, 7, 7)) / np.sqrt(147.0)).astype(np.float32)
    p["stem_bn"] = bn_params(g, 64)
    p["block_w"], p["block_bn"], p["down_w"], p["down_bn"] = [], [], [], []
    C = 64
    for b in range(16):
        O = STAGE_C[b // 4]
        p["block_w"].append(g.standard_normal(size=(O, C, 3, 3), dtype=np.float32))
        p["block_bn"].append(bn_params(g, O))
        if b % 4 == 0 and b > 0:
            p["down_w"].append((g.standard_normal(size=(O, C)) / np.sqrt(float(C))).astype(np.float32))
            p["down_bn"].append(bn_params(g, O))
        C = O
    p["fc_w"] = (g.standard_normal(size=(1000, 512)) / np.sqrt(512.0)).astype(np.float32)
    p["fc_b"] = (0.1 * g.standard_normal(size=1000)).astype(np.float32)
    return p


def stem_module_params(config_id: int = 4) -> dict:
    """Random-init parameters of the STEM module (Section 2.3): four fp32 convolutions (OIHW, N(0,1)/sqrt(fan_in)) with a
    BN each: 3x3/2 3->32, 1x1 32->16, 3x3/2 16->32, 1x1 64->64."""
    g = rng(config_id, 2)
    shapes = ((32, 3, 3, 3), (16, 32, 1, 1), (32, 16, 3, 3), (64, 64, 1, 1))
    w = [(g.standard_normal(size=sh) / np.sqrt(float(sh[1] * sh[2] * sh[3]))).astype(np.float32) for sh in shapes]
    return {"w": w, "bn": [bn_params(g, sh[0]) for sh in shapes]}


def bireal18_images(N: int, config_id: int = 4) -> np.ndarray:
    """fp32 NCHW N x 3 x 224 x 224, N(0,1); image n is the same for every N (drawn one by one)."""
    out = np.empty((N, 3, 224, 224), dtype=np.float32)
    for n in range(N):
        out[n] = np.random.default_rng(BASE_SEED + 10 * config_id + 1000 * (n + 1)).standard_normal(
            size=(3, 224, 224), dtype=np.float32)
    return out
