"""Seeded synthetic inputs shaped like the paper's two deployment workloads.

This module only *draws numbers and arranges them*: it contains no quantiser,
no packing and no matmul, and it imports neither the CUDA binding nor the CPU
oracle, so both sides can be fed the same tensors.

Workloads (shapes follow the models the paper deploys, Sec. 2.2 and Sec. 5.4):
  * ``cfg0``  one weight-only linear, M=1, K=N=4096;
  * ``cfg1``  the seven linears of a Llama-2-7B decoder layer (the OpenVLA
              backbone) x 32 layers at decode batch 1, weights N(0, 0.02) with
              0.1 % of entries replaced by +-6 sigma;
  * ``cfg2``  the same shapes at prefill length 280;
  * ``cfg3``  M sweep on 4096->11008 and 11008->4096;
  * ``cfg4``  3x3 convolutions of a ResNet-34-like encoder (the CILRS image
              encoder) lowered to GEMM by im2col, batch 32, input 3x88x200.

bf16 tensors are carried as uint16 bit patterns.
"""
from __future__ import annotations

import numpy as np

GROUP_SIZE = 128
SIGMA_LLM = 0.02
SIGMA_CONV = 0.05
HIDDEN = 4096
FFN = 11008
N_LAYERS = 32
ACTION_TOKENS = 7
PREFILL_M = 280

# (name, N = out features, K = in features) of one Llama-2-7B decoder layer
LLAMA2_7B_LAYER = (
    ("q", HIDDEN, HIDDEN), ("k", HIDDEN, HIDDEN), ("v", HIDDEN, HIDDEN), ("o", HIDDEN, HIDDEN),
    ("gate", FFN, HIDDEN), ("up", FFN, HIDDEN), ("down", HIDDEN, FFN),
)

# The same layer with the projections that read the same input stored as one linear each (q, k, v and gate, up:
# group-wise quantisation is per output row, so stacking rows changes no code, scale or result)
LLAMA2_7B_LAYER_FUSED = (
    ("qkv", 3 * HIDDEN, HIDDEN), ("o", HIDDEN, HIDDEN), ("gate_up", 2 * FFN, HIDDEN), ("down", HIDDEN, FFN),
)

# (Cin = Cout, H, W) of the four 3x3 conv stages at batch 32, input 3x88x200
CONV_STAGES = ((64, 22, 50), (128, 11, 25), (256, 6, 13), (512, 3, 7))
CONV_BATCH = 32


def generator(cfg: int, tensor_id: int) -> np.random.Generator:
    """One independent stream per (config, tensor)."""
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(cfg), int(tensor_id)])))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_weights(cfg: int, tensor_id: int, N: int, K: int, sigma: float,
                   outlier_prob: float = 0.0, outlier_sigmas: float = 6.0) -> np.ndarray:
    """fp32 [N][K] ~ N(0, sigma); optionally each entry is, independently with
    probability ``outlier_prob``, replaced by +-outlier_sigmas*sigma (fair sign).

    The replaced positions are drawn as the success times of a Bernoulli process (gaps between
    successes are geometric), which has the same law as one Bernoulli draw per entry.
    """
    g = generator(cfg, tensor_id)
    w = g.standard_normal((N, K), dtype=np.float32)
    w *= np.float32(sigma)
    if outlier_prob > 0.0:
        total = N * K
        pos = np.empty(0, dtype=np.int64)
        last = -1
        while last < total:
            gaps = g.geometric(outlier_prob, size=int(total * outlier_prob * 1.2) + 64)
            more = last + np.cumsum(gaps, dtype=np.int64)
            pos = np.concatenate([pos, more])
            last = int(more[-1])
        pos = pos[pos < total]
        sign = g.integers(0, 2, size=pos.size).astype(np.float32) * 2.0 - 1.0
        w.reshape(-1)[pos] = sign * np.float32(outlier_sigmas * sigma)
    return w


def normal_activations_bf16(cfg: int, tensor_id: int, M: int, K: int) -> np.ndarray:
    """bf16 bits [M][K] of N(0,1) draws."""
    g = generator(cfg, tensor_id)
    return f32_to_bf16_bits(g.standard_normal((M, K), dtype=np.float32))


# ---- config 0 ---------------------------------------------------------------
def cfg0():
    w = normal_weights(0, 0, HIDDEN, HIDDEN, SIGMA_LLM)
    x = normal_activations_bf16(0, 1, 1, HIDDEN)
    return w, x


# ---- config 1 / 2 -----------------------------------------------------------
def llama_linear_ids():
    """[(layer, name, N, K, tensor_id_w, tensor_id_x)] for all 224 linears, in stream order."""
    out = []
    for layer in range(N_LAYERS):
        for j, (name, N, K) in enumerate(LLAMA2_7B_LAYER):
            idx = layer * len(LLAMA2_7B_LAYER) + j
            out.append((layer, name, N, K, 2 * idx, 2 * idx + 1))
    return out


def llama_weight(cfg: int, tensor_id_w: int, N: int, K: int, outliers: bool = True) -> np.ndarray:
    return normal_weights(cfg, tensor_id_w, N, K, SIGMA_LLM, 0.001 if outliers else 0.0)


def cfg1_bytes_per_step() -> int:
    """Algorithmic weight-side bytes of one decode pass: packed codes + fp16 scale + fp16 zero."""
    total = 0
    for _, N, K in LLAMA2_7B_LAYER:
        total += N * K // 2 + 2 * 2 * N * (K // GROUP_SIZE)
    return total * N_LAYERS


# ---- config 4 ---------------------------------------------------------------
def im2col_3x3(fmap_bits: np.ndarray) -> np.ndarray:
    """[B][H][W][C] -> [B*H*W][9*C], 3x3 window, stride 1, zero pad 1,
    column index = (kh*3 + kw)*C + c."""
    B, H, W, Cc = fmap_bits.shape
    padded = np.zeros((B, H + 2, W + 2, Cc), dtype=fmap_bits.dtype)
    padded[:, 1:H + 1, 1:W + 1, :] = fmap_bits
    cols = np.empty((B, H, W, 9, Cc), dtype=fmap_bits.dtype)
    for kh in range(3):
        for kw in range(3):
            cols[:, :, :, kh * 3 + kw, :] = padded[:, kh:kh + H, kw:kw + W, :]
    return cols.reshape(B * H * W, 9 * Cc)


def conv_stage(stage: int, batch: int = CONV_BATCH):
    """(x bf16 bits [M][K], w fp32 [N][K]) of conv stage 0..3: ReLU(N(0,1)) feature map, N(0,0.05) weights."""
    Cc, H, W = CONV_STAGES[stage]
    g = generator(4, 2 * stage)
    fmap = np.maximum(g.standard_normal((batch, H, W, Cc), dtype=np.float32), np.float32(0))
    x = im2col_3x3(f32_to_bf16_bits(fmap))
    w = normal_weights(4, 2 * stage + 1, Cc, 9 * Cc, SIGMA_CONV)
    return x, w


def conv_gemm_shape(stage: int, batch: int = CONV_BATCH):
    Cc, H, W = CONV_STAGES[stage]
    return batch * H * W, 9 * Cc, Cc
