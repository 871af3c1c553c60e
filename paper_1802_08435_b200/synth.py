"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

Holds none of the method's arithmetic: only numpy random draws with the shapes
of the WaveRNN workloads (24 kHz / 16-bit audio, H = 896 dense, H = 2048 with
4x4 blocks at 96 % sparsity, 16-way subscale folding, 5 ms conditioning hop).
The paper's own data (a proprietary single-speaker corpus with linguistic
features, Section 5) is not available; these inputs stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

SEED_WEIGHTS = 1802
SEED_BIASES = 1803
SEED_MASK = 96
SEED_COND = 8435
SEED_SAMPLING = 20180223   # Philox key
HOP = 120                  # samples per conditioning frame (5 ms at 24 kHz)
COND_DIM = 64


def make_weights(H: int, cond_dim: int = COND_DIM, seed_w: int = SEED_WEIGHTS,
                 seed_b: int = SEED_BIASES, head_scale: float = 1.0, n_inputs: int = 3,
                 n_logits: int = 256) -> Dict[str, np.ndarray]:
    """All matrices i.i.d. N(0, 1/H), biases N(0, 1/H); fp32, row-major.

    head_scale multiplies O2 and O4 (peaky output distributions for range tests).  n_inputs = 12 and n_logits = 64 give
    the shapes of the Fused Subscale WaveRNN 2x (twelve nibble inputs, four 16-way softmaxes per head).
    """
    assert H % 8 == 0
    Hh = H // 2
    rw = np.random.default_rng(seed_w)
    rb = np.random.default_rng(seed_b)
    s = 1.0 / np.sqrt(H)

    def mat(rng, *shape):
        return (rng.standard_normal(shape) * s).astype(np.float32)

    w = {
        "R": mat(rw, 3 * H, H),
        "I": mat(rw, 3 * H, n_inputs),
        "W_cond": mat(rw, 3 * H, cond_dim) if cond_dim else None,
        "O1": mat(rw, Hh, Hh),
        "O2": mat(rw, n_logits, Hh) * np.float32(head_scale),
        "O3": mat(rw, Hh, Hh),
        "O4": mat(rw, n_logits, Hh) * np.float32(head_scale),
        "b_gate": mat(rb, 3 * H),
        "b1": mat(rb, Hh),
        "b2": mat(rb, n_logits),
        "b3": mat(rb, Hh),
        "b4": mat(rb, n_logits),
    }
    return w


def make_block_masks(H: int, sparsity: float = 0.96, seed: int = SEED_MASK, block=(4, 4)) -> Dict[str, np.ndarray]:
    """Uniform random block masks (block = (rows, columns) of one block: 4 x 4, 16 x 1 or 1 x 1) with exactly
    round((1-sparsity) * n_blocks) kept blocks per matrix; R_u, R_r, R_e are masked separately (stacked as one
    [3H/br][H/bc])."""
    rng = np.random.default_rng(seed)
    Hh = H // 2
    br, bc = block

    def one(rows, cols):
        nb = (rows // br) * (cols // bc)
        keep = int(round((1.0 - sparsity) * nb))
        m = np.zeros(nb, np.uint8)
        m[rng.permutation(nb)[:keep]] = 1
        return m.reshape(rows // br, cols // bc)

    mR = np.concatenate([one(H, H) for _ in range(3)], axis=0)
    return {"R": mR, "O1": one(Hh, Hh), "O3": one(Hh, Hh)}


def rescale_kept(weights: Dict[str, np.ndarray], masks: Dict[str, np.ndarray], sparsity: float = 0.96):
    """Multiply the maskable matrices by 1/sqrt(1-sparsity) so that pre-activation
    variance of the pruned model matches the dense one (a property of the synthetic
    workload, not of the method)."""
    g = np.float32(1.0 / np.sqrt(1.0 - sparsity))
    out = dict(weights)
    for k in masks:
        out[k] = (weights[k] * g).astype(np.float32)
    return out


def make_cond(batch: int, n_frames: int, cond_dim: int = COND_DIM, seed: int = SEED_COND) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.standard_normal((batch, n_frames, cond_dim)).astype(np.float32)


def make_subscale_conv(B: int, F: int, cond_dim: int = COND_DIM, seed: int = 417):
    """Synthetic weights of the one-layer masked convolution that conditions sub-tensor s on sub-tensors z < s
    (Section 4.1): V [B-1][F+1][cond_dim] ~ N(0, 1 / ((F+1) (B-1))) scaled to unit-order outputs, b [cond_dim]."""
    rng = np.random.default_rng(seed)
    V = (rng.standard_normal((max(B - 1, 1), F + 1, cond_dim)) * (3.0 / np.sqrt((F + 1) * max(B - 1, 1)))).astype(np.float32)
    b = (rng.standard_normal(cond_dim) * 0.1).astype(np.float32)
    return V, b


@dataclass
class Workload:
    name: str
    H: int
    dtype: str               # "f32" | "bf16"
    batch: int
    n_steps: int
    n_frames: int
    row_stride: int = 1
    row_offset_mul: int = 0
    sparsity: Optional[float] = None
    subscale_B: int = 0       # >0: fold/unfold of one n_steps*B sequence
    block: tuple = (4, 4)     # shape of one block of the sparsity masks (rows, columns)
    variant: int = 0          # 1: Fused Subscale WaveRNN 2x (two samples per step)
    dependent: Optional[tuple] = None   # (F, chunk, lag): subscale rows conditioned on the earlier rows, staggered schedule
    net: bool = False         # dependent rows conditioned through the ten-layer masked dilated network (else one convolution)


# The five named workloads (index = position in the benchmark's config list), then three extra ones.
WORKLOADS = [
    Workload("dense896_f32_b1_1200", 896, "f32", 1, 1200, 10),
    Workload("dense896_bf16_b1_24000", 896, "bf16", 1, 24000, 200),
    Workload("sparse2048_bf16_b1_24000", 2048, "bf16", 1, 24000, 200, sparsity=0.96),
    Workload("subscale16_896_bf16_1500", 896, "bf16", 16, 1500, 200, row_stride=16, row_offset_mul=1, subscale_B=16),
    Workload("batched256_896_bf16_24000", 896, "bf16", 256, 24000, 200),
    # beyond the five benchmark configurations: the other block shapes of Section 3.2 (same model, same sparsity)
    Workload("sparse2048_16x1_bf16_b1_24000", 2048, "bf16", 1, 24000, 200, sparsity=0.96, block=(16, 1)),
    Workload("sparse2048_1x1_bf16_b1_2400", 2048, "bf16", 1, 2400, 20, sparsity=0.96, block=(1, 1)),
    # the paper's own small-batch point (Section 5.1: four utterances at once)
    Workload("batched4_896_bf16_24000", 896, "bf16", 4, 24000, 200),
    # Fused Subscale WaveRNN 2x (Section 4.4): 12,002 steps = 24,000 samples after the two pre-roll samples
    Workload("fused2x_896_bf16_24000", 896, "bf16", 1, 12002, 102, variant=1),
    # Subscale 16x with dependent rows (Sections 4.1, 4.2): 4 s of audio, F = 128, conditioning 128 positions at a time,
    # rows 256 steps apart (the batch is full after 15 x 256 of the 9,840 global steps)
    Workload("subscale16_dependent_896_bf16_6000", 896, "bf16", 16, 6000, 802, row_stride=16, row_offset_mul=1, subscale_B=16,
             dependent=(128, 128, 256)),
    # the same through the conditioning network with the paper's shape (Section 5.3)
    Workload("subscale16_net_896_bf16_6000", 896, "bf16", 16, 6000, 802, row_stride=16, row_offset_mul=1, subscale_B=16,
             dependent=(128, 128, 256), net=True),
]


def build_workload(wl: Workload, n_steps: Optional[int] = None, batch: Optional[int] = None):
    """-> (weights, masks or None, cond[batch][n_frames][64]).  n_steps/batch shrink the case."""
    w = make_weights(wl.H, n_inputs=12, n_logits=64) if wl.variant == 1 else make_weights(wl.H)
    masks = None
    if wl.sparsity is not None:
        masks = make_block_masks(wl.H, wl.sparsity, block=wl.block)
        w = rescale_kept(w, masks, wl.sparsity)
    b = wl.batch if batch is None else batch
    cond = make_cond(b, wl.n_frames)
    return w, masks, cond


# Shape of the paper's conditioning network of the Subscale WaveRNN (Section 5.3): ten layers, kernel size 3, 384
# convolution channels, 768 residual channels, five stages of increasing dilation.
NET_DILATIONS = (1, 1, 2, 2, 4, 4, 8, 8, 16, 16)
NET_CONV_CH = 384
NET_RES_CH = 768


def make_subscale_net(B: int, cond_dim: int = COND_DIM, conv_ch: int = NET_CONV_CH, res_ch: int = NET_RES_CH,
                      dilations=NET_DILATIONS, taps: int = 3, seed: int = 418) -> Dict[str, np.ndarray]:
    """Synthetic weights of the masked dilated conditioning network (the trained ones do not exist here): every matrix
    i.i.d. normal, scaled so that activations stay of order one through the residual stack (the residual branch of a
    layer adds about 0.3 rms); small biases.  fp32, row-major:
        W_in [res][B], b_in [res]; W_conv [layers][taps][conv][res], b_conv [layers][conv];
        W_res [layers][res][conv], b_res [layers][res]; W_out [cond_dim][res], b_out [cond_dim]; dilation int32 [layers].
    """
    rng = np.random.default_rng(seed)
    nl = len(dilations)

    def mat(scale, *shape):
        return (rng.standard_normal(shape) * scale).astype(np.float32)

    return {
        "dilation": np.asarray(dilations, np.int32),
        "W_in": mat(1.0 / np.sqrt(max(B - 1, 1) / 3.0), res_ch, B), "b_in": mat(0.1, res_ch),
        "W_conv": mat(1.0 / np.sqrt(taps * res_ch), nl, taps, conv_ch, res_ch), "b_conv": mat(0.1, nl, conv_ch),
        "W_res": mat(0.5 / np.sqrt(conv_ch), nl, res_ch, conv_ch), "b_res": mat(0.02, nl, res_ch),
        "W_out": mat(1.5 / np.sqrt(res_ch), cond_dim, res_ch), "b_out": mat(0.1, cond_dim),
    }
