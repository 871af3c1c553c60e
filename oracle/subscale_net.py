"""CPU oracle of the conditioning network of the Subscale WaveRNN (Sections 4.1, 5.3).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the benchmark's CPU-baseline leg may import
this.  Plain numpy in float64, one statement per step of the definition; the matrix products are numpy's.

What the paper fixes: the WaveRNN that generates sub-tensor s is conditioned on the FUTURE context of the sub-tensors
z < s through a masked dilated 1-D CNN with relus, "the mask applied over past connections instead of future ones";
the network has ten layers, kernels of size 3, 384 convolution channels, 768 residual channels, five stages of
increasing dilation, and sees a future horizon of F = 128 positions (a position = one block of B samples).  The paper
prints neither equations nor weights for it, so everything below is a stated reading (parity unpinned beyond the
structural pins of tests/test_oracle_subscale_net.py):

  N1  input of sub-tensor s at position i: the block X[i][z] = x(u_{B i + z}) for z < s, 0 for z >= s, x(u) = u / 32768
  N2  x_0[i] = W_in X[i] + b_in                                   (B -> 768 residual channels)
  N3  layer l = 0..9 with dilation d_l = 1, 1, 2, 2, 4, 4, 8, 8, 16, 16 (five stages of two layers):
          a_l[i]     = relu(b_conv[l] + sum_{t=0..2} W_conv[l][t] x_l[i + t d_l])      (768 -> 384; taps at 0, +d, +2d:
                                                                                       a size-3 kernel whose connections
                                                                                       reach forward only)
          x_{l+1}[i] = x_l[i] + W_res[l] a_l[i] + b_res[l]                             (384 -> 768, residual)
      positions at or beyond the row length hold the zero vector in every layer (they contribute nothing)
  N4  v_s[i] = frame_s[(B i + s) div hop] + W_out relu(x_10[i]) + b_out               (768 -> conditioning vector)
  N5  reach: sum_l 2 d_l = 124 positions <= F = 128; the staggered schedule keeps rows F + chunk apart
  N6  the weights are rounded to bf16 (round to nearest even) when the network is created, as the WaveRNN's are
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

from oracle import wrnn_oracle as orc

_MATS = ("W_in", "W_conv", "W_res", "W_out")


class SubscaleNet:
    """The stored network: matrices rounded to bf16 (N6), biases fp32."""

    def __init__(self, weights: Dict[str, np.ndarray], round_bf16: bool = True):
        self.w = {}
        for k, a in weights.items():
            a = np.ascontiguousarray(a)
            if k in _MATS:
                a = orc.bf16_round(a.astype(np.float32)).reshape(a.shape) if round_bf16 else a.astype(np.float32)
            self.w[k] = a
        self.dilation = [int(d) for d in self.w["dilation"]]
        self.n_layers = len(self.dilation)
        self.taps = int(self.w["W_conv"].shape[1])
        self.B = int(self.w["W_in"].shape[1])
        self.cond_dim = int(self.w["W_out"].shape[0])
        self.reach = sum((self.taps - 1) * d for d in self.dilation)

    def conditioning(self, history: np.ndarray, s: int) -> np.ndarray:
        """history int16 [B][L] (rows z < s complete) -> the network term of v_s for all positions, float32 [L][cond_dim]."""
        w = self.w
        B, L = history.shape
        assert B == self.B
        X = history.astype(np.float64).T / 32768.0                 # [L][B]
        X[:, s:] = 0.0                                             # N1: only the sub-tensors z < s are visible
        x = X @ w["W_in"].astype(np.float64).T + w["b_in"].astype(np.float64)          # N2
        for l, d in enumerate(self.dilation):                      # N3
            acc = np.tile(w["b_conv"][l].astype(np.float64), (L, 1))
            for t in range(self.taps):
                o = t * d
                if o < L:
                    acc[:L - o] += x[o:] @ w["W_conv"][l, t].astype(np.float64).T
            a = np.maximum(acc, 0.0)
            x = x + a @ w["W_res"][l].astype(np.float64).T + w["b_res"][l].astype(np.float64)
        v = np.maximum(x, 0.0) @ w["W_out"].astype(np.float64).T + w["b_out"].astype(np.float64)   # N4
        return v.astype(np.float32)


def subscale_net_run(om: "orc.OracleModel", net: SubscaleNet, frames: np.ndarray, L: int, hop: int, seed: int,
                     forced: Optional[np.ndarray] = None, teacher: bool = False):
    """Generate the B sub-tensors one after the other (the order of Eq. 4), row s an ordinary WaveRNN stream (Philox
    stream id s, step = position) whose conditioning vector at step i is v_s[i] (N4).  forced / teacher as in
    wrnn_oracle.subscale_dependent_run.  -> (samples int16 [B][L], cond float32 [B][L][D], margins [B][L][2])."""
    B, D = net.B, om.cond_dim
    out = np.zeros((B, L), np.int16)
    cond = np.zeros((B, L, D), np.float32)
    margins = np.zeros((B, L, 2), np.float64)
    for s in range(B):
        hist = out if forced is None else forced
        idx = (B * np.arange(L) + s) // hop
        cond[s] = frames[s][idx] + net.conditioning(hist, s)
        if teacher and forced is not None:
            cf, ff = orc.split_samples(forced[s])
            r = om.run(cond[s][None], L, 1, seed, hop=1, stream0=s, c_forced=cf, f_forced=ff)
            out[s] = orc.join_samples(r.c_out[0], r.f_out[0])
        else:
            r = om.run(cond[s][None], L, 1, seed, hop=1, stream0=s)
            out[s] = r.out[0]
        margins[s] = r.margins[0]
    return out, cond, margins
