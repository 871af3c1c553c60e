"""Independent brute-force restatement of the WaveRNN step for tiny sizes.

Written separately from the C oracle, directly from Eq. 2 in matrix form: the
masked matrix I* is built explicitly (its c_t column zeroed on the coarse rows),
the whole gate vector is evaluated from x_t = [c_{t-1}, f_{t-1}, c_t], and the
coarse / fine halves are read out of it.  numpy float64 / Python ints only.
"""
from __future__ import annotations

import numpy as np

M32 = 0xFFFFFFFF


def philox4x32_10_py(ctr, key):
    """Second, independent Philox4x32-10 (Python integers)."""
    c = [int(v) & M32 for v in ctr]
    k = [int(v) & M32 for v in key]
    for r in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & M32, p1 & M32, ((p0 >> 32) ^ c[3] ^ k[1]) & M32, p0 & M32]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def uniform_py(seed, stream, step, head):
    out = philox4x32_10_py([step & M32, head, stream, step >> 32], [seed & M32, seed >> 32])
    return (out[0] >> 8) / float(1 << 24)


def masked_I(I, H):
    """I* of Eq. 2: the c_t column reaches only the fine half of each gate."""
    Is = np.array(I, dtype=np.float64, copy=True)
    Hh = H // 2
    for gate in range(3):
        Is[gate * H: gate * H + Hh, 2] = 0.0
    return Is


def gates_full(w, h_prev, x, g):
    """u, r, e, h_new for the whole state from Eq. 2 (x already scaled)."""
    H = h_prev.shape[0]
    R = w["R"].astype(np.float64)
    Is = masked_I(w["I"], H)
    a = R @ h_prev.astype(np.float64)
    ix = Is @ x + g
    u = 1.0 / (1.0 + np.exp(-(a[:H] + ix[:H])))
    r = 1.0 / (1.0 + np.exp(-(a[H:2 * H] + ix[H:2 * H])))
    e = np.tanh(r * a[2 * H:] + ix[2 * H:])
    hn = u * h_prev.astype(np.float64) + (1.0 - u) * e
    return u, r, e, hn


def draw(logits, u):
    l = logits.astype(np.float64)
    p = np.exp(l - l.max())
    cdf = np.cumsum(p)
    k = int(np.searchsorted(cdf, u * cdf[-1], side="right"))
    return min(k, len(l) - 1)


def step(w, h_prev, c_prev, f_prev, frame, seed, stream, t, c_forced=None, f_forced=None):
    """One sampling step in the order of Fig. 1; returns dict of everything."""
    H = h_prev.shape[0]
    Hh = H // 2
    g = np.zeros(3 * H)
    if w.get("b_gate") is not None:
        g = g + w["b_gate"].astype(np.float64)
    if w.get("W_cond") is not None:
        g = g + w["W_cond"].astype(np.float64) @ frame.astype(np.float64)
    sc = lambda v: v / 127.5 - 1.0
    # coarse: c_t unknown; its column is masked on the coarse rows anyway
    x = np.array([sc(c_prev), sc(f_prev), 0.0])
    u, r, e, hn = gates_full(w, h_prev, x, g)
    yc = hn[:Hh].astype(np.float32).astype(np.float64)
    qc = np.maximum(w["O1"].astype(np.float64) @ yc + w["b1"], 0.0)
    lc = (w["O2"].astype(np.float64) @ qc + w["b2"]).astype(np.float32)
    c_draw = draw(lc, uniform_py(seed, stream, t, 0))
    c_t = c_draw if c_forced is None else c_forced
    x = np.array([sc(c_prev), sc(f_prev), sc(c_t)])
    u2, r2, e2, hn2 = gates_full(w, h_prev, x, g)
    yf = hn2[Hh:].astype(np.float32).astype(np.float64)
    qf = np.maximum(w["O3"].astype(np.float64) @ yf + w["b3"], 0.0)
    lf = (w["O4"].astype(np.float64) @ qf + w["b4"]).astype(np.float32)
    f_draw = draw(lf, uniform_py(seed, stream, t, 1))
    f_t = f_draw if f_forced is None else f_forced
    h_new = np.concatenate([hn[:Hh], hn2[Hh:]]).astype(np.float32)
    gates = np.concatenate([
        np.concatenate([u[:Hh], u2[Hh:]]), np.concatenate([r[:Hh], r2[Hh:]]),
        np.concatenate([e[:Hh], e2[Hh:]])])
    return dict(h=h_new, c=c_t, f=f_t, c_draw=c_draw, f_draw=f_draw, lc=lc, lf=lf, gates=gates,
                coarse_after=hn2[:Hh].astype(np.float32))
