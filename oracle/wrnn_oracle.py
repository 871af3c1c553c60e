"""ctypes front end of the CPU oracle (``wrnn_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the
benchmark's CPU-baseline leg may import this.  It holds no arithmetic of the
method: it builds the C file with gcc, marshals numpy arrays and calls it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wrnn_oracle.c")
_LIB = os.path.join(_HERE, "libwrnn_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2: no fast-math, no reassociation)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [("H", C.c_int32), ("cond_dim", C.c_int32)] + [
        (n, C.c_void_p)
        for n in ("R", "I", "b_gate", "W_cond", "O1", "b1", "O2", "b2", "O3", "b3", "O4", "b4")
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_uniform.restype = C.c_double
        L.orc_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32]
        L.orc_philox4x32_10.argtypes = [C.c_void_p] * 3
        L.orc_bf16_round.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.orc_apply_block_mask.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_apply_block_mask_shape.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int]
        L.orc_scale8.restype = C.c_double
        L.orc_scale8.argtypes = [C.c_int]
        L.orc_to_int16.restype = C.c_int16
        L.orc_to_int16.argtypes = [C.c_uint8, C.c_uint8]
        L.orc_join16.restype = C.c_uint16
        L.orc_join16.argtypes = [C.c_uint8, C.c_uint8]
        L.orc_split16.argtypes = [C.c_uint16, C.c_void_p, C.c_void_p]
        L.orc_fold.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p]
        L.orc_unfold.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p]
        L.orc_softmax_sample.restype = C.c_int
        L.orc_softmax_sample.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_run.restype = C.c_int
        L.orc_run.argtypes = (
            [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int,
             C.c_int64, C.c_uint64, C.c_uint32] + [C.c_void_p] * 12 + [C.c_int]
        )
        L.orc_scale4.restype = C.c_double
        L.orc_scale4.argtypes = [C.c_int]
        L.orc_split_nibbles.argtypes = [C.c_uint16, C.c_void_p]
        L.orc_join_nibbles.restype = C.c_uint16
        L.orc_join_nibbles.argtypes = [C.c_void_p]
        L.orc_fs2_run.restype = C.c_int
        L.orc_fs2_run.argtypes = ([C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_uint64, C.c_uint32]
                                  + [C.c_void_p] * 12)
        L.orc_fs2_unfold.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def uniform(seed: int, stream: int, step: int, head: int) -> float:
    return lib().orc_uniform(seed, stream, step, head)


def bf16_round(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty_like(x)
    lib().orc_bf16_round(_ptr(x), _ptr(out), x.size)
    return out


def apply_block_mask(W: np.ndarray, mask: np.ndarray, block=(4, 4)) -> np.ndarray:
    """Zero the blocks of W (block = (rows, columns) of one block) whose mask entry is 0."""
    W = np.array(W, dtype=np.float32, order="C", copy=True)
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    br, bc = int(block[0]), int(block[1])
    assert W.shape[0] % br == 0 and W.shape[1] % bc == 0 and m.shape == (W.shape[0] // br, W.shape[1] // bc)
    lib().orc_apply_block_mask_shape(_ptr(W), W.shape[0], W.shape[1], _ptr(m), br, bc)
    return W


def scale8(v: int) -> float:
    return lib().orc_scale8(int(v))


def to_int16(c: int, f: int) -> int:
    return lib().orc_to_int16(int(c), int(f))


def join16(c: int, f: int) -> int:
    return lib().orc_join16(int(c), int(f))


def split16(x: int):
    c = C.c_uint8()
    f = C.c_uint8()
    lib().orc_split16(int(x), C.byref(c), C.byref(f))
    return c.value, f.value


def split_samples(x: np.ndarray):
    """int16 samples -> (coarse, fine) uint8 arrays, element by element through the C routines."""
    x = np.ascontiguousarray(x, dtype=np.int16)
    cf = [split16((int(v) + 32768) & 0xFFFF) for v in x.reshape(-1)]
    c = np.array([a for a, _ in cf], np.uint8).reshape(x.shape)
    f = np.array([b for _, b in cf], np.uint8).reshape(x.shape)
    return c, f


def join_samples(c: np.ndarray, f: np.ndarray) -> np.ndarray:
    """(coarse, fine) uint8 arrays -> int16 samples, element by element through the C routine."""
    c = np.asarray(c, np.uint8)
    f = np.asarray(f, np.uint8)
    return np.array([to_int16(int(a), int(b)) for a, b in zip(c.reshape(-1), f.reshape(-1))], np.int16).reshape(c.shape)


def fold(x: np.ndarray, B: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.int16)
    assert x.size % B == 0
    sub = np.empty((B, x.size // B), dtype=np.int16)
    lib().orc_fold(_ptr(x), x.size, B, _ptr(sub))
    return sub


def unfold(sub: np.ndarray) -> np.ndarray:
    sub = np.ascontiguousarray(sub, dtype=np.int16)
    B = sub.shape[0]
    x = np.empty(sub.size, dtype=np.int16)
    lib().orc_unfold(_ptr(sub), sub.size, B, _ptr(x))
    return x


def softmax_sample(logits: np.ndarray, u: float):
    """-> (index, probs[n], margin)."""
    l = np.ascontiguousarray(logits, dtype=np.float32)
    probs = np.empty(l.size, dtype=np.float64)
    margin = C.c_double()
    idx = lib().orc_softmax_sample(_ptr(l), l.size, float(u), _ptr(probs), C.byref(margin))
    return idx, probs, margin.value


_WEIGHT_KEYS = ("R", "I", "W_cond", "O1", "O2", "O3", "O4")
_BIAS_KEYS = ("b_gate", "b1", "b2", "b3", "b4")


@dataclass
class RunResult:
    out: np.ndarray            # int16 [batch][n_steps]
    c_out: np.ndarray          # uint8 [batch][n_steps]  indices the oracle drew
    f_out: np.ndarray
    margins: np.ndarray        # float64 [batch][n_steps][2]
    h: np.ndarray              # float32 [batch][H]  final state
    c_prev: np.ndarray
    f_prev: np.ndarray
    gates: Optional[np.ndarray] = None   # [n_steps][batch][3H]
    hs: Optional[np.ndarray] = None      # [n_steps][batch][H]
    logits: Optional[np.ndarray] = None  # [n_steps][batch][2][256]


class OracleModel:
    """The stored model: masks applied, then weights rounded to the storage type.

    `weights` is a dict of fp32 arrays (R, I, b_gate, W_cond, O1, b1, ... b4);
    `masks` an optional dict with block masks for "R" [3H/br][H/bc], "O1",
    "O3" [H/2/br][H/2/bc], `block` = (br, bc) the shape of one block (4 x 4,
    16 x 1 or 1 x 1, Section 3.2); dtype "f32" or "bf16" (weights R, I, W_cond,
    O1..O4 rounded to bf16; biases stay fp32).
    """

    def __init__(self, weights: dict, dtype: str = "f32", masks: Optional[dict] = None, block=(4, 4)):
        assert dtype in ("f32", "bf16")
        self.H = int(weights["R"].shape[1])
        assert weights["R"].shape == (3 * self.H, self.H)
        self.cond_dim = 0 if weights.get("W_cond") is None else int(weights["W_cond"].shape[1])
        self.dtype = dtype
        w = {}
        for k in _WEIGHT_KEYS:
            a = weights.get(k)
            if a is None:
                w[k] = None
                continue
            a = np.array(a, dtype=np.float32, order="C", copy=True)
            if masks and masks.get(k) is not None:
                a = apply_block_mask(a, masks[k], block)
            if dtype == "bf16":
                a = bf16_round(a)
            w[k] = a
        for k in _BIAS_KEYS:
            a = weights.get(k)
            w[k] = None if a is None else np.array(a, dtype=np.float32, order="C", copy=True)
        self.w = w
        self._p = _Params(self.H, self.cond_dim, *[_ptr(w[k]) for k in (
            "R", "I", "b_gate", "W_cond", "O1", "b1", "O2", "b2", "O3", "b3", "O4", "b4")])

    def run(self, cond: Optional[np.ndarray], n_steps: int, batch: int = 1, seed: int = 0, *,
            hop: int = 120, row_stride: int = 1, row_offset_mul: int = 0, step0: int = 0,
            stream0: int = 0,
            h: Optional[np.ndarray] = None, c_prev=None, f_prev=None,
            c_forced: Optional[np.ndarray] = None, f_forced: Optional[np.ndarray] = None,
            dump: bool = False, threads: int = 1) -> RunResult:
        H = self.H
        n_frames = 0
        if self.cond_dim:
            cond = np.ascontiguousarray(cond, dtype=np.float32)
            assert cond.ndim == 3 and cond.shape[0] == batch and cond.shape[2] == self.cond_dim
            n_frames = cond.shape[1]
        else:
            cond = None
        hh = np.zeros((batch, H), np.float32) if h is None else np.array(h, np.float32, copy=True).reshape(batch, H)
        cp = np.full(batch, 128, np.uint8) if c_prev is None else np.array(c_prev, np.uint8, copy=True).reshape(batch)
        fp = np.zeros(batch, np.uint8) if f_prev is None else np.array(f_prev, np.uint8, copy=True).reshape(batch)
        if c_forced is not None:
            c_forced = np.ascontiguousarray(c_forced, np.uint8).reshape(batch, n_steps)
            f_forced = np.ascontiguousarray(f_forced, np.uint8).reshape(batch, n_steps)
        out = np.zeros((batch, n_steps), np.int16)
        c_out = np.zeros((batch, n_steps), np.uint8)
        f_out = np.zeros((batch, n_steps), np.uint8)
        margins = np.zeros((batch, n_steps, 2), np.float64)
        gates = hs = logits = None
        if dump:
            gates = np.zeros((n_steps, batch, 3 * H), np.float32)
            hs = np.zeros((n_steps, batch, H), np.float32)
            logits = np.zeros((n_steps, batch, 2, 256), np.float32)
        rc = lib().orc_run(C.byref(self._p), _ptr(cond), n_frames, hop, row_stride, row_offset_mul,
                           n_steps, batch, step0, seed, stream0, _ptr(hh), _ptr(cp), _ptr(fp),
                           _ptr(c_forced), _ptr(f_forced), _ptr(out), _ptr(c_out), _ptr(f_out),
                           _ptr(margins), _ptr(gates), _ptr(hs), _ptr(logits), threads)
        if rc != 0:
            raise ValueError("conditioning frame index out of range")
        return RunResult(out, c_out, f_out, margins, hh, cp, fp, gates, hs, logits)


# ----------------------------------------------------------------------------------------------
# Fused Subscale WaveRNN 2x

def scale4(v: int) -> float:
    return lib().orc_scale4(int(v))


def split_nibbles(x: int):
    n = (C.c_uint8 * 4)()
    lib().orc_split_nibbles(int(x), n)
    return list(n)


def join_nibbles(n) -> int:
    a = (C.c_uint8 * 4)(*[int(v) for v in n])
    return lib().orc_join_nibbles(a)


def fs2_unfold(ab: np.ndarray) -> np.ndarray:
    ab = np.ascontiguousarray(ab, dtype=np.int16)
    n = ab.shape[1]
    u = np.zeros(2 * max(n - 2, 0), dtype=np.int16)
    lib().orc_fs2_unfold(_ptr(ab), n, _ptr(u))
    return u


@dataclass
class Fs2Result:
    out: np.ndarray            # int16 [2][n_steps]: row 0 a_t, row 1 the b of step t
    a_out: np.ndarray          # uint16 [n_steps] samples the oracle drew
    b_out: np.ndarray
    margins: np.ndarray        # float64 [n_steps][8]
    h: np.ndarray
    a_prev: int
    b_prev: int
    gates: Optional[np.ndarray] = None   # [n_steps][3H]
    hs: Optional[np.ndarray] = None      # [n_steps][H]
    logits: Optional[np.ndarray] = None  # [n_steps][2][64]


class Fs2OracleModel(OracleModel):
    """Fused Subscale WaveRNN 2x: the same cell with I of 12 columns and heads of 64 logits (4 softmaxes of 4 bits)."""

    def __init__(self, weights: dict, dtype: str = "f32"):
        super().__init__(weights, dtype)
        H = self.H
        assert self.w["I"].shape == (3 * H, 12) and self.w["O2"].shape == (64, H // 2) and self.w["O4"].shape == (64, H // 2)

    def run(self, cond: Optional[np.ndarray], n_steps: int, seed: int = 0, *, hop: int = 120, step0: int = 0, stream: int = 0,
            h: Optional[np.ndarray] = None, a_prev: int = 0x8000, b_prev: int = 0x8000,
            a_forced: Optional[np.ndarray] = None, b_forced: Optional[np.ndarray] = None, dump: bool = False) -> Fs2Result:
        H = self.H
        n_frames = 0
        if self.cond_dim:
            cond = np.ascontiguousarray(cond, dtype=np.float32).reshape(-1, self.cond_dim)
            n_frames = cond.shape[0]
        else:
            cond = None
        hh = np.zeros(H, np.float32) if h is None else np.array(h, np.float32, copy=True).reshape(H)
        ap = np.array([a_prev], np.uint16)
        bp = np.array([b_prev], np.uint16)
        if a_forced is not None:
            a_forced = np.ascontiguousarray(a_forced, np.uint16).reshape(n_steps)
            b_forced = np.ascontiguousarray(b_forced, np.uint16).reshape(n_steps)
        out = np.zeros((2, n_steps), np.int16)
        a_out = np.zeros(n_steps, np.uint16)
        b_out = np.zeros(n_steps, np.uint16)
        margins = np.zeros((n_steps, 8), np.float64)
        gates = hs = logits = None
        if dump:
            gates = np.zeros((n_steps, 3 * H), np.float32)
            hs = np.zeros((n_steps, H), np.float32)
            logits = np.zeros((n_steps, 2, 64), np.float32)
        rc = lib().orc_fs2_run(C.byref(self._p), _ptr(cond), n_frames, hop, n_steps, step0, seed, stream, _ptr(hh), _ptr(ap), _ptr(bp),
                               _ptr(a_forced), _ptr(b_forced), _ptr(a_out), _ptr(b_out), _ptr(out), _ptr(margins),
                               _ptr(gates), _ptr(hs), _ptr(logits))
        if rc != 0:
            raise ValueError("conditioning frame index out of range")
        return Fs2Result(out, a_out, b_out, margins, hh, int(ap[0]), int(bp[0]), gates, hs, logits)


# ----------------------------------------------------------------------------------------------
# Subscale generation with dependent rows (Section 4.1 ordering, Section 4.2 future horizon)
#
# What the paper fixes: sub-tensor s (samples u_{B i + s}) is generated after sub-tensors z < s and is conditioned on
# their past and on their future up to a horizon of F positions, through a conditioning network whose mask removes the
# past connections; the WaveRNN itself is shared by all sub-tensors.  The network used here is a stated reading (one
# masked convolution layer instead of the paper's ten, synthetic weights; parity for it is unpinned outside this file):
#     v_s[i] = frame_s[(B i + s) div hop] + relu(b + sum_{delta=1..s} sum_{d=0..F} V[delta-1][d] . x(u_{s-delta}[i+d]))
# with x(u) = u / 32768 for the int16 sample u, positions at or beyond the row length contributing nothing; row s is
# an ordinary WaveRNN stream (Philox stream id s, step = position) whose conditioning vector at step i is v_s[i].

def subscale_conditioning(history: np.ndarray, s: int, V: np.ndarray, b: np.ndarray) -> np.ndarray:
    """The convolution term of v_s for all positions: history int16 [B][L] (rows < s must be complete), V [B-1][F+1][D],
    b [D] -> float32 [L][D].  Plain double loops over (delta, d); row 0 has no earlier row: relu(b)."""
    B, L = history.shape
    F1, D = V.shape[1], V.shape[2]
    acc = np.tile(b.astype(np.float64), (L, 1))
    for delta in range(1, s + 1):
        x = history[s - delta].astype(np.float64) / 32768.0
        for d in range(F1):
            n = L - d
            if n <= 0:
                break
            acc[:n] += np.outer(x[d:], V[delta - 1, d].astype(np.float64))
    return np.maximum(acc, 0.0).astype(np.float32)


def subscale_dependent_run(om: "OracleModel", frames: np.ndarray, V: np.ndarray, b: np.ndarray, B: int, L: int, hop: int,
                           seed: int, forced: Optional[np.ndarray] = None, teacher: bool = False):
    """Generate the B sub-tensors one after the other (the order of Eq. 4).  frames: float32 [B][n_frames][D] (row s,
    frame (B i + s) div hop at position i).  forced: optional int16 [B][L]; when given, row s is conditioned on the
    forced samples of rows < s (the drawn ones are still returned); with teacher = True the forced samples of row s
    itself are fed back inside the row as well, so that every returned sample is the oracle's draw given the forced
    history up to that point.  -> (samples int16 [B][L], cond float32 [B][L][D], margins [B][L][2])."""
    D = om.cond_dim
    out = np.zeros((B, L), np.int16)
    cond = np.zeros((B, L, D), np.float32)
    margins = np.zeros((B, L, 2), np.float64)
    for s in range(B):
        hist = out if forced is None else forced
        idx = (B * np.arange(L) + s) // hop
        cond[s] = frames[s][idx] + (subscale_conditioning(hist, s, V, b) if s > 0 else np.maximum(b, 0.0).astype(np.float32)[None, :])
        if teacher and forced is not None:
            cf, ff = split_samples(forced[s])
            r = om.run(cond[s][None], L, 1, seed, hop=1, stream0=s, c_forced=cf, f_forced=ff)
            out[s] = join_samples(r.c_out[0], r.f_out[0])
        else:
            r = om.run(cond[s][None], L, 1, seed, hop=1, stream0=s)
            out[s] = r.out[0]
        margins[s] = r.margins[0]
    return out, cond, margins
