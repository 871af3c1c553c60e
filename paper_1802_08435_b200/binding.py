"""Python binding of libwrnn.so: the same entry points as include/wrnn.h.

Argument marshalling only.  Device buffers are torch CUDA tensors (torch is used for
device memory and streams, nothing else); every step of the sampling path runs in
the library's CUDA kernels.  There is no CPU path: if the library has not been built
the import of any entry point raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwrnn.so")

WRNN_OK, WRNN_ERR_INVALID_ARG, WRNN_ERR_UNSUPPORTED, WRNN_ERR_NOMEM, WRNN_ERR_CUDA, WRNN_ERR_TIMEOUT, WRNN_ERR_CHECK = range(7)
WRNN_F32, WRNN_BF16 = 0, 1
WRNN_KERNEL_AUTO, WRNN_KERNEL_GENERIC, WRNN_KERNEL_RESIDENT, WRNN_KERNEL_BATCHED, WRNN_KERNEL_SPARSE = 0, 1, 2, 3, 4
WRNN_KERNEL_BCLUSTER = 5
_STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "NOMEM", "CUDA", "TIMEOUT", "CHECK"]

EXPORTS = [
    "wrnn_create", "wrnn_destroy", "wrnn_sample", "wrnn_step_teacher_forced", "wrnn_fold", "wrnn_unfold",
    "wrnn_sample_subscale", "wrnn_sample_host", "wrnn_poll_status", "wrnn_last_error", "wrnn_launch_info",
    "wrnn_launch_count", "wrnn_phase_cycles", "wrnn_phase_profile", "wrnn_phase_names", "wrnn_measure_exchange_floor", "wrnn_measure_smem_stream", "wrnn_sample_noalloc",
    "wrnn_selftest_bounded_wait", "wrnn_selftest_lost_word", "wrnn_fs2_sample", "wrnn_fs2_step_teacher_forced", "wrnn_fs2_unfold", "wrnn_fs2_sample_host",
    "wrnn_sample_subscale_dependent", "wrnn_subscale_conditioning", "wrnn_subscale_schedule",
    "wrnn_subscale_net_create", "wrnn_subscale_net_destroy", "wrnn_subscale_net_conditioning", "wrnn_subscale_net_status", "wrnn_sample_subscale_net", "wrnn_subscale_net_rows",
]


class WrnnError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("wrnn status %d (%s): %s" % (code, _STATUS_NAMES[code] if 0 <= code < 7 else "?", msg))
        self.code = code


class wrnn_params(C.Structure):
    _fields_ = (
        [("H", C.c_int32), ("cond_dim", C.c_int32)]
        + [(n, C.c_void_p) for n in ("R", "I", "b_gate", "W_cond", "O1", "b1", "O2", "b2", "O3", "b3", "O4", "b4",
                                     "mask_R", "mask_O1", "mask_O3")]
        + [("dtype", C.c_int32), ("kernel", C.c_int32), ("mask_block_rows", C.c_int32), ("mask_block_cols", C.c_int32),
           ("variant", C.c_int32)]
    )


class wrnn_state(C.Structure):
    _fields_ = [("h", C.c_void_p), ("c_prev", C.c_void_p), ("f_prev", C.c_void_p), ("step0", C.c_int64),
                ("stream0", C.c_uint32), ("reserved", C.c_uint32)]


class wrnn_fs2_state(C.Structure):
    _fields_ = [("h", C.c_void_p), ("a_prev", C.c_void_p), ("b_prev", C.c_void_p), ("step0", C.c_int64),
                ("stream0", C.c_uint32), ("reserved", C.c_uint32)]


class wrnn_cond(C.Structure):
    _fields_ = [("cond", C.c_void_p), ("n_frames", C.c_int32), ("hop", C.c_int32), ("row_stride", C.c_int32),
                ("row_offset_mul", C.c_int32)]


_lib = None


def lib():
    """Load libwrnn.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libwrnn.so is missing: build it with `python -m paper_1802_08435_b200.build` "
                "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        L.wrnn_create.argtypes = [C.POINTER(wrnn_params), i32, C.POINTER(vp)]
        L.wrnn_destroy.argtypes = [vp]
        L.wrnn_destroy.restype = None
        L.wrnn_sample.argtypes = [vp, C.POINTER(wrnn_cond), i64, i32, u64, C.POINTER(wrnn_state), vp, vp]
        L.wrnn_sample_noalloc.argtypes = [vp, C.POINTER(wrnn_cond), i64, i32, u64, C.POINTER(wrnn_state), vp, vp]
        L.wrnn_step_teacher_forced.argtypes = [vp, C.POINTER(wrnn_cond), i64, i32, u64, C.POINTER(wrnn_state)] + [vp] * 8
        L.wrnn_fs2_sample.argtypes = [vp, C.POINTER(wrnn_cond), i64, u64, C.POINTER(wrnn_fs2_state), vp, vp]
        L.wrnn_fs2_step_teacher_forced.argtypes = [vp, C.POINTER(wrnn_cond), i64, u64, C.POINTER(wrnn_fs2_state)] + [vp] * 8
        L.wrnn_fs2_unfold.argtypes = [vp, i64, vp, vp]
        L.wrnn_fs2_sample_host.argtypes = [vp, vp, i32, i32, i64, u64, vp]
        L.wrnn_sample_subscale_dependent.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i64, i32, u64, vp, vp]
        L.wrnn_subscale_schedule.argtypes = [i32, i64, i32, i32, vp, i32]
        L.wrnn_subscale_conditioning.argtypes = [vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, i32, vp, vp]
        L.wrnn_fold.argtypes = [vp, i64, i32, vp, vp]
        L.wrnn_unfold.argtypes = [vp, i64, i32, vp, vp]
        L.wrnn_sample_subscale.argtypes = [vp, vp, i32, i32, i64, i32, u64, vp, vp]
        L.wrnn_sample_host.argtypes = [vp, vp, i32, i32, i32, i32, i64, i32, u64, vp]
        L.wrnn_poll_status.argtypes = [vp]
        L.wrnn_last_error.argtypes = [vp]
        L.wrnn_last_error.restype = C.c_char_p
        L.wrnn_launch_info.argtypes = [vp, i32] + [vp] * 5
        L.wrnn_phase_cycles.argtypes = [vp, vp]
        L.wrnn_phase_profile.argtypes = [vp, i32]
        L.wrnn_phase_names.argtypes = [vp, vp, i32]
        L.wrnn_measure_exchange_floor.argtypes = [i32, i32, i32, i32, vp]
        L.wrnn_measure_smem_stream.argtypes = [i32, i32, i32, i32, vp]
        L.wrnn_selftest_bounded_wait.argtypes = [i64] + [vp] * 5
        L.wrnn_selftest_lost_word.argtypes = [vp, i64, i32, i64]
        L.wrnn_subscale_net_create.argtypes = [vp, vp]
        L.wrnn_subscale_net_destroy.argtypes = [vp]
        L.wrnn_subscale_net_destroy.restype = None
        L.wrnn_subscale_net_conditioning.argtypes = [vp, vp, vp, i32, i32, i32, i64, vp, vp]
        L.wrnn_subscale_net_status.argtypes = [vp]
        L.wrnn_sample_subscale_net.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i64, C.c_uint64, vp, vp]
        L.wrnn_subscale_net_rows.argtypes = [vp, vp, vp, i32, i32, i32, vp, i64, vp, vp, vp, i32, i32, i64, i32, C.c_uint64, vp]
        L.wrnn_launch_count.argtypes = []
        L.wrnn_launch_count.restype = i64
        _lib = L
    return _lib


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t):
    """Device pointer of a contiguous torch CUDA tensor (or None)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device buffers must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(rc: int, model=None):
    if rc != WRNN_OK:
        msg = lib().wrnn_last_error(model)
        raise WrnnError(rc, msg.decode() if msg else "")


def wrnn_last_error(model=None) -> str:
    msg = lib().wrnn_last_error(model)
    return msg.decode() if msg else ""


def wrnn_create(weights: Dict[str, np.ndarray], dtype: str = "f32", masks: Optional[Dict[str, np.ndarray]] = None,
                max_batch: int = 1, kernel: int = WRNN_KERNEL_AUTO, block=(4, 4), variant: int = 0):
    """weights: fp32 numpy arrays R [3H][H], I [3H][3], W_cond [3H][D] or None, O1..O4, b_gate, b1..b4 (or None);
    masks: optional block masks {"R": [3H/br][H/bc], "O1": [H/2/br][H/2/bc], "O3": ...} with block = (br, bc).
    variant = 1: Fused Subscale WaveRNN 2x (I [3H][12], O2 / O4 [64][H/2], b2 / b4 [64]).
    Returns an opaque handle."""
    keep = {}

    def f32(k):
        a = weights.get(k)
        if a is None:
            return None
        keep[k] = np.ascontiguousarray(a, dtype=np.float32)
        return keep[k]

    def u8(k):
        a = None if masks is None else masks.get(k)
        if a is None:
            return None
        keep["m" + k] = np.ascontiguousarray(a, dtype=np.uint8)
        return keep["m" + k]

    R = f32("R")
    H = R.shape[1]
    Wc = f32("W_cond")
    p = wrnn_params()
    p.H = H
    p.cond_dim = 0 if Wc is None else Wc.shape[1]
    for k in ("R", "I", "b_gate", "W_cond", "O1", "b1", "O2", "b2", "O3", "b3", "O4", "b4"):
        setattr(p, k, _np_ptr(f32(k)))
    p.mask_R, p.mask_O1, p.mask_O3 = _np_ptr(u8("R")), _np_ptr(u8("O1")), _np_ptr(u8("O3"))
    p.dtype = {"f32": WRNN_F32, "bf16": WRNN_BF16}[dtype]
    p.kernel = kernel
    p.mask_block_rows, p.mask_block_cols = int(block[0]), int(block[1])
    p.variant = int(variant)
    out = C.c_void_p()
    _check(lib().wrnn_create(C.byref(p), max_batch, C.byref(out)))
    return out


def wrnn_destroy(model):
    lib().wrnn_destroy(model)


def _mk_cond(cond, hop, row_stride, row_offset_mul):
    if cond is None:
        return None
    c = wrnn_cond(_dev_ptr(cond), int(cond.shape[1]), hop, row_stride, row_offset_mul)
    return C.byref(c)


def _mk_state(h, c_prev, f_prev, step0, stream0):
    if h is None and c_prev is None and f_prev is None and step0 == 0 and stream0 == 0:
        return None
    return C.byref(wrnn_state(_dev_ptr(h), _dev_ptr(c_prev), _dev_ptr(f_prev), step0, stream0, 0))


def wrnn_sample(model, cond, n_steps: int, batch: int, seed: int, out, *, hop: int = 120, row_stride: int = 1,
                row_offset_mul: int = 0, h=None, c_prev=None, f_prev=None, step0: int = 0, stream0: int = 0,
                stream=None):
    """cond: CUDA float32 [batch][n_frames][cond_dim] or None; out: CUDA int16 [batch][n_steps]."""
    _check(lib().wrnn_sample(model, _mk_cond(cond, hop, row_stride, row_offset_mul), n_steps, batch, seed,
                             _mk_state(h, c_prev, f_prev, step0, stream0), _dev_ptr(out), _stream_ptr(stream)), model)


def wrnn_step_teacher_forced(model, cond, n_steps: int, batch: int, seed: int, c_forced, f_forced, c_out, f_out, *,
                             dbg_gates=None, dbg_h=None, dbg_logits=None, hop: int = 120, row_stride: int = 1,
                             row_offset_mul: int = 0, h=None, c_prev=None, f_prev=None, step0: int = 0,
                             stream0: int = 0, stream=None):
    _check(lib().wrnn_step_teacher_forced(
        model, _mk_cond(cond, hop, row_stride, row_offset_mul), n_steps, batch, seed,
        _mk_state(h, c_prev, f_prev, step0, stream0), _dev_ptr(c_forced), _dev_ptr(f_forced), _dev_ptr(c_out),
        _dev_ptr(f_out), _dev_ptr(dbg_gates), _dev_ptr(dbg_h), _dev_ptr(dbg_logits), _stream_ptr(stream)), model)


def wrnn_fold(x, B: int, sub, stream=None):
    _check(lib().wrnn_fold(_dev_ptr(x), x.numel(), B, _dev_ptr(sub), _stream_ptr(stream)))


def wrnn_unfold(sub, B: int, x, stream=None):
    _check(lib().wrnn_unfold(_dev_ptr(sub), sub.numel(), B, _dev_ptr(x), _stream_ptr(stream)))


def _mk_fs2_state(h, a_prev, b_prev, step0, stream0):
    if h is None and a_prev is None and b_prev is None and step0 == 0 and stream0 == 0:
        return None
    return C.byref(wrnn_fs2_state(_dev_ptr(h), _dev_ptr(a_prev), _dev_ptr(b_prev), step0, stream0, 0))


def wrnn_fs2_sample(model, cond, n_steps: int, seed: int, out, *, hop: int = 120, h=None, a_prev=None, b_prev=None,
                    step0: int = 0, stream0: int = 0, stream=None):
    """Fused Subscale WaveRNN 2x.  cond: CUDA float32 [1][n_frames][cond_dim] or None; out: CUDA int16 [2][n_steps]
    (row 0: a_t, row 1: the sample part B emitted in step t); a_prev / b_prev: CUDA uint16 [1] carry state."""
    _check(lib().wrnn_fs2_sample(model, _mk_cond(cond, hop, 1, 0), n_steps, seed, _mk_fs2_state(h, a_prev, b_prev, step0, stream0),
                                 _dev_ptr(out), _stream_ptr(stream)), model)


def wrnn_fs2_step_teacher_forced(model, cond, n_steps: int, seed: int, a_forced, b_forced, a_out, b_out, *, dbg_gates=None,
                                 dbg_h=None, dbg_logits=None, hop: int = 120, h=None, a_prev=None, b_prev=None,
                                 step0: int = 0, stream0: int = 0, stream=None):
    _check(lib().wrnn_fs2_step_teacher_forced(
        model, _mk_cond(cond, hop, 1, 0), n_steps, seed, _mk_fs2_state(h, a_prev, b_prev, step0, stream0),
        _dev_ptr(a_forced), _dev_ptr(b_forced), _dev_ptr(a_out), _dev_ptr(b_out), _dev_ptr(dbg_gates), _dev_ptr(dbg_h),
        _dev_ptr(dbg_logits), _stream_ptr(stream)), model)


def wrnn_fs2_unfold(ab, n_steps: int, u, stream=None):
    """ab: CUDA int16 [2][n_steps] from wrnn_fs2_sample; u: CUDA int16 [2 (n_steps - 2)]."""
    _check(lib().wrnn_fs2_unfold(_dev_ptr(ab), n_steps, _dev_ptr(u), _stream_ptr(stream)))


def wrnn_sample_subscale_dependent(model, frames, V, bias, F: int, chunk: int, lag: int, n_total: int, B: int, seed: int, out, *,
                                   hop: int = 120, stream=None):
    """Subscale generation with dependent rows on the staggered schedule.  frames: CUDA float32 [B][n_frames][D];
    V: CUDA float32 [B-1][F+1][D]; bias: CUDA float32 [D]; out: CUDA int16 [n_total] in the original order."""
    _check(lib().wrnn_sample_subscale_dependent(model, _dev_ptr(frames), int(frames.shape[1]), hop, _dev_ptr(V), _dev_ptr(bias), F,
                                                chunk, lag, n_total, B, seed, _dev_ptr(out), _stream_ptr(stream)), model)


class wrnn_subscale_net_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "n_layers", "taps", "conv_ch", "res_ch", "cond_dim")] + \
               [(n, C.c_void_p) for n in ("dilation", "W_in", "b_in", "W_conv", "b_conv", "W_res", "b_res", "W_out", "b_out")]


def wrnn_subscale_net_create(w: Dict[str, np.ndarray]):
    """The conditioning network of the Subscale WaveRNN from a dict of fp32 numpy arrays: dilation int32 [layers], W_in
    [res][B], b_in, W_conv [layers][taps][conv][res], b_conv, W_res [layers][res][conv], b_res, W_out [D][res], b_out.
    Returns an opaque handle."""
    keep = {k: np.ascontiguousarray(w[k], dtype=np.int32 if k == "dilation" else np.float32) for k in
            ("dilation", "W_in", "b_in", "W_conv", "b_conv", "W_res", "b_res", "W_out", "b_out")}
    nl, taps, conv, res = keep["W_conv"].shape
    p = wrnn_subscale_net_params(int(keep["W_in"].shape[1]), int(nl), int(taps), int(conv), int(res), int(keep["W_out"].shape[0]),
                                 *[_np_ptr(keep[k]) for k in ("dilation", "W_in", "b_in", "W_conv", "b_conv", "W_res", "b_res", "W_out", "b_out")])
    out = C.c_void_p()
    _check(lib().wrnn_subscale_net_create(C.byref(p), C.byref(out)))
    return out


def wrnn_subscale_net_destroy(net) -> None:
    lib().wrnn_subscale_net_destroy(net)


def wrnn_subscale_net_conditioning(net, hist, frames, row: int, v, *, hop: int = 120, stream=None):
    """v (CUDA float32 [L][D]) = conditioning vectors of sub-tensor `row` from the history hist (CUDA int16 [B][L])."""
    _check(lib().wrnn_subscale_net_conditioning(net, _dev_ptr(hist), _dev_ptr(frames), int(frames.shape[1]), hop, row, int(hist.shape[1]),
                                                _dev_ptr(v), _stream_ptr(stream)))


def wrnn_subscale_net_status(net) -> int:
    return lib().wrnn_subscale_net_status(net)


def wrnn_sample_subscale_net(model, net, frames, F: int, chunk: int, lag: int, n_total: int, seed: int, out, *, hop: int = 120, stream=None):
    """Subscale generation with dependent rows on the staggered schedule, conditioned through the masked dilated network.
    frames: CUDA float32 [B][n_frames][D]; out: CUDA int16 [n_total] in the original order."""
    _check(lib().wrnn_sample_subscale_net(model, net, _dev_ptr(frames), int(frames.shape[1]), hop, F, chunk, lag, n_total, seed, _dev_ptr(out),
                                          _stream_ptr(stream)), model)


def wrnn_subscale_net_rows(model, net, frames, lag: int, hist, h, c_prev, f_prev, r_lo: int, n_rows: int, p_lo: int, n_steps: int, seed: int, *,
                           hop: int = 120, stream=None):
    """One stepping call of the staggered schedule on caller-owned CUDA buffers: hist int16 [B][L] (in / out), h float32 [B][H],
    c_prev / f_prev uint8 [B] (carry state of all rows); rows r_lo .. r_lo + n_rows - 1, row b from position p_lo - b * lag on."""
    _check(lib().wrnn_subscale_net_rows(model, net, _dev_ptr(frames), int(frames.shape[1]), hop, lag, _dev_ptr(hist), int(hist.shape[1]), _dev_ptr(h),
                                        _dev_ptr(c_prev), _dev_ptr(f_prev), r_lo, n_rows, p_lo, n_steps, seed, _stream_ptr(stream)), model)


def wrnn_subscale_schedule(B: int, L: int, chunk: int, lag: int):
    """The stepping launches of the staggered schedule as a list of (first row, rows, position of the first row, steps).
    Host arithmetic only: works without a GPU."""
    n = lib().wrnn_subscale_schedule(B, L, chunk, lag, None, 0)
    if n < 0:
        raise WrnnError(-n, "bad schedule arguments")
    buf = (C.c_int64 * (4 * max(n, 1)))()
    lib().wrnn_subscale_schedule(B, L, chunk, lag, buf, n)
    return [tuple(buf[4 * i: 4 * i + 4]) for i in range(n)]


def wrnn_subscale_conditioning(hist, frames, V, bias, F: int, row: int, v, *, hop: int = 120, stream=None):
    """v (CUDA float32 [L][D]) = conditioning vectors of sub-tensor `row` from the history hist (CUDA int16 [B][L])."""
    B, L = int(hist.shape[0]), int(hist.shape[1])
    _check(lib().wrnn_subscale_conditioning(_dev_ptr(hist), _dev_ptr(frames), _dev_ptr(V), _dev_ptr(bias), B, L, F, int(frames.shape[2]),
                                            int(frames.shape[1]), hop, row, _dev_ptr(v), _stream_ptr(stream)))


def wrnn_fs2_sample_host(model, cond_host: Optional[np.ndarray], n_steps: int, seed: int, u_host: np.ndarray, *, hop: int = 120):
    """Host buffers in and out: cond_host [n_frames][cond_dim] float32, u_host int16 [2 (n_steps - 2)]; synchronous."""
    n_frames = 0 if cond_host is None else int(cond_host.shape[-2])
    assert u_host.dtype == np.int16 and u_host.flags.c_contiguous and u_host.size >= 2 * max(n_steps - 2, 0)
    _check(lib().wrnn_fs2_sample_host(model, _np_ptr(cond_host), n_frames, hop, n_steps, seed, _np_ptr(u_host)), model)


def wrnn_sample_subscale(model, cond, n_total: int, B: int, seed: int, out, *, hop: int = 120, stream=None):
    _check(lib().wrnn_sample_subscale(model, _dev_ptr(cond), int(cond.shape[1]), hop, n_total, B, seed, _dev_ptr(out),
                                      _stream_ptr(stream)), model)


def wrnn_sample_host(model, cond_host: Optional[np.ndarray], n_steps: int, batch: int, seed: int,
                     out_host: np.ndarray, *, hop: int = 120, row_stride: int = 1, row_offset_mul: int = 0):
    """Host buffers in and out (numpy, ideally backed by pinned memory); synchronous."""
    n_frames = 0 if cond_host is None else int(cond_host.shape[1])
    assert out_host.dtype == np.int16 and out_host.flags.c_contiguous
    _check(lib().wrnn_sample_host(model, _np_ptr(cond_host), n_frames, hop, row_stride, row_offset_mul, n_steps, batch,
                                  seed, _np_ptr(out_host)), model)


def wrnn_poll_status(model) -> int:
    return lib().wrnn_poll_status(model)


def wrnn_launch_info(model, batch: int = 1) -> dict:
    k, n, t, s = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    w = C.c_int64()
    _check(lib().wrnn_launch_info(model, batch, C.byref(k), C.byref(n), C.byref(t), C.byref(w), C.byref(s)), model)
    return dict(kernel=k.value, n_ctas=n.value, n_threads=t.value, weight_bytes_per_step=w.value, smem_bytes=s.value)


def wrnn_launch_count() -> int:
    return lib().wrnn_launch_count()


def wrnn_phase_profile(model, enable: bool) -> None:
    """Switch the phase stamps of the resident kernels on or off (off by default: they cost cycles on the critical warp)."""
    _check(lib().wrnn_phase_profile(model, 1 if enable else 0), model)


def wrnn_phase_names(model):
    """Names of the sixteen phase slots of the last profiled call."""
    buf = C.create_string_buffer(1024)
    _check(lib().wrnn_phase_names(model, buf, 1024), model)
    return buf.value.decode().split(",")


def wrnn_phase_cycles(model):
    """SM-clock cycles CTA 0 spent per phase of the resident kernel over the last call (list of 12)."""
    buf = (C.c_int64 * 16)()
    _check(lib().wrnn_phase_cycles(model, buf), model)
    return list(buf)


def wrnn_measure_exchange_floor(n_ctas: int, n_threads: int, K: int, iters: int = 20000) -> float:
    """Nanoseconds per chip-wide all-gather of K tagged values through L2 (empty persistent kernel)."""
    out = C.c_float()
    _check(lib().wrnn_measure_exchange_floor(n_ctas, n_threads, K, iters, C.byref(out)))
    return out.value


def wrnn_measure_smem_stream(n_ctas: int, n_threads: int, bytes_per_cta: int, iters: int = 2000) -> float:
    """Aggregate GB/s of 16-byte shared-memory loads over a resident buffer on n_ctas CTAs (stream micro-benchmark)."""
    out = C.c_float()
    _check(lib().wrnn_measure_smem_stream(n_ctas, n_threads, bytes_per_cta, iters, C.byref(out)))
    return out.value


def wrnn_selftest_bounded_wait(limit_ns: int = 50_000_000) -> dict:
    """Run the bounded-wait self-test; returns the device status word, where it was recorded and the kernel time."""
    code, cta, step, phase, ms = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32(), C.c_float()
    _check(lib().wrnn_selftest_bounded_wait(limit_ns, C.byref(code), C.byref(cta), C.byref(step), C.byref(phase), C.byref(ms)))
    return {"code": code.value, "cta": cta.value, "step": step.value, "phase": phase.value, "waited_ms": ms.value}


def wrnn_selftest_lost_word(model, limit_ns: int = 0, cta: int = -1, step: int = -1) -> None:
    """From the next launch on: CTA `cta` withholds at `step` what it hands to the other CTAs and every device-side wait
    is bounded by limit_ns (0 = default); cta = -1 restores normal operation."""
    _check(lib().wrnn_selftest_lost_word(model, limit_ns, cta, step), model)


def wrnn_sample_noalloc(model, cond, n_steps: int, batch: int, seed: int, out, *, hop: int = 120, row_stride: int = 1,
                        row_offset_mul: int = 0, h=None, c_prev=None, f_prev=None, step0: int = 0, stream0: int = 0,
                        stream=None):
    """Same arguments and samples as wrnn_sample, for callers that cannot allocate device memory at run time
    (real-time threads, allocation-free regions, fixed memory budgets): all scratch sits in a fixed 8 MiB array
    of the library image; requests that do not fit raise WrnnError(UNSUPPORTED).  Calls share that array, so
    they must not overlap on the GPU."""
    _check(lib().wrnn_sample_noalloc(model, _mk_cond(cond, hop, row_stride, row_offset_mul), n_steps, batch, seed,
                                     _mk_state(h, c_prev, f_prev, step0, stream0), _dev_ptr(out), _stream_ptr(stream)),
           model)
