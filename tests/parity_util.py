"""Helpers for the GPU-vs-oracle parity tests (comparison rules and plumbing)."""
from __future__ import annotations

import os

import numpy as np

from oracle import wrnn_oracle as orc

TOL = {"f32": 1e-4, "bf16": 2e-3}   # relative, per vector, see rel_err
MARGIN = 1e-5                       # draws whose uniform lies this close to a CDF boundary may differ
NCPU = max(1, min(os.cpu_count() or 1, 32))


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max_i |gpu_i - ref_i| / max(|ref_i|, rms(ref)) with the rms taken per vector (last axis)."""
    g = gpu.astype(np.float64)
    r = ref.astype(np.float64)
    rms = np.sqrt((r * r).mean(axis=-1, keepdims=True))
    den = np.maximum(np.abs(r), np.maximum(rms, 1e-30))
    return float((np.abs(g - r) / den).max())


def check_indices(gpu_idx: np.ndarray, ref_idx: np.ndarray, margins: np.ndarray):
    """Bit-exact except near-boundary draws.  -> (number of differing draws, all of them near a boundary)."""
    diff = gpu_idx != ref_idx
    bad = diff & (margins >= MARGIN)
    return int(diff.sum()), int(bad.sum())


def teacher_forced_parity(torch, B, model, om, cond_np, n_steps, batch, seed, *, hop=120, row_stride=1,
                          row_offset_mul=0, stream0=0, threads=1, dump=True, oracle_free=None):
    """Oracle free-runs (or oracle_free is given); the GPU is teacher-forced on that stream.
    Returns a dict of error figures."""
    res = oracle_free if oracle_free is not None else om.run(
        cond_np, n_steps, batch, seed, hop=hop, row_stride=row_stride, row_offset_mul=row_offset_mul,
        stream0=stream0, dump=dump, threads=threads)
    dev = "cuda:0"
    cond = None if cond_np is None else torch.from_numpy(cond_np).to(dev)
    cf = torch.from_numpy(res.c_out).to(dev)
    ff = torch.from_numpy(res.f_out).to(dev)
    co = torch.zeros_like(cf)
    fo = torch.zeros_like(ff)
    H = om.H
    gates = hs = logits = None
    if dump:
        gates = torch.zeros((n_steps, batch, 3 * H), dtype=torch.float32, device=dev)
        hs = torch.zeros((n_steps, batch, H), dtype=torch.float32, device=dev)
        logits = torch.zeros((n_steps, batch, 2, 256), dtype=torch.float32, device=dev)
    hfin = torch.zeros((batch, H), dtype=torch.float32, device=dev)
    cp = torch.full((batch,), 128, dtype=torch.uint8, device=dev)
    fp = torch.zeros((batch,), dtype=torch.uint8, device=dev)
    B.wrnn_step_teacher_forced(model, cond, n_steps, batch, seed, cf, ff, co, fo, dbg_gates=gates, dbg_h=hs,
                               dbg_logits=logits, hop=hop, row_stride=row_stride, row_offset_mul=row_offset_mul,
                               h=hfin, c_prev=cp, f_prev=fp, stream0=stream0)
    torch.cuda.synchronize()
    assert B.wrnn_poll_status(model) == 0, B.wrnn_last_error(model)
    out = {}
    nd_c, bad_c = check_indices(co.cpu().numpy(), res.c_out, res.margins[:, :, 0])
    nd_f, bad_f = check_indices(fo.cpu().numpy(), res.f_out, res.margins[:, :, 1])
    out["idx_diff"] = nd_c + nd_f
    out["idx_bad"] = bad_c + bad_f
    out["near_boundary"] = int((res.margins < MARGIN).sum())
    out["h_final_err"] = rel_err(hfin.cpu().numpy(), res.h)
    assert np.array_equal(cp.cpu().numpy(), res.c_out[:, -1]) and np.array_equal(fp.cpu().numpy(), res.f_out[:, -1])
    if dump:
        out["gates_err"] = rel_err(gates.cpu().numpy(), res.gates)
        out["h_err"] = rel_err(hs.cpu().numpy(), res.hs)
        out["logits_err"] = rel_err(logits.cpu().numpy(), res.logits)
    out["oracle"] = res
    return out


def first_divergence(a: np.ndarray, b: np.ndarray) -> int:
    """Index of the first differing sample along the last axis (any row); -1 if none."""
    d = np.nonzero((a != b).any(axis=0))[0] if a.ndim == 2 else np.nonzero(a != b)[0]
    return int(d[0]) if d.size else -1


def oracle_on_gpu_stream(om, cond_np, rows, gpu_out, seed, *, hop=120, row_stride=1, row_offset_mul=0, stream0=0,
                         h_final=None):
    """The oracle teacher-forced on the samples the GPU itself generated, one stream row at a time: at every step the
    oracle sees the GPU's history and reports what it would draw, so every draw of the chosen rows is compared (a
    free-run comparison alone stops at a row's first near-boundary draw).  rows index gpu_out's first axis (row b has
    the global row id stream0 + b); cond_np is [batch][n_frames][D] or None.  -> dict of counts and the worst
    final-state error (h_final = the GPU's [batch][H] final state, optional)."""
    from concurrent.futures import ThreadPoolExecutor

    n = gpu_out.shape[1]

    def one(b):
        cf, ff = _split(gpu_out[b])
        r = om.run(None if cond_np is None else cond_np[b:b + 1], n, 1, seed, hop=hop, row_stride=row_stride,
                   row_offset_mul=row_offset_mul, stream0=stream0 + b, c_forced=cf, f_forced=ff)
        nd_c, bad_c = check_indices(cf, r.c_out[0], r.margins[0, :, 0])
        nd_f, bad_f = check_indices(ff, r.f_out[0], r.margins[0, :, 1])
        herr = rel_err(h_final[b], r.h[0]) if h_final is not None else 0.0
        return nd_c + nd_f, bad_c + bad_f, int((r.margins[0] < MARGIN).sum()), herr

    with ThreadPoolExecutor(max_workers=NCPU) as ex:
        res = list(ex.map(one, rows))
    return {"rows": list(rows), "draws": 2 * n * len(res), "idx_diff": sum(r[0] for r in res), "idx_bad": sum(r[1] for r in res),
            "near_boundary": sum(r[2] for r in res), "h_final_err": max(r[3] for r in res)}


def _split(x):
    """int16 samples -> the (coarse, fine) bytes the device emitted them from (plumbing for the forced arrays)."""
    u = (x.astype(np.int32) + 32768).astype(np.uint16)
    return (u >> 8).astype(np.uint8), (u & 255).astype(np.uint8)
