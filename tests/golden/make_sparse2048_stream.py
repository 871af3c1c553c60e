#!/usr/bin/env python
"""Writes tests/golden/sparse2048_bf16_b1_24000_oracle.npz: the CPU oracle's own 24,000-step free run of the
block-sparse H = 2048 workload (Section 3.2: 4 x 4 blocks, 96 % pruned; the sparse model is the dense equations of
Eq. 2 on the masked matrices).

The dense-with-zeros oracle needs about 15 ms per step at this width, six minutes for the whole second of audio, so
its stream is stored once instead of being recomputed by every GPU test run.  This script calls only the seeded input
generator and `oracle/`; nothing in the file comes from the CUDA path.  Stored:

  c_out, f_out   uint8 [24000]   the symbols the oracle drew (the stream the GPU is teacher-forced on)
  nb_index       int32 [k]       flat indices into [24000][2] (step, head) of the draws whose uniform lies within 1e-4
  nb_margin      float64 [k]     of a CDF boundary, and that distance (every other draw is further away)
  snap_steps     int32 [24]      steps 999, 1999, ... whose vectors are kept
  snap_h         float32 [24][2048], snap_logits float32 [24][2][256]
  snap_gates_steps int32 [6]     steps 3999, 7999, ... and snap_gates float32 [6][6144], the gate vectors there
  h_final        float32 [2048]
  inputs_sha256  hex digest of the weights, masks and conditioning frames the run used (a test refuses a file that
                 does not belong to the current input generator)

Run from the repository root:  python tests/golden/make_sparse2048_stream.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import wrnn_oracle as orc  # noqa: E402
from paper_1802_08435_b200 import synth  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sparse2048_bf16_b1_24000_oracle.npz")
CHUNK = 1000
NB_STORE = 1e-4


def inputs_digest(w, masks, cond) -> str:
    h = hashlib.sha256()
    for k in sorted(w):
        if w[k] is not None:
            h.update(k.encode())
            h.update(np.ascontiguousarray(w[k]).tobytes())
    for k in sorted(masks):
        h.update(k.encode())
        h.update(np.ascontiguousarray(masks[k]).tobytes())
    h.update(np.ascontiguousarray(cond).tobytes())
    return h.hexdigest()


def main():
    wl = synth.WORKLOADS[2]
    assert wl.name == "sparse2048_bf16_b1_24000"
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype, masks, wl.block)
    n = wl.n_steps
    c_out = np.zeros(n, np.uint8)
    f_out = np.zeros(n, np.uint8)
    margins = np.zeros((n, 2), np.float64)
    snap_steps, snap_h, snap_logits, snap_gates = [], [], [], []
    h = cp = fp = None
    for s0 in range(0, n, CHUNK):
        r = om.run(cond, CHUNK, 1, synth.SEED_SAMPLING, hop=synth.HOP, step0=s0, h=h, c_prev=cp, f_prev=fp, dump=True)
        c_out[s0:s0 + CHUNK] = r.c_out[0]
        f_out[s0:s0 + CHUNK] = r.f_out[0]
        margins[s0:s0 + CHUNK] = r.margins[0]
        snap_steps.append(s0 + CHUNK - 1)
        snap_h.append(r.hs[-1, 0].copy())
        snap_logits.append(r.logits[-1, 0].copy())
        snap_gates.append(r.gates[-1, 0].copy())
        h, cp, fp = r.h, r.c_prev, r.f_prev
        print("step %d" % (s0 + CHUNK), flush=True)
    flat = margins.reshape(-1)
    nb = np.nonzero(flat < NB_STORE)[0].astype(np.int32)
    every4 = np.arange(3, len(snap_steps), 4)
    np.savez_compressed(
        OUT, c_out=c_out, f_out=f_out, nb_index=nb, nb_margin=flat[nb], snap_steps=np.array(snap_steps, np.int32),
        snap_h=np.stack(snap_h), snap_logits=np.stack(snap_logits), snap_gates_steps=np.array(snap_steps, np.int32)[every4],
        snap_gates=np.stack(snap_gates)[every4], h_final=h[0],
        inputs_sha256=np.array(inputs_digest(w, masks, cond)))
    print("wrote %s (%d bytes), %d draws within %g of a boundary" % (OUT, os.path.getsize(OUT), nb.size, NB_STORE))


if __name__ == "__main__":
    main()
