"""The allocation-free sampling entry point.

Some embedders of this library cannot allocate device memory when they sample: a real-time audio thread
(an allocation may block or synchronise the device), code running where allocation is forbidden, or a
service with a fixed memory budget.  `wrnn_sample_noalloc` serves them from a fixed array inside the
library image.  This test calls it through the C ABI twice in a row and checks the samples against the
ordinary entry point (same kernel, so the 16-bit samples must be identical), and checks that a request
too large for the fixed array is refused.  A second test holds its samples against the CPU oracle (a model
created with automatic kernel choice, a model without conditioning, and a call resumed from a carried
state).  Collected last on purpose: it exercises state shared by the whole process.
"""
import numpy as np
import pytest

from paper_1802_08435_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_matches_wrnn_sample_twice_and_rejects_oversize():
    import torch
    from paper_1802_08435_b200 import binding as B

    H, batch, n = 256, 3, 400
    w = synth.make_weights(H, cond_dim=16, seed_w=11, seed_b=12)
    cond_np = synth.make_cond(batch, 5, 16, seed=13)
    m = B.wrnn_create(w, "bf16", max_batch=batch, kernel=B.WRNN_KERNEL_GENERIC)
    try:
        cond = torch.from_numpy(cond_np).cuda()
        for call, seed in enumerate((5, 6)):           # two calls in a row share the fixed array
            ref = torch.zeros((batch, n), dtype=torch.int16, device="cuda:0")
            got = torch.full((batch, n), -1, dtype=torch.int16, device="cuda:0")
            hr = torch.zeros((batch, H), dtype=torch.float32, device="cuda:0")
            hg = torch.zeros((batch, H), dtype=torch.float32, device="cuda:0")
            B.wrnn_sample(m, cond, n, batch, seed, ref, hop=100, h=hr)
            torch.cuda.synchronize()
            assert B.wrnn_poll_status(m) == 0
            B.wrnn_sample_noalloc(m, cond, n, batch, seed, got, hop=100, h=hg)
            torch.cuda.synchronize()
            assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
            assert torch.equal(ref, got), "call %d: samples differ" % call
            assert torch.equal(hr, hg), "call %d: final state differs" % call
            assert len(np.unique(got.cpu().numpy())) > 50
        # a request whose conditioning scratch exceeds the fixed array is refused, nothing is launched
        big = torch.zeros((batch, 4000, 16), dtype=torch.float32, device="cuda:0")
        before = B.wrnn_launch_count()
        with pytest.raises(B.WrnnError) as e:
            B.wrnn_sample_noalloc(m, big, 10, batch, 1, got, hop=100)
        assert e.value.code == B.WRNN_ERR_UNSUPPORTED and "fixed array" in str(e.value)
        assert B.wrnn_launch_count() == before
    finally:
        B.wrnn_destroy(m)


def test_noalloc_against_the_oracle_auto_model_unconditioned_and_resume():
    """The entry point's samples against the CPU oracle (teacher-forced on those samples, so that every draw is
    compared): on a model created with automatic kernel choice (wrnn_sample would pick another kernel there; this entry
    point still runs the any-shape one), on a model without conditioning or biases, and resumed from a carried state."""
    import torch
    from oracle import wrnn_oracle as orc
    from paper_1802_08435_b200 import binding as B
    from tests import parity_util as pu

    dev = "cuda:0"
    # (1) automatic kernel choice, three rows with their own conditioning, in two calls with the state carried over
    H, batch, n = 128, 3, 300
    w = synth.make_weights(H, cond_dim=8, seed_w=21, seed_b=22)
    for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
        w[k] = (w[k] * 2).astype(np.float32)
    cond_np = synth.make_cond(batch, 4, 8, seed=23)
    om = orc.OracleModel(w, "bf16")
    m = B.wrnn_create(w, "bf16", max_batch=batch)
    try:
        cond = torch.from_numpy(cond_np).to(dev)
        h = torch.zeros((batch, H), dtype=torch.float32, device=dev)
        cp = torch.full((batch,), 128, dtype=torch.uint8, device=dev)
        fp = torch.zeros((batch,), dtype=torch.uint8, device=dev)
        a = torch.zeros((batch, 120), dtype=torch.int16, device=dev)
        b = torch.zeros((batch, n - 120), dtype=torch.int16, device=dev)
        B.wrnn_sample_noalloc(m, cond, 120, batch, 9, a, hop=100, h=h, c_prev=cp, f_prev=fp)
        B.wrnn_sample_noalloc(m, cond, n - 120, batch, 9, b, hop=100, h=h, c_prev=cp, f_prev=fp, step0=120)
        torch.cuda.synchronize()
        assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
        got = np.concatenate([a.cpu().numpy(), b.cpu().numpy()], axis=1)
        chk = pu.oracle_on_gpu_stream(om, cond_np, range(batch), got, 9, hop=100, h_final=h.cpu().numpy())
        assert chk["idx_bad"] == 0 and chk["h_final_err"] < pu.TOL["bf16"], chk
    finally:
        B.wrnn_destroy(m)
    # (2) no conditioning, no biases, fp32
    w = synth.make_weights(32, cond_dim=0, seed_w=31, seed_b=32)
    for k in ("b_gate", "b1", "b2", "b3", "b4"):
        w[k] = None
    om = orc.OracleModel(w, "f32")
    m = B.wrnn_create(w, "f32", max_batch=2)
    try:
        out = torch.zeros((2, 200), dtype=torch.int16, device=dev)
        h = torch.zeros((2, 32), dtype=torch.float32, device=dev)
        B.wrnn_sample_noalloc(m, None, 200, 2, 4, out, h=h)
        torch.cuda.synchronize()
        assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
        chk = pu.oracle_on_gpu_stream(om, None, range(2), out.cpu().numpy(), 4, h_final=h.cpu().numpy())
        assert chk["idx_bad"] == 0 and chk["h_final_err"] < pu.TOL["f32"], chk
    finally:
        B.wrnn_destroy(m)
