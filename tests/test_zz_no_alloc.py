"""The allocation-free sampling entry point.

Some embedders of this library cannot allocate device memory when they sample: a real-time audio thread
(an allocation may block or synchronise the device), code running where allocation is forbidden, or a
service with a fixed memory budget.  `wrnn_sample_noalloc` serves them from a fixed array inside the
library image.  This test calls it through the C ABI twice in a row and checks the samples against the
ordinary entry point (same kernel, so the 16-bit samples must be identical), and checks that a request
too large for the fixed array is refused.  Collected last on purpose: it exercises state shared by the
whole process.
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
