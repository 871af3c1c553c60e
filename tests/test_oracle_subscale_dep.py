"""Pins of the oracle's dependent subscale generation (Sections 4.1, 4.2): the ordering of Eq. 4 (sub-tensor s after all
z < s), the future horizon F, and the reductions that the definition implies.  The conditioning network itself (one
masked convolution) is the oracle's stated reading."""
import numpy as np
import pytest
from scipy import signal

from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth


def _setup(H=16, B=4, L=40, F=5, D=4, hop=7):
    w = synth.make_weights(H, cond_dim=D, seed_w=21, seed_b=22)
    for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
        w[k] = (w[k] * 2.0).astype(np.float32)
    om = orc.OracleModel(w, "f32")
    V, b = synth.make_subscale_conv(B, F, D, seed=5)
    frames = synth.make_cond(B, (B * L) // hop + 2, D)
    return om, V, b, frames, B, L, F, hop


def test_convolution_matches_scipy_correlate():
    rng = np.random.default_rng(0)
    B, L, F, D = 4, 50, 6, 3
    hist = rng.integers(-32768, 32767, size=(B, L)).astype(np.int16)
    V, b = synth.make_subscale_conv(B, F, D, seed=1)
    s = 3
    got = orc.subscale_conditioning(hist, s, V, b)
    ref = np.tile(b.astype(np.float64), (L, 1))
    for delta in range(1, s + 1):
        x = np.concatenate([hist[s - delta].astype(np.float64) / 32768.0, np.zeros(F)])
        for k in range(D):
            ref[:, k] += signal.correlate(x, V[delta - 1, :, k].astype(np.float64), mode="valid")
    assert np.allclose(got, np.maximum(ref, 0.0), rtol=1e-6, atol=1e-6)


def test_row_zero_is_an_ordinary_stream_and_zero_weights_give_independent_rows():
    om, V, b, frames, B, L, F, hop = _setup()
    out, cond, _ = orc.subscale_dependent_run(om, frames, V, b, B, L, hop, seed=3)
    idx = (B * np.arange(L)) // hop
    plain = om.run((frames[0][idx] + np.maximum(b, 0.0)[None, :])[None], L, 1, 3, hop=1, stream0=0)
    assert np.array_equal(out[0], plain.out[0])
    # V = 0, b = 0: every row is the independent stream of the lock-step fold (frame (B i + s) div hop, stream id s)
    out0, _, _ = orc.subscale_dependent_run(om, frames, np.zeros_like(V), np.zeros_like(b), B, L, hop, seed=3)
    lock = om.run(frames, L, B, 3, hop=hop, row_stride=B, row_offset_mul=1)
    assert np.array_equal(out0, lock.out)


def test_dependency_order_and_future_horizon():
    om, V, b, frames, B, L, F, hop = _setup()
    base, cond, _ = orc.subscale_dependent_run(om, frames, V, b, B, L, hop, seed=9)
    s, i = 2, 11
    hist = base.copy()
    # a sample of an earlier row beyond the horizon, or any sample of this or a later row, does not reach v_s[i]
    for (z, j) in ((1, i + F + 1), (0, i + F + 3), (1, i - 1), (2, i), (3, i + 1)):
        h2 = hist.copy(); h2[z, j] ^= 0x4000
        assert np.array_equal(orc.subscale_conditioning(h2, s, V, b)[i], orc.subscale_conditioning(hist, s, V, b)[i]), (z, j)
    # inside the horizon of an earlier row it does
    for (z, j) in ((1, i), (0, i + F), (1, i + 2)):
        h2 = hist.copy(); h2[z, j] ^= 0x4000
        assert not np.array_equal(orc.subscale_conditioning(h2, s, V, b)[i], orc.subscale_conditioning(hist, s, V, b)[i]), (z, j)
    # forcing the earlier rows to the generated ones reproduces the run
    again, cond2, _ = orc.subscale_dependent_run(om, frames, V, b, B, L, hop, seed=9, forced=base)
    assert np.array_equal(again, base) and np.array_equal(cond2, cond)
    # teacher mode: every row also fed its own forced samples; on the oracle's own output nothing changes, and a
    # flipped sample inside a row changes only what is drawn after it in that row and in later rows
    t, cond3, mg = orc.subscale_dependent_run(om, frames, V, b, B, L, hop, seed=9, forced=base, teacher=True)
    assert np.array_equal(t, base) and np.array_equal(cond3, cond)
    bent = base.copy(); bent[1, 20] ^= 0x0100
    t2, _, mg2 = orc.subscale_dependent_run(om, frames, V, b, B, L, hop, seed=9, forced=bent, teacher=True)
    assert np.array_equal(t2[0], base[0]) and np.array_equal(t2[1, :21], base[1, :21])
    # (the distance of a draw's uniform from its CDF boundary moves with every change of the logits)
    # the bent bit is in the coarse byte of position 20: the fine draw of that very step already sees it (Eq. 2: c_t
    # enters the fine gates), the coarse draw of the step and everything before it does not
    assert np.array_equal(mg2[0], mg[0]) and np.array_equal(mg2[1, :20], mg[1, :20]) and mg2[1, 20, 0] == mg[1, 20, 0]
    assert mg2[1, 20, 1] != mg[1, 20, 1] and not np.array_equal(mg2[1, 21], mg[1, 21]) and not np.array_equal(mg2[2], mg[2])


def test_split_join_samples_roundtrip():
    x = np.array([-32768, -1, 0, 1, 255, 256, 32767, -12345], np.int16)
    c, f = orc.split_samples(x)
    assert np.array_equal(orc.join_samples(c, f), x)
    assert (c[0], f[0]) == (0, 0) and (c[2], f[2]) == (128, 0) and (c[6], f[6]) == (255, 255)
