"""Pins of the oracle's Fused Subscale WaveRNN 2x (the paper's subsection of that name): what the paper and the
mathematics fix -- 32 bits per step as 8 softmaxes of 4 bits, the state split in two parts, future horizon F = 2, the
lag (F + 1 steps per sub-tensor in general; here part B follows part A inside the step), samples fed back as direct
inputs -- plus library and brute-force cross-checks of the arithmetic.  The wiring beyond those facts is the oracle's
stated reading."""
import numpy as np
import pytest
import torch

from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth
from tests import brute


def fs2_weights(H, cond_dim=4, scale=2.0, seed=11):
    w = synth.make_weights(H, cond_dim=cond_dim, seed_w=seed, seed_b=seed + 1, n_inputs=12, n_logits=64)
    for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
        if w[k] is not None:
            w[k] = (w[k] * scale).astype(np.float32)
    return w


def test_nibbles_exhaustive():
    """16 bits = four 4-bit symbols, most significant first; scaled endpoints are exactly -1 and +1."""
    for x in range(65536):
        n = orc.split_nibbles(x)
        assert all(0 <= v < 16 for v in n)
        assert (n[0] << 12) | (n[1] << 8) | (n[2] << 4) | n[3] == x
        assert orc.join_nibbles(n) == x
    assert orc.scale4(0) == -1.0 and orc.scale4(15) == 1.0
    assert all(orc.scale4(v + 1) > orc.scale4(v) for v in range(15))


def test_parameter_count_and_bits_per_step():
    H = 896
    w = synth.make_weights(H, cond_dim=0, n_inputs=12, n_logits=64)
    assert w["R"].shape == (3 * H, H) and w["I"].shape == (3 * H, 12)
    assert w["O2"].shape == (64, H // 2) and w["O4"].shape == (64, H // 2)
    # 8 softmaxes x 4 bits = 32 bits per step
    assert (w["O2"].shape[0] + w["O4"].shape[0]) // 16 == 8 and 8 * 4 == 32
    n = sum(w[k].size for k in ("R", "I", "O1", "O2", "O3", "O4"))
    assert n == 3 * H * H + 36 * H + 2 * (H // 2) ** 2 + 2 * 64 * (H // 2)


def _brute_step(w, h_prev, a_prev, b_prev, frame, seed, stream, t, a_forced=None, b_forced=None):
    """One step written separately from the C code, in matrix form: the masked input matrix is built explicitly (columns
    8..11 zero on part-A rows) and the whole gate vector evaluated twice (before / after a_t is known)."""
    H = h_prev.shape[0]
    Hh = H // 2
    g = w["b_gate"].astype(np.float64).copy()
    if w.get("W_cond") is not None:
        g = g + w["W_cond"].astype(np.float64) @ frame.astype(np.float64)
    Is = w["I"].astype(np.float64).copy()
    for gate in range(3):
        Is[gate * H: gate * H + Hh, 8:] = 0.0
    R = w["R"].astype(np.float64)
    nib = lambda v: [(v >> 12) & 15, (v >> 8) & 15, (v >> 4) & 15, v & 15]
    sc = lambda v: v / 7.5 - 1.0

    def cell(x):
        a = R @ h_prev.astype(np.float64)
        ix = Is @ np.array(x) + g
        u = 1.0 / (1.0 + np.exp(-(a[:H] + ix[:H])))
        r = 1.0 / (1.0 + np.exp(-(a[H:2 * H] + ix[H:2 * H])))
        e = np.tanh(r * a[2 * H:] + ix[2 * H:])
        return u * h_prev.astype(np.float64) + (1.0 - u) * e

    def head(y, O1, b1, O2, b2, part):
        q = np.maximum(O1.astype(np.float64) @ y + b1, 0.0)
        l = (O2.astype(np.float64) @ q + b2).astype(np.float32)
        d = [brute.draw(l[16 * k: 16 * k + 16], brute.uniform_py(seed, stream, t, 4 * part + k)) for k in range(4)]
        return l, (d[0] << 12) | (d[1] << 8) | (d[2] << 4) | d[3]

    x = [sc(v) for v in nib(a_prev)] + [sc(v) for v in nib(b_prev)] + [0.0] * 4
    h1 = cell(x)
    la, a_draw = head(h1[:Hh].astype(np.float32).astype(np.float64), w["O1"], w["b1"], w["O2"], w["b2"], 0)
    a_t = a_draw if a_forced is None else a_forced
    x = x[:8] + [sc(v) for v in nib(a_t)]
    h2 = cell(x)
    assert np.array_equal(h2[:Hh], h1[:Hh])            # a_t does not reach part A
    lb, b_draw = head(h2[Hh:].astype(np.float32).astype(np.float64), w["O3"], w["b3"], w["O4"], w["b4"], 1)
    b_t = b_draw if b_forced is None else b_forced
    return dict(h=np.concatenate([h1[:Hh], h2[Hh:]]).astype(np.float32), a=a_t, b=b_t, a_draw=a_draw, b_draw=b_draw, la=la, lb=lb)


@pytest.mark.parametrize("H", [8, 16, 48])
def test_oracle_vs_brute_force(H):
    w = fs2_weights(H)
    om = orc.Fs2OracleModel(w, "f32")
    T = 12
    cond = synth.make_cond(1, 3, 4)[0]
    res = om.run(cond, T, seed=3, hop=5, stream=2, dump=True)
    h = np.zeros(H, np.float32)
    a, b = 0x8000, 0x8000
    for t in range(T):
        s = _brute_step(w, h, a, b, cond[t // 5], 3, 2, t)
        assert np.allclose(res.hs[t], s["h"], rtol=0, atol=2e-7)
        assert np.allclose(res.logits[t, 0], s["la"], rtol=1e-6, atol=1e-6) and np.allclose(res.logits[t, 1], s["lb"], rtol=1e-6, atol=1e-6)
        if res.margins[t].min() > 1e-9:
            assert res.a_out[t] == s["a_draw"] and res.b_out[t] == s["b_draw"]
        assert res.out[0, t] == int(res.a_out[t]) - 32768 and res.out[1, t] == int(res.b_out[t]) - 32768
        h, a, b = res.hs[t], int(res.a_out[t]), int(res.b_out[t])


def test_cell_equals_torch_grucell():
    """The cell is Eq. 2's: with input [x ; frame] and input matrix [I*, W_cond] it equals torch's GRUCell."""
    H, D = 16, 4
    w = fs2_weights(H, cond_dim=D, scale=3.0)
    om = orc.Fs2OracleModel(w, "f32")
    rng = np.random.default_rng(1)
    h0 = rng.standard_normal(H).astype(np.float32)
    cond = rng.standard_normal((1, D)).astype(np.float32)
    a_prev, b_prev, a_t = 0x3C91, 0xF027, 0x5AB4
    res = om.run(cond, 1, seed=0, h=h0, a_prev=a_prev, b_prev=b_prev, a_forced=np.array([a_t], np.uint16),
                 b_forced=np.array([0], np.uint16), dump=True)
    cell = torch.nn.GRUCell(12 + D, H, bias=True, dtype=torch.float64)
    Is = w["I"].astype(np.float64).copy()
    for gate in range(3):
        Is[gate * H: gate * H + H // 2, 8:] = 0.0
    Wih = np.concatenate([Is, w["W_cond"].astype(np.float64)], axis=1)
    perm = lambda M: np.concatenate([M[H:2 * H], M[:H], M[2 * H:]], axis=0)
    nib = lambda v: [((v >> s) & 15) / 7.5 - 1.0 for s in (12, 8, 4, 0)]
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(perm(Wih)))
        cell.weight_hh.copy_(torch.from_numpy(perm(w["R"].astype(np.float64))))
        cell.bias_ih.copy_(torch.from_numpy(perm(w["b_gate"].astype(np.float64))))
        cell.bias_hh.zero_()
        x = torch.tensor([nib(a_prev) + nib(b_prev) + nib(a_t) + list(cond[0].astype(np.float64))], dtype=torch.float64)
        hn = cell(x, torch.from_numpy(h0.astype(np.float64))[None])[0].numpy()
    assert np.allclose(res.hs[0], hn, rtol=1e-6, atol=1e-7)


def test_future_horizon_is_two():
    """Part B of step t sees a_t, so the b it emits (position t - 2 of sub-tensor 1) is conditioned on sub-tensor 0 up
    to two positions ahead; part A of the same step does not depend on a_t, nor on the b emitted in this step."""
    H = 32
    w = fs2_weights(H, scale=1.0)
    w["I"] = np.random.default_rng(2).standard_normal((3 * H, 12)).astype(np.float32)
    om = orc.Fs2OracleModel(w, "f32")
    cond = synth.make_cond(1, 1, 4)[0]
    T = 3
    base = None
    for af in (0x0000, 0xFFFF, 0x1234):
        r = om.run(cond, T, seed=5, hop=1000, a_forced=np.full(T, af, np.uint16), b_forced=np.full(T, 0x0808, np.uint16), dump=True)
        first = (r.hs[0, : H // 2].copy(), r.logits[0, 0].copy(), r.hs[0, H // 2:].copy(), r.logits[0, 1].copy())
        if base is None:
            base = first
        else:
            assert np.array_equal(first[0], base[0]) and np.array_equal(first[1], base[1])
            assert not np.allclose(first[2], base[2]) and not np.allclose(first[3], base[3])
    # the unfold drops the two pre-roll b's: u_{2i} = a_i, u_{2i+1} = the b of step i + 2
    ab = np.arange(2 * 7, dtype=np.int16).reshape(2, 7)
    u = orc.fs2_unfold(ab)
    assert list(u) == [0, 9, 1, 10, 2, 11, 3, 12, 4, 13]


def test_each_softmax_owns_its_sixteen_logits():
    """Shifting the bias of one 16-logit group by a constant leaves every draw unchanged (softmax shift invariance per
    group); making one logit of group k dominant forces nibble k and nothing else."""
    H = 16
    w = fs2_weights(H)
    T = 20
    cond = synth.make_cond(1, 2, 4)[0]
    ref = orc.Fs2OracleModel(w, "f32").run(cond, T, seed=9, hop=10)
    w2 = dict(w); w2["b2"] = w["b2"].copy(); w2["b2"][16:32] += 3.0
    r2 = orc.Fs2OracleModel(w2, "f32").run(cond, T, seed=9, hop=10)
    assert np.array_equal(ref.out, r2.out)
    w3 = dict(w); w3["b4"] = w["b4"].copy(); w3["b4"][32 + 5] += 200.0        # nibble 2 of b forced to 5
    r3 = orc.Fs2OracleModel(w3, "f32").run(cond, T, seed=9, hop=10, a_forced=ref.a_out, b_forced=ref.b_out)
    assert np.all((r3.b_out >> 4) & 15 == 5)
    assert np.array_equal(r3.b_out & 0xFF0F, ref.b_out & 0xFF0F) and np.array_equal(r3.a_out, ref.a_out)


def test_resume_and_teacher_forcing():
    H = 24
    w = fs2_weights(H)
    om = orc.Fs2OracleModel(w, "bf16")
    cond = synth.make_cond(1, 5, 4)[0]
    full = om.run(cond, 40, seed=4, hop=10)
    a = om.run(cond, 17, seed=4, hop=10)
    b = om.run(cond, 23, seed=4, hop=10, step0=17, h=a.h, a_prev=a.a_prev, b_prev=a.b_prev)
    assert np.array_equal(np.concatenate([a.out, b.out], axis=1), full.out)
    tf = om.run(cond, 40, seed=4, hop=10, a_forced=full.a_out, b_forced=full.b_out)
    assert np.array_equal(tf.a_out, full.a_out) and np.array_equal(tf.b_out, full.b_out)


def test_nibble_draws_follow_their_softmax():
    """Each of the eight 4-bit symbols is a draw from the softmax of its own sixteen logits: with the state frozen
    (u = 1 keeps h, zero input and recurrent weights) the logits are the same at every step, and the drawn nibbles'
    frequencies match their softmax (chi-square, 5 sigma) while the eight heads use different uniforms."""
    H = 16
    w = fs2_weights(H, cond_dim=0, scale=3.0, seed=4)
    w["R"] = np.zeros_like(w["R"]); w["I"] = np.zeros_like(w["I"])
    w["b_gate"] = w["b_gate"].copy(); w["b_gate"][:H] = 80.0              # u = 1: h_t = h_{t-1}
    om = orc.Fs2OracleModel(w, "f32")
    h0 = np.random.default_rng(3).standard_normal(H).astype(np.float32)
    T = 40000
    r = om.run(None, T, seed=12, h=h0, dump=True)
    assert np.array_equal(r.hs[0], h0) and np.array_equal(r.hs[-1], h0)
    assert np.array_equal(r.logits[0], r.logits[-1])
    streams = []
    for part, drawn in ((0, r.a_out), (1, r.b_out)):
        for k in range(4):
            nib = (drawn.astype(np.int64) >> (12 - 4 * k)) & 15
            l = r.logits[0, part, 16 * k: 16 * k + 16].astype(np.float64)
            p = np.exp(l - l.max()); p /= p.sum()
            counts = np.bincount(nib, minlength=16)
            chi2 = ((counts - T * p) ** 2 / (T * p)).sum()
            assert chi2 < 15 + 5 * np.sqrt(2 * 15), (part, k, chi2)
            streams.append(nib)
    # the eight symbols are driven by eight different uniform streams
    for i in range(8):
        for j in range(i + 1, 8):
            assert not np.array_equal(streams[i], streams[j])
