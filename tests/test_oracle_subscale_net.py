"""Pins of the oracle's conditioning network (Sections 4.1, 5.3): the mask (no sample of a sub-tensor z >= s, of the
past, or beyond the reach of the dilated stack enters v_s[i]), every layer against a library convolution, the whole
network against naive loops on a tiny case, and the shape the paper states."""
import numpy as np
import pytest
import torch

from oracle import subscale_net as sn
from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth


def _small(B=4, D=3, conv=6, res=8, dil=(1, 2, 2), seed=3):
    return synth.make_subscale_net(B, cond_dim=D, conv_ch=conv, res_ch=res, dilations=dil, seed=seed)


def test_paper_shape_and_reach():
    w = synth.make_subscale_net(16)
    net = sn.SubscaleNet(w)
    assert net.n_layers == 10 and net.taps == 3                                      # ten layers, kernels of size 3
    assert w["W_conv"].shape == (10, 3, 384, 768) and w["W_res"].shape == (10, 768, 384)   # 384 / 768 channels
    assert len(set(net.dilation)) == 5 and net.dilation == sorted(net.dilation)      # five stages of increasing dilation
    assert net.reach == 124 and net.reach <= 128                                     # inside the future horizon F = 128


def test_mask_and_receptive_field():
    net = sn.SubscaleNet(_small())
    rng = np.random.default_rng(1)
    B, L = 4, 40
    hist = rng.integers(-32768, 32767, size=(B, L)).astype(np.int16)
    s, i = 2, 9
    base = net.conditioning(hist, s)
    assert net.reach == 10
    # no effect: the sub-tensor itself and later ones, the past of earlier ones, anything beyond the reach
    for (z, j) in ((2, i), (2, i + 1), (3, i + 3), (1, i - 1), (0, i - 3), (0, i + net.reach + 1), (1, i + net.reach + 4)):
        h2 = hist.copy(); h2[z, j] ^= 0x4000
        assert np.array_equal(net.conditioning(h2, s)[i], base[i]), (z, j)
    # an effect: positions i .. i + reach of the earlier sub-tensors
    for (z, j) in ((0, i), (1, i), (0, i + 1), (1, i + net.reach), (0, i + 5)):
        h2 = hist.copy(); h2[z, j] ^= 0x4000
        assert not np.array_equal(net.conditioning(h2, s)[i], base[i]), (z, j)
    # sub-tensor 0 sees nothing: its conditioning is the same vector at every position that is a full reach from the end
    v0 = net.conditioning(hist, 0)
    assert np.array_equal(v0[0], v0[L - net.reach - 1]) and not np.array_equal(v0[0], v0[L - 1])


def test_every_layer_against_torch_conv1d():
    """The same network, layer by layer, with torch's dilated cross-correlation on the zero-padded sequence."""
    w = _small(B=5, D=4, conv=7, res=9, dil=(1, 1, 2, 4))
    net = sn.SubscaleNet(w)
    rng = np.random.default_rng(2)
    L, s = 33, 3
    hist = rng.integers(-32768, 32767, size=(5, L)).astype(np.int16)
    f64 = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    X = hist.astype(np.float64).T / 32768.0
    X[:, s:] = 0.0
    x = f64(X) @ f64(net.w["W_in"]).T + f64(net.w["b_in"])                      # [L][res]
    for l, d in enumerate(net.dilation):
        xp = torch.nn.functional.pad(x.T[None], (0, 2 * d))                        # [1][res][L + 2 d], zeros beyond the row
        W = f64(net.w["W_conv"][l]).permute(1, 2, 0).contiguous()                  # [conv][res][tap]
        a = torch.relu(torch.nn.functional.conv1d(xp, W, f64(net.w["b_conv"][l]), dilation=d))[0].T
        x = x + a @ f64(net.w["W_res"][l]).T + f64(net.w["b_res"][l])
    v = torch.relu(x) @ f64(net.w["W_out"]).T + f64(net.w["b_out"])
    assert np.allclose(net.conditioning(hist, s), v.numpy(), rtol=1e-6, atol=1e-6)


def test_against_naive_loops():
    w = _small(B=3, D=2, conv=3, res=4, dil=(1, 2))
    net = sn.SubscaleNet(w)
    rng = np.random.default_rng(5)
    L, s = 9, 2
    hist = rng.integers(-32768, 32767, size=(3, L)).astype(np.int16)
    W = {k: np.asarray(v, np.float64) for k, v in net.w.items()}
    x = [[W["b_in"][c] + sum(W["W_in"][c][z] * (hist[z][i] / 32768.0) for z in range(s)) for c in range(4)] for i in range(L)]
    for l, d in enumerate(net.dilation):
        a = [[max(0.0, W["b_conv"][l][c] + sum(W["W_conv"][l][t][c][r] * x[i + t * d][r] for t in range(3) if i + t * d < L for r in range(4)))
              for c in range(3)] for i in range(L)]
        x = [[x[i][r] + W["b_res"][l][r] + sum(W["W_res"][l][r][c] * a[i][c] for c in range(3)) for r in range(4)] for i in range(L)]
    v = [[W["b_out"][k] + sum(W["W_out"][k][r] * max(0.0, x[i][r]) for r in range(4)) for k in range(2)] for i in range(L)]
    assert np.allclose(net.conditioning(hist, s), np.array(v), rtol=1e-6, atol=1e-7)


def test_weights_are_rounded_to_bf16_and_biases_are_not():
    w = _small()
    net = sn.SubscaleNet(w)
    for k in ("W_in", "W_conv", "W_res", "W_out"):
        assert np.array_equal(net.w[k], torch.from_numpy(w[k]).to(torch.bfloat16).to(torch.float32).numpy())
    assert np.array_equal(net.w["b_conv"], w["b_conv"])


def test_generation_order_and_teacher_mode():
    H, B, L, D, hop = 16, 4, 30, 3, 7
    ww = synth.make_weights(H, cond_dim=D, seed_w=21, seed_b=22)
    om = orc.OracleModel(ww, "f32")
    net = sn.SubscaleNet(_small(B=B, D=D))
    frames = synth.make_cond(B, (B * L) // hop + 2, D)
    out, cond, mg = sn.subscale_net_run(om, net, frames, L, hop, seed=4)
    # row 0 is an ordinary stream with the row-0 conditioning; forcing the generated history reproduces the run
    idx = (B * np.arange(L)) // hop
    r0 = om.run((frames[0][idx] + net.conditioning(np.zeros((B, L), np.int16), 0))[None], L, 1, 4, hop=1, stream0=0)
    assert np.array_equal(out[0], r0.out[0])
    again, cond2, _ = sn.subscale_net_run(om, net, frames, L, hop, seed=4, forced=out, teacher=True)
    assert np.array_equal(again, out) and np.array_equal(cond2, cond)
    # activations stay of order one with the synthetic weights (the conditioning matters, and nothing blows up)
    big = sn.SubscaleNet(synth.make_subscale_net(16))
    rng = np.random.default_rng(0)
    v = big.conditioning(rng.integers(-32768, 32767, size=(16, 200)).astype(np.int16), 9)
    assert 0.2 < float(np.sqrt((v[:60] ** 2).mean())) < 5.0
