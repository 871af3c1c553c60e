"""Pins for the CPU oracle: each check compares it with something it did not
produce itself (published known answers, library routines, closed forms,
brute force written separately, invariants of the method)."""
import os

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth
from tests import brute

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_weights(H, cond_dim=4, seed=7, scale=None):
    w = synth.make_weights(H, cond_dim=cond_dim, seed_w=seed, seed_b=seed + 1)
    if scale:
        for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
            if w[k] is not None:
                w[k] = (w[k] * scale).astype(np.float32)
    return w


# ---------------------------------------------------------------- Philox

def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(x, 16) for x in line.split()]
        got = orc.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in got] == v[6:10]
        n += 1
    assert n == 3


def test_philox_matches_second_implementation():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        ctr = rng.integers(0, 2**32, 4, dtype=np.uint64)
        key = rng.integers(0, 2**32, 2, dtype=np.uint64)
        assert [int(x) for x in orc.philox4x32_10(ctr, key)] == brute.philox4x32_10_py(ctr, key)


def test_uniform_keying_and_range():
    # (seed, stream, step, head) -> counter/key placement, incl. 64-bit step and seed
    for seed, stream, step, head in [(0, 0, 0, 0), (20180223, 3, 17, 1), (2**40 + 5, 255, 2**33 + 9, 0)]:
        assert orc.uniform(seed, stream, step, head) == brute.uniform_py(seed, stream, step, head)
    us = np.array([orc.uniform(1, 0, t, 0) for t in range(20000)])
    assert us.min() >= 0.0 and us.max() < 1.0
    assert np.all(us * 2**24 == np.round(us * 2**24))           # multiples of 2^-24
    assert abs(us.mean() - 0.5) < 0.01 and abs(us.var() - 1 / 12) < 0.005
    # distinct heads / streams / steps give distinct draws
    assert len({orc.uniform(1, s, t, h) for s in range(4) for t in range(4) for h in range(2)}) == 32


# ---------------------------------------------------------------- bf16

def test_bf16_round_matches_torch_exhaustive():
    hi = np.arange(1 << 16, dtype=np.uint32) << 16
    lows = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x1234, 0xC000], dtype=np.uint32)
    bits = (hi[:, None] | lows[None, :]).reshape(-1)
    x = bits.view(np.float32)
    finite = np.isfinite(x)
    got = orc.bf16_round(x)
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(got[finite].view(np.uint32), ref[finite].view(np.uint32))
    assert np.all(np.isnan(got[np.isnan(x)]))
    assert np.all((got.view(np.uint32) & 0xFFFF) == 0)


# ---------------------------------------------------------------- split / scale / fold

def test_split_join_exhaustive():
    seen = set()
    for x in range(65536):
        c, f = orc.split16(x)
        assert c == x >> 8 and f == x & 255
        assert orc.join16(c, f) == x
        s = orc.to_int16(c, f)
        assert s == x - 32768 and -32768 <= s <= 32767
        seen.add(s)
    assert len(seen) == 65536


def test_scale_endpoints():
    assert orc.scale8(0) == -1.0 and orc.scale8(255) == 1.0
    assert abs(orc.scale8(128) - (128 / 127.5 - 1)) < 1e-16
    d = np.diff([orc.scale8(v) for v in range(256)])
    assert np.allclose(d, 2 / 255, atol=1e-15)


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 32), st.integers(1, 200), st.integers(0, 2**31))
def test_fold_unfold_permutation(B, length, seed):
    n = B * length
    x = np.random.default_rng(seed).integers(-32768, 32768, n).astype(np.int16)
    sub = orc.fold(x, B)
    assert sub.shape == (B, length)
    for s in range(min(B, 3)):
        assert np.array_equal(sub[s], x[s::B])        # sub-tensor s holds u_{B i + s}
    assert np.array_equal(orc.unfold(sub), x)
    idx = orc.fold(np.arange(n).astype(np.int16) if n < 32768 else (np.arange(n) % 30000).astype(np.int16), B)
    if n < 32768:
        assert np.array_equal(np.sort(idx.reshape(-1)), np.arange(n))


# ---------------------------------------------------------------- softmax + sampler

def test_softmax_matches_scipy_and_searchsorted():
    from scipy.special import softmax
    rng = np.random.default_rng(3)
    for trial in range(200):
        l = (rng.standard_normal(256) * rng.choice([0.3, 3.0, 30.0])).astype(np.float32)
        u = rng.integers(0, 2**24) / 2**24
        idx, p, margin = orc.softmax_sample(l, u)
        ref = softmax(l.astype(np.float64))
        assert abs(p.sum() - 1.0) < 1e-12
        assert np.allclose(p, ref, rtol=1e-12, atol=1e-300)
        cdf = np.cumsum(ref)
        k = int(np.searchsorted(cdf, u, side="right"))
        if margin > 1e-9:
            assert idx == min(k, 255)
        assert abs(margin - np.abs(cdf[:-1] - u).min()) < 1e-9


def test_sampler_degenerate_cases():
    l = np.zeros(256, np.float32)
    for u in [0.0, 0.1, 0.5, 0.999, (2**24 - 1) / 2**24]:
        idx, _, _ = orc.softmax_sample(l, u)            # uniform: index = floor(256 u)
        assert idx == int(np.floor(256 * u))
    l = np.full(256, -1000.0, np.float32)     # exp underflows to exactly 0 for the others
    l[77] = 60.0
    for u in [0.0, 0.3, (2**24 - 1) / 2**24]:
        assert orc.softmax_sample(l, u)[0] == 77
    l = np.array([1000.0] + [-1000.0] * 255, np.float32)     # exp range: no overflow / NaN
    idx, p, _ = orc.softmax_sample(l, 0.7)
    assert idx == 0 and np.isfinite(p).all()


def test_sampler_distribution_chi2():
    rng = np.random.default_rng(5)
    l = (rng.standard_normal(256)).astype(np.float32)
    _, p, _ = orc.softmax_sample(l, 0.0)
    n = 200000
    counts = np.zeros(256)
    for t in range(n):
        counts[orc.softmax_sample(l, orc.uniform(99, 0, t, 0))[0]] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 255 + 5 * np.sqrt(2 * 255)       # 5 sigma


# ---------------------------------------------------------------- the cell and the step

def test_parameter_count_and_shapes():
    # "about 3M parameters" at H = 896 (Section 2.1); op list at H = 1024 (Section 5.2)
    H = 896
    w = synth.make_weights(H, cond_dim=0)
    n = sum(w[k].size for k in ("R", "I", "O1", "O2", "O3", "O4"))
    assert n == 3 * H * H + 2 * (H // 2) ** 2 + 512 * (H // 2) + 9 * H == 3047296
    assert abs(n - 3e6) / 3e6 < 0.02
    w = synth.make_weights(1024, cond_dim=0)
    assert w["R"].shape == (3 * 1024, 1024) and w["O1"].shape == (512, 512) and w["O2"].shape == (256, 512)


@pytest.mark.parametrize("H", [8, 16, 32])
def test_oracle_vs_brute_force(H):
    w = tiny_weights(H, scale=2.0)
    om = orc.OracleModel(w, "f32")
    cond = synth.make_cond(1, 3, 4, seed=H)
    T = 12
    res = om.run(cond, T, 1, seed=42, hop=5, dump=True)
    h = np.zeros(H, np.float32)
    c, f = 128, 0
    for t in range(T):
        s = brute.step(w, h, c, f, cond[0, t // 5], 42, 0, t)
        assert np.allclose(res.logits[t, 0, 0], s["lc"], rtol=1e-6, atol=1e-6)
        assert np.allclose(res.logits[t, 0, 1], s["lf"], rtol=1e-6, atol=1e-6)
        assert np.allclose(res.gates[t, 0], s["gates"], rtol=1e-6, atol=1e-7)
        assert np.allclose(res.hs[t, 0], s["h"], rtol=1e-6, atol=1e-7)
        assert (res.c_out[0, t], res.f_out[0, t]) == (s["c"], s["f"])
        assert res.out[0, t] == 256 * s["c"] + s["f"] - 32768
        # mask: recomputing the whole state with c_t present leaves the coarse half alone
        assert np.array_equal(s["coarse_after"], s["h"][: H // 2])
        h, c, f = s["h"], s["c"], s["f"]


def test_cell_equals_torch_grucell():
    """Eq. 2's cell is the GRU form with r applied after the recurrent product;
    with input [x ; frame] and input matrix [I*, W_cond] it equals torch's GRUCell
    (gate blocks (r, z, n) <- (r, u, e), z = u, hidden bias of n zero)."""
    H, D = 16, 4
    w = tiny_weights(H, cond_dim=D, scale=3.0)
    om = orc.OracleModel(w, "f32")
    rng = np.random.default_rng(1)
    h0 = rng.standard_normal(H).astype(np.float32)
    cond = rng.standard_normal((1, 1, D)).astype(np.float32)
    c_prev, f_prev, c_t = 200, 13, 91
    res = om.run(cond, 1, 1, seed=0, h=h0[None], c_prev=[c_prev], f_prev=[f_prev],
                 c_forced=np.array([[c_t]], np.uint8), f_forced=np.array([[0]], np.uint8), dump=True)
    cell = torch.nn.GRUCell(3 + D, H, bias=True, dtype=torch.float64)
    Is = brute.masked_I(w["I"], H)
    Wih = np.concatenate([Is, w["W_cond"].astype(np.float64)], axis=1)   # rows u|r|e
    perm = lambda M: np.concatenate([M[H:2 * H], M[:H], M[2 * H:]], axis=0)  # -> r|z|n
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(perm(Wih)))
        cell.weight_hh.copy_(torch.from_numpy(perm(w["R"].astype(np.float64))))
        cell.bias_ih.copy_(torch.from_numpy(perm(w["b_gate"].astype(np.float64))))
        cell.bias_hh.zero_()
        sc = lambda v: v / 127.5 - 1.0
        x = torch.tensor([[sc(c_prev), sc(f_prev), sc(c_t)] + list(cond[0, 0].astype(np.float64))], dtype=torch.float64)
        hn = cell(x, torch.from_numpy(h0.astype(np.float64))[None])[0].numpy()
    assert np.allclose(res.hs[0, 0], hn, rtol=1e-6, atol=1e-7)


def test_update_gate_limits():
    H = 8
    w = tiny_weights(H, cond_dim=0)
    h0 = np.linspace(-0.9, 0.9, H).astype(np.float32)
    w1 = dict(w); w1["b_gate"] = w["b_gate"].copy(); w1["b_gate"][:H] = 80.0     # u == 1 -> h_t = h_{t-1}
    r1 = orc.OracleModel(w1, "f32").run(None, 1, 1, h=h0[None], dump=True)
    assert np.array_equal(r1.hs[0, 0], h0)
    w0 = dict(w); w0["b_gate"] = w["b_gate"].copy(); w0["b_gate"][:H] = -80.0    # u == 0 -> h_t = e
    r0 = orc.OracleModel(w0, "f32").run(None, 1, 1, h=h0[None], dump=True)
    assert np.allclose(r0.hs[0, 0], r0.gates[0, 0, 2 * H:], rtol=0, atol=1e-7)


def test_mask_invariant_coarse_ignores_ct():
    H = 32
    w = tiny_weights(H, scale=1.0)
    w["I"] = (np.random.default_rng(2).standard_normal((3 * H, 3))).astype(np.float32)   # large I
    om = orc.OracleModel(w, "f32")
    cond = synth.make_cond(1, 1, 4)
    T = 4
    base = None
    for cf in (0, 255, 77):
        r = om.run(cond, T, 1, seed=5, hop=1000, c_forced=np.full((1, T), cf, np.uint8),
                   f_forced=np.full((1, T), 9, np.uint8), dump=True)
        first = (r.hs[0, 0, : H // 2].copy(), r.logits[0, 0, 0].copy(), r.hs[0, 0, H // 2:].copy(), r.logits[0, 0, 1].copy())
        if base is None:
            base = first
        else:
            assert np.array_equal(first[0], base[0]) and np.array_equal(first[1], base[1])
            assert not np.allclose(first[2], base[2]) and not np.allclose(first[3], base[3])


def test_supplied_ct_column_on_coarse_rows_is_ignored():
    H = 16
    w = tiny_weights(H)
    w2 = dict(w); w2["I"] = w["I"].copy()
    for gate in range(3):
        w2["I"][gate * H: gate * H + H // 2, 2] = 123.0
    cond = synth.make_cond(1, 2, 4)
    a = orc.OracleModel(w, "f32").run(cond, 20, 1, seed=1, hop=10)
    b = orc.OracleModel(w2, "f32").run(cond, 20, 1, seed=1, hop=10)
    assert np.array_equal(a.out, b.out)


def test_five_sequential_products_dependency():
    """N = 5 (Section 1): zeroing any one of R, O1..O4 changes the draw stream."""
    H = 16
    w = tiny_weights(H, scale=4.0)
    cond = synth.make_cond(1, 2, 4)
    base = orc.OracleModel(w, "f32").run(cond, 64, 1, seed=3, hop=32, dump=True)
    for k in ("R", "O1", "O2", "O3", "O4"):
        w2 = dict(w); w2[k] = np.zeros_like(w[k])
        r = orc.OracleModel(w2, "f32").run(cond, 64, 1, seed=3, hop=32, dump=True)
        assert not np.array_equal(r.logits, base.logits), k


def test_batched_rows_equal_single_streams():
    H = 16
    w = tiny_weights(H, scale=3.0)
    om = orc.OracleModel(w, "bf16")
    cond = synth.make_cond(5, 7, 4)
    full = om.run(cond, 30, 5, seed=11, hop=10, row_stride=2, row_offset_mul=1, threads=3)
    for b in range(5):
        one = om.run(cond[b:b + 1], 30, 1, seed=11, hop=10, row_stride=2, row_offset_mul=1, stream0=b)
        assert np.array_equal(one.out[0], full.out[b])
        assert np.array_equal(one.h[0], full.h[b])


def test_resume_is_bit_identical():
    H = 16
    w = tiny_weights(H, scale=3.0)
    om = orc.OracleModel(w, "f32")
    cond = synth.make_cond(2, 5, 4)
    full = om.run(cond, 50, 2, seed=8, hop=10)
    a = om.run(cond, 20, 2, seed=8, hop=10)
    b = om.run(cond, 30, 2, seed=8, hop=10, step0=20, h=a.h, c_prev=a.c_prev, f_prev=a.f_prev)
    assert np.array_equal(np.concatenate([a.out, b.out], axis=1), full.out)
    assert np.array_equal(b.h, full.h)


def test_teacher_forcing_with_own_stream_reproduces_free_run():
    H = 16
    w = tiny_weights(H, scale=3.0)
    om = orc.OracleModel(w, "f32")
    cond = synth.make_cond(1, 5, 4)
    free = om.run(cond, 40, 1, seed=2, hop=10, dump=True)
    tf = om.run(cond, 40, 1, seed=2, hop=10, c_forced=free.c_out, f_forced=free.f_out, dump=True)
    assert np.array_equal(tf.c_out, free.c_out) and np.array_equal(tf.f_out, free.f_out)
    assert np.array_equal(tf.hs, free.hs)
    u = (free.out.astype(np.int32) + 32768)
    assert np.array_equal(u >> 8, free.c_out) and np.array_equal(u & 255, free.f_out)


@pytest.mark.parametrize("block", [(4, 4), (16, 1), (1, 1)])
def test_sparse_model_is_dense_model_with_zero_blocks(block):
    """Section 3.2's block shapes: 4 x 4, m x 1 with m = 16 (16 rows of one column), and unstructured."""
    H = 32
    br, bc = block
    w = tiny_weights(H, scale=3.0)
    masks = synth.make_block_masks(H, sparsity=0.5, seed=1, block=block)
    assert masks["R"].shape == (3 * H // br, H // bc) and masks["O1"].shape == (H // 2 // br, H // 2 // bc)
    for g in range(3):
        assert masks["R"][g * H // br:(g + 1) * H // br].sum() == round(0.5 * (H // br) * (H // bc))   # per-gate masks
    wz = dict(w)
    for k, m in masks.items():
        wz[k] = w[k] * np.kron(m, np.ones((br, bc), np.float32))
        assert np.array_equal(orc.apply_block_mask(w[k], m, block), wz[k])
    cond = synth.make_cond(1, 2, 4)
    a = orc.OracleModel(w, "bf16", masks, block).run(cond, 25, 1, seed=4, hop=20, dump=True)
    b = orc.OracleModel(wz, "bf16").run(cond, 25, 1, seed=4, hop=20, dump=True)
    assert np.array_equal(a.out, b.out) and np.array_equal(a.logits, b.logits)
    d = orc.OracleModel(w, "bf16").run(cond, 25, 1, seed=4, hop=20, dump=True)
    assert not np.array_equal(a.logits, d.logits)                   # the mask does something


def test_frame_index_out_of_range_is_an_error():
    w = tiny_weights(8)
    with pytest.raises(ValueError):
        orc.OracleModel(w, "f32").run(synth.make_cond(1, 2, 4), 30, 1, hop=10)


def test_conditioning_frame_hold():
    """The frame is held for `hop` steps; row offsets shift the frame boundary (subscale rows)."""
    H = 8
    w = tiny_weights(H, scale=3.0)
    om = orc.OracleModel(w, "f32")
    cond = synth.make_cond(1, 3, 4)
    r = om.run(cond, 30, 1, seed=1, hop=10, dump=True)
    cond2 = cond.copy(); cond2[0, 1] += 1.0            # changing frame 1 changes steps 10..19 onward only
    r2 = om.run(cond2, 30, 1, seed=1, hop=10, dump=True)
    assert np.array_equal(r.gates[:10], r2.gates[:10]) and not np.array_equal(r.gates[10], r2.gates[10])
    # stride 4, offset 3: frame boundary for global row 3 falls at the first s with 4 s + 3 >= 10 -> s = 2
    r3 = om.run(cond, 6, 1, seed=1, hop=10, row_stride=4, row_offset_mul=1, stream0=3, dump=True)
    r4 = om.run(cond2, 6, 1, seed=1, hop=10, row_stride=4, row_offset_mul=1, stream0=3, dump=True)
    assert np.array_equal(r3.gates[:2], r4.gates[:2]) and not np.array_equal(r3.gates[2], r4.gates[2])


def test_stored_sparse_run_is_this_oracles():
    """The stored 24,000-step run of the block-sparse workload (tests/golden/make_sparse2048_stream.py) belongs to the
    current input generator, and the oracle reproduces its first 120 steps and their near-boundary record."""
    import hashlib
    import os
    g = np.load(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "sparse2048_bf16_b1_24000_oracle.npz"))
    wl = synth.WORKLOADS[2]
    w, masks, cond = synth.build_workload(wl)
    hsh = hashlib.sha256()
    for k in sorted(w):
        if w[k] is not None:
            hsh.update(k.encode()); hsh.update(np.ascontiguousarray(w[k]).tobytes())
    for k in sorted(masks):
        hsh.update(k.encode()); hsh.update(np.ascontiguousarray(masks[k]).tobytes())
    hsh.update(np.ascontiguousarray(cond).tobytes())
    assert hsh.hexdigest() == str(g["inputs_sha256"])
    om = orc.OracleModel(w, wl.dtype, masks, wl.block)
    r = om.run(cond, 120, 1, synth.SEED_SAMPLING, hop=synth.HOP)
    assert np.array_equal(r.c_out[0], g["c_out"][:120]) and np.array_equal(r.f_out[0], g["f_out"][:120])
    near = np.nonzero(r.margins[0].reshape(-1) < 1e-4)[0]
    assert np.array_equal(near, g["nb_index"][g["nb_index"] < 240])
    assert g["c_out"].shape == (24000,) and g["snap_h"].shape == (24, 2048) and int(g["snap_steps"][-1]) == 23999
