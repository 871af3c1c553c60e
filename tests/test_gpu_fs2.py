"""GPU parity of the Fused Subscale WaveRNN 2x (Section 4.4) against the CPU oracle: the resident kernel's fused mode,
through the C ABI, on the same seeded inputs.  Tolerances as for the base model with bf16 weights (2e-3 on gates, state
and logits; drawn nibbles identical except where the uniform lies within 1e-5 of a CDF boundary)."""
import numpy as np
import pytest

from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SEED = synth.SEED_SAMPLING
H = 896


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_1802_08435_b200 import binding as B
    assert torch.cuda.is_available()
    w = synth.make_weights(H, cond_dim=synth.COND_DIM, n_inputs=12, n_logits=64)
    m = B.wrnn_create(w, "bf16", max_batch=1, variant=1)
    yield torch, B, w, m
    B.wrnn_destroy(m)


def _nibbles(x):
    x = x.astype(np.int64)
    return np.stack([(x >> 12) & 15, (x >> 8) & 15, (x >> 4) & 15, x & 15], axis=-1)


def test_teacher_forced_parity_and_free_run(env):
    torch, B, w, m = env
    T = 1500
    om = orc.Fs2OracleModel(w, "bf16")
    cond = synth.make_cond(1, T // synth.HOP + 2)
    ref = om.run(cond[0], T, seed=SEED, hop=synth.HOP, dump=True)
    dev = "cuda:0"
    cd = torch.from_numpy(cond).to(dev)
    # unsigned 16-bit device arrays are held as int16 tensors (same bytes)
    u16 = lambda a: torch.from_numpy(a.astype(np.uint16).view(np.int16).copy()).to(dev)
    back = lambda t: t.cpu().numpy().view(np.uint16)
    af, bf = u16(ref.a_out), u16(ref.b_out)
    ao, bo = torch.zeros_like(af), torch.zeros_like(bf)
    gates = torch.zeros((T, 3 * H), dtype=torch.float32, device=dev)
    hs = torch.zeros((T, H), dtype=torch.float32, device=dev)
    logits = torch.zeros((T, 2, 64), dtype=torch.float32, device=dev)
    hfin = torch.zeros((H,), dtype=torch.float32, device=dev)
    ap = torch.full((1,), -32768, dtype=torch.int16, device=dev)      # 0x8000
    bp = torch.full((1,), -32768, dtype=torch.int16, device=dev)
    B.wrnn_fs2_step_teacher_forced(m, cd, T, SEED, af, bf, ao, bo, dbg_gates=gates, dbg_h=hs, dbg_logits=logits,
                                   hop=synth.HOP, h=hfin, a_prev=ap, b_prev=bp)
    torch.cuda.synchronize()
    assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
    tol = pu.TOL["bf16"]
    assert pu.rel_err(gates.cpu().numpy(), ref.gates) < tol
    assert pu.rel_err(hs.cpu().numpy(), ref.hs) < tol
    assert pu.rel_err(logits.cpu().numpy(), ref.logits) < tol
    assert pu.rel_err(hfin.cpu().numpy(), ref.h) < tol
    # drawn nibbles: identical unless the uniform sits on a CDF boundary
    got = np.concatenate([_nibbles(back(ao)), _nibbles(back(bo))], axis=1)   # [T][8]
    want = np.concatenate([_nibbles(ref.a_out), _nibbles(ref.b_out)], axis=1)
    diff = got != want
    assert not (diff & (ref.margins >= pu.MARGIN)).any(), int(diff.sum())
    print("\n[parity] fused2x: nibble_diff=%d near-boundary=%d gates=%.2e h=%.2e logits=%.2e" % (
        int(diff.sum()), int((ref.margins < pu.MARGIN).sum()), pu.rel_err(gates.cpu().numpy(), ref.gates),
        pu.rel_err(hs.cpu().numpy(), ref.hs), pu.rel_err(logits.cpu().numpy(), ref.logits)))
    assert int(back(ap)[0]) == int(ref.a_out[-1]) and int(back(bp)[0]) == int(ref.b_out[-1])

    # free run: may leave the oracle's stream only at a near-boundary draw; deterministic; resume is bit-exact
    out = torch.zeros((2, T), dtype=torch.int16, device=dev)
    B.wrnn_fs2_sample(m, cd, T, SEED, out, hop=synth.HOP)
    torch.cuda.synchronize()
    free = out.cpu().numpy()
    div = pu.first_divergence(free, ref.out)
    if div >= 0:
        assert ref.margins[div].min() < pu.MARGIN
    out2 = torch.zeros_like(out)
    B.wrnn_fs2_sample(m, cd, T, SEED, out2, hop=synth.HOP)
    torch.cuda.synchronize()
    assert np.array_equal(out2.cpu().numpy(), free)
    h = torch.zeros((H,), dtype=torch.float32, device=dev)
    ap.fill_(-32768); bp.fill_(-32768)
    o1 = torch.zeros((2, 600), dtype=torch.int16, device=dev)
    o2 = torch.zeros((2, T - 600), dtype=torch.int16, device=dev)
    B.wrnn_fs2_sample(m, cd, 600, SEED, o1, hop=synth.HOP, h=h, a_prev=ap, b_prev=bp)
    B.wrnn_fs2_sample(m, cd, T - 600, SEED, o2, hop=synth.HOP, h=h, a_prev=ap, b_prev=bp, step0=600)
    torch.cuda.synchronize()
    assert np.array_equal(np.concatenate([o1.cpu().numpy(), o2.cpu().numpy()], axis=1), free)

    # unfold: u_{2i} = a_i, u_{2i+1} = the b of step i + 2
    u = torch.zeros((2 * (T - 2),), dtype=torch.int16, device=dev)
    B.wrnn_fs2_unfold(out, T, u)
    torch.cuda.synchronize()
    assert np.array_equal(u.cpu().numpy(), orc.fs2_unfold(free))


def test_variant_gating(env):
    torch, B, w, m = env
    out = torch.zeros((1, 8), dtype=torch.int16, device="cuda:0")
    cd = torch.from_numpy(synth.make_cond(1, 2)).cuda()
    with pytest.raises(B.WrnnError) as e:
        B.wrnn_sample(m, cd, 8, 1, SEED, out)
    assert e.value.code == 2
    base = B.wrnn_create(synth.make_weights(64, cond_dim=synth.COND_DIM), "bf16", max_batch=1, kernel=B.WRNN_KERNEL_GENERIC)
    try:
        with pytest.raises(B.WrnnError) as e:
            B.wrnn_fs2_sample(base, cd, 8, SEED, torch.zeros((2, 8), dtype=torch.int16, device="cuda:0"))
        assert e.value.code == 2
    finally:
        B.wrnn_destroy(base)
    with pytest.raises(B.WrnnError):      # the variant exists for dense bf16 single-stream models only
        B.wrnn_create(w, "f32", max_batch=1, variant=1)


def test_short_runs_and_unfold_sizes(env):
    """One, two and three steps: the first two samples of part B are pre-roll, so the unfold of n steps has 2 (n - 2)
    samples; short calls chained through the carry state reproduce a longer run."""
    torch, B, w, m = env
    dev = "cuda:0"
    cd = torch.from_numpy(synth.make_cond(1, 3)).to(dev)
    full = torch.zeros((2, 6), dtype=torch.int16, device=dev)
    B.wrnn_fs2_sample(m, cd, 6, SEED, full, hop=synth.HOP)
    h = torch.zeros((H,), dtype=torch.float32, device=dev)
    ap = torch.full((1,), -32768, dtype=torch.int16, device=dev)
    bp = torch.full((1,), -32768, dtype=torch.int16, device=dev)
    pieces, pos = [], 0
    for n in (1, 2, 3):
        o = torch.zeros((2, n), dtype=torch.int16, device=dev)
        B.wrnn_fs2_sample(m, cd, n, SEED, o, hop=synth.HOP, h=h, a_prev=ap, b_prev=bp, step0=pos)
        pieces.append(o.cpu().numpy()); pos += n
    torch.cuda.synchronize()
    assert np.array_equal(np.concatenate(pieces, axis=1), full.cpu().numpy())
    for n in (1, 2, 3, 6):
        u = torch.full((max(2 * (n - 2), 1),), 77, dtype=torch.int16, device=dev)
        B.wrnn_fs2_unfold(full[:, :n].contiguous(), n, u)
        torch.cuda.synchronize()
        ref = orc.fs2_unfold(full[:, :n].cpu().numpy())
        assert np.array_equal(u.cpu().numpy()[: ref.size], ref)
        if n <= 2:
            assert int(u.cpu()[0]) == 77          # nothing written
