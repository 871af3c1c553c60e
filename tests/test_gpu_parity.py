"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (per vector v at each step: |gpu_i - ref_i| <= tol * max(|ref_i|, rms(ref))):
1e-4 for fp32 weights, 2e-3 for bf16 weights (the oracle uses the same bf16-rounded weights);
drawn indices bit-exact except where the uniform lies within 1e-5 of a CDF boundary.
"""
import numpy as np
import pytest

from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SEED = synth.SEED_SAMPLING


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_1802_08435_b200 import binding as B
    assert torch.cuda.is_available()
    return torch, B


def _tiny(H, cond_dim=4, scale=2.0):
    w = synth.make_weights(H, cond_dim=cond_dim, seed_w=7, seed_b=8)
    for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
        if w[k] is not None:
            w[k] = (w[k] * scale).astype(np.float32)
    return w


@pytest.mark.parametrize("kernel", ["generic"])
@pytest.mark.parametrize("H,dtype,batch,sparse", [
    (8, "f32", 1, False), (16, "f32", 3, False), (32, "bf16", 1, False), (64, "bf16", 11, False),
    (40, "f32", 1, False), (32, "bf16", 2, True), (128, "f32", 9, True),
])
def test_tiny_teacher_forced(env, kernel, H, dtype, batch, sparse):
    torch, B = env
    w = _tiny(H)
    masks = synth.make_block_masks(H, 0.5, seed=3) if sparse else None
    om = orc.OracleModel(w, dtype, masks)
    m = B.wrnn_create(w, dtype, masks, max_batch=batch, kernel=B.WRNN_KERNEL_GENERIC)
    try:
        cond = synth.make_cond(batch, 6, 4)
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 50, batch, SEED, hop=10, row_stride=1, row_offset_mul=1)
        assert r["idx_bad"] == 0, r
        tol = pu.TOL[dtype]
        assert r["gates_err"] < tol and r["h_err"] < tol and r["logits_err"] < tol, r
    finally:
        B.wrnn_destroy(m)


def test_unconditioned_model_and_null_biases(env):
    torch, B = env
    w = _tiny(16, cond_dim=0)
    for k in ("b_gate", "b1", "b2", "b3", "b4"):
        w[k] = None
    om = orc.OracleModel(w, "f32")
    m = B.wrnn_create(w, "f32", kernel=B.WRNN_KERNEL_GENERIC)
    try:
        r = pu.teacher_forced_parity(torch, B, m, om, None, 40, 1, 5)
        assert r["idx_bad"] == 0 and r["gates_err"] < 1e-4 and r["logits_err"] < 1e-4, r
    finally:
        B.wrnn_destroy(m)


def _free_run(torch, B, m, cond_np, n_steps, batch, seed, **kw):
    cond = None if cond_np is None else torch.from_numpy(cond_np).cuda()
    out = torch.zeros((batch, n_steps), dtype=torch.int16, device="cuda:0")
    B.wrnn_sample(m, cond, n_steps, batch, seed, out, **kw)
    torch.cuda.synchronize()
    assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
    return out.cpu().numpy()


def _report(name, r, extra=""):
    print("\n[parity] %s: idx_diff=%d (near-boundary draws %d, bad %d) gates=%.2e h=%.2e logits=%.2e %s" % (
        name, r["idx_diff"], r["near_boundary"], r["idx_bad"], r.get("gates_err", -1), r.get("h_err", -1),
        r.get("logits_err", -1), extra))


@pytest.mark.parametrize("kernel", ["generic", "auto"])
def test_config0_dense_f32_1200(env, kernel):
    """Dense H=896 fp32, batch 1, 1200 steps: every step's gates / h / logits and both draws."""
    torch, B = env
    wl = synth.WORKLOADS[0]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    m = B.wrnn_create(w, wl.dtype, kernel=B.WRNN_KERNEL_GENERIC if kernel == "generic" else B.WRNN_KERNEL_AUTO)
    try:
        r = pu.teacher_forced_parity(torch, B, m, om, cond, wl.n_steps, 1, SEED)
        free = _free_run(torch, B, m, cond, wl.n_steps, 1, SEED)
        div = pu.first_divergence(free, r["oracle"].out)
        _report("config0/%s" % kernel, r, "free-run first divergence step %d" % div)
        assert r["idx_bad"] == 0
        assert r["gates_err"] < 1e-4 and r["h_err"] < 1e-4 and r["logits_err"] < 1e-4, r
        if div >= 0:   # a free run may only leave the oracle's stream at a near-boundary draw
            assert r["oracle"].margins[0, div].min() < pu.MARGIN
        free2 = _free_run(torch, B, m, cond, wl.n_steps, 1, SEED)
        assert np.array_equal(free, free2)          # deterministic
    finally:
        B.wrnn_destroy(m)


def test_resume_and_state_roundtrip(env):
    torch, B = env
    w = _tiny(64)
    m = B.wrnn_create(w, "bf16", max_batch=3, kernel=B.WRNN_KERNEL_AUTO)
    try:
        cond = synth.make_cond(3, 10, 4)
        full = _free_run(torch, B, m, cond, 90, 3, 77, hop=10)
        h = torch.zeros((3, 64), dtype=torch.float32, device="cuda:0")
        cp = torch.full((3,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((3,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond, 35, 3, 77, hop=10, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond, 55, 3, 77, hop=10, h=h, c_prev=cp, f_prev=fp, step0=35)
        assert np.array_equal(np.concatenate([a, b], axis=1), full)
        # rows are independent streams: row 2 alone with stream0 = 2
        one = _free_run(torch, B, m, cond[2:3], 90, 1, 77, hop=10, stream0=2)
        assert np.array_equal(one[0], full[2])
    finally:
        B.wrnn_destroy(m)


def test_fold_unfold_exact_permutation(env):
    torch, B = env
    for n, Bf in [(24000, 16), (16, 16), (35, 5), (7, 1)]:
        x = torch.randint(-32768, 32767, (n,), dtype=torch.int16, device="cuda:0")
        sub = torch.zeros((Bf, n // Bf), dtype=torch.int16, device="cuda:0")
        B.wrnn_fold(x, Bf, sub)
        assert np.array_equal(sub.cpu().numpy(), orc.fold(x.cpu().numpy(), Bf))
        y = torch.zeros_like(x)
        B.wrnn_unfold(sub, Bf, y)
        assert torch.equal(x, y)


def test_argument_errors(env):
    torch, B = env
    w = _tiny(16)
    m = B.wrnn_create(w, "f32", max_batch=2, kernel=B.WRNN_KERNEL_GENERIC)
    try:
        cond = torch.zeros((2, 2, 4), device="cuda:0")
        out = torch.zeros((2, 100), dtype=torch.int16, device="cuda:0")
        with pytest.raises(B.WrnnError) as e:
            B.wrnn_sample(m, cond, 100, 2, 1, out, hop=10)      # frames run out
        assert e.value.code == B.WRNN_ERR_INVALID_ARG
        with pytest.raises(B.WrnnError):
            B.wrnn_sample(m, cond, 10, 3, 1, out, hop=10)       # batch > max_batch
        with pytest.raises(B.WrnnError):
            B.wrnn_sample(m, None, 10, 1, 1, out, hop=10)       # conditioned model without cond
        B.wrnn_sample(m, cond, 0, 2, 1, out, hop=10)            # zero steps is a no-op
    finally:
        B.wrnn_destroy(m)
    with pytest.raises(B.WrnnError):
        B.wrnn_create(synth.make_weights(8, cond_dim=0) | {"R": np.zeros((30, 10), np.float32)}, "f32")   # H = 10
