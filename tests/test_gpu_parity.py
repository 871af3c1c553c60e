"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (per vector v at each step: |gpu_i - ref_i| <= tol * max(|ref_i|, rms(ref))):
1e-4 for fp32 weights, 2e-3 for bf16 weights (the oracle uses the same bf16-rounded weights);
drawn indices bit-exact except where the uniform lies within 1e-5 of a CDF boundary.
"""
import os

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


@pytest.mark.parametrize("kernel,H,batch", [
    ("BATCHED", 128, 2), ("BATCHED", 128, 11), ("BATCHED", 256, 33), ("BATCHED", 384, 16), ("BATCHED", 128, 70),
    ("BCLUSTER", 128, 2), ("BCLUSTER", 128, 11), ("BCLUSTER", 256, 33), ("BCLUSTER", 384, 16), ("BCLUSTER", 128, 70),
    ("BCLUSTER", 256, 130), ("BCLUSTER", 128, 300)])
def test_tiny_batched_kernel(env, kernel, H, batch):
    """The two multi-row kernels on small shapes: ragged batches; one and several stream blocks (grid-phased kernel);
    one and several clusters, one to three lane quadrants per cluster (cluster-partitioned kernel)."""
    torch, B = env
    w = _tiny(H)
    om = orc.OracleModel(w, "bf16")
    kid = getattr(B, "WRNN_KERNEL_" + kernel)
    m = B.wrnn_create(w, "bf16", max_batch=batch, kernel=kid)
    try:
        assert B.wrnn_launch_info(m, batch)["kernel"] == kid
        cond = synth.make_cond(batch, (40 + batch) // 10 + 2, 4)
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 40, batch, SEED, hop=10, row_stride=1, row_offset_mul=1,
                                     threads=pu.NCPU)
        assert r["idx_bad"] == 0, {k: v for k, v in r.items() if k != "oracle"}
        tol = pu.TOL["bf16"]
        assert r["gates_err"] < tol and r["h_err"] < tol and r["logits_err"] < tol, {k: v for k, v in r.items() if k != "oracle"}
        # a smaller batch on the same model, with a row offset, and resume
        lo = batch - 2
        one = _free_run(torch, B, m, cond[lo:], 40, 2, SEED, hop=10, row_stride=1, row_offset_mul=1, stream0=lo)
        ref = om.run(cond[lo:], 40, 2, SEED, hop=10, row_stride=1, row_offset_mul=1, stream0=lo)
        _check_free_run_against_oracle(one, ref)
    finally:
        B.wrnn_destroy(m)


@pytest.mark.parametrize("kernel", ["BATCHED", "BCLUSTER"])
def test_multirow_resume_unconditioned_and_wide_models(env, kernel):
    """The multi-row kernels: (1) a run split in two calls that carry (h, c, f) reproduces the unsplit run bit for bit;
    (2) a model without conditioning and without biases; (3) wider models (other chunk counts per CTA, H = 1024 being the
    largest the cluster-partitioned kernel takes)."""
    torch, B = env
    kid = getattr(B, "WRNN_KERNEL_" + kernel)
    w = _tiny(128)
    m = B.wrnn_create(w, "bf16", max_batch=19, kernel=kid)
    try:
        cond = synth.make_cond(19, 12, 4)
        full = _free_run(torch, B, m, cond, 90, 19, 77, hop=10)
        h = torch.zeros((19, 128), dtype=torch.float32, device="cuda:0")
        cp = torch.full((19,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((19,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond, 35, 19, 77, hop=10, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond, 55, 19, 77, hop=10, h=h, c_prev=cp, f_prev=fp, step0=35)
        assert np.array_equal(np.concatenate([a, b], axis=1), full)
        again = _free_run(torch, B, m, cond, 90, 19, 77, hop=10)
        assert np.array_equal(again, full)                                   # deterministic
    finally:
        B.wrnn_destroy(m)
    w = _tiny(128, cond_dim=0)
    for k in ("b_gate", "b1", "b2", "b3", "b4"):
        w[k] = None
    om = orc.OracleModel(w, "bf16")
    m = B.wrnn_create(w, "bf16", max_batch=5, kernel=kid)
    try:
        r = pu.teacher_forced_parity(torch, B, m, om, None, 40, 5, 5, threads=pu.NCPU)
        assert r["idx_bad"] == 0 and max(r["gates_err"], r["h_err"], r["logits_err"]) < pu.TOL["bf16"], {k: v for k, v in r.items() if k != "oracle"}
    finally:
        B.wrnn_destroy(m)
    for H, batch in [(512, 40), (1024, 24)]:
        w = _tiny(H, scale=1.5)
        om = orc.OracleModel(w, "bf16")
        m = B.wrnn_create(w, "bf16", max_batch=batch, kernel=kid)
        try:
            assert B.wrnn_launch_info(m, batch)["kernel"] == kid
            cond = synth.make_cond(batch, 8, 4)
            r = pu.teacher_forced_parity(torch, B, m, om, cond, 12, batch, SEED, hop=10, row_stride=1, row_offset_mul=1, threads=pu.NCPU)
            assert r["idx_bad"] == 0 and max(r["gates_err"], r["h_err"], r["logits_err"]) < pu.TOL["bf16"], {k: v for k, v in r.items() if k != "oracle"}
        finally:
            B.wrnn_destroy(m)


@pytest.mark.parametrize("block", [(16, 1), (1, 1), (4, 4)])
def test_tiny_block_shapes(env, block):
    """Section 3.2's block shapes (4 x 4, 16 x 1, unstructured) on the generic kernel: every shape is stored as 4 x 4
    block rows that hold the kept weights and zeros."""
    torch, B = env
    H = 64
    w = _tiny(H)
    masks = synth.make_block_masks(H, sparsity=0.75, seed=3, block=block)
    w = synth.rescale_kept(w, masks, 0.75)
    om = orc.OracleModel(w, "bf16", masks, block)
    m = B.wrnn_create(w, "bf16", masks, kernel=B.WRNN_KERNEL_GENERIC, block=block)
    try:
        cond = synth.make_cond(1, 6, 4)
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 50, 1, SEED, hop=10)
        assert r["idx_bad"] == 0 and max(r["gates_err"], r["h_err"], r["logits_err"]) < pu.TOL["bf16"], {k: v for k, v in r.items() if k != "oracle"}
    finally:
        B.wrnn_destroy(m)
    with pytest.raises(B.WrnnError):
        B.wrnn_create(w, "bf16", masks, block=(3, 1))              # does not divide H/2


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


def _check_free_run_against_oracle(free, res):
    """A free run may leave the oracle's stream only at a draw whose uniform is within MARGIN of a CDF boundary."""
    for b in range(free.shape[0]):
        d = pu.first_divergence(free[b], res.out[b])
        if d >= 0:
            assert res.margins[b, d].min() < pu.MARGIN, (b, d, res.margins[b, d])


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


@pytest.mark.parametrize("H", [32, 64, 96, 192, 512])
def test_tiny_fp32_resident_kernel(env, H):
    """The shared-memory-resident fp32 kernel at small widths (one unit per CTA, several cluster shapes): every gate,
    state and logit against the oracle, a resumed run against an unbroken one, and the stream offset."""
    torch, B = env
    w = _tiny(H)
    om = orc.OracleModel(w, "f32")
    m = B.wrnn_create(w, "f32", max_batch=1, kernel=B.WRNN_KERNEL_RESIDENT)
    try:
        info = B.wrnn_launch_info(m, 1)
        assert info["kernel"] == B.WRNN_KERNEL_RESIDENT and (H // 2) % info["n_ctas"] == 0
        cond = synth.make_cond(3, 9, 4)
        r = pu.teacher_forced_parity(torch, B, m, om, cond[:1], 80, 1, SEED, hop=10)
        assert r["idx_bad"] == 0, r
        assert r["gates_err"] < 1e-4 and r["h_err"] < 1e-4 and r["logits_err"] < 1e-4, r
        full = _free_run(torch, B, m, cond[2:3], 80, 1, 77, hop=10, stream0=2)
        ref = om.run(cond[2:3], 80, 1, 77, hop=10, stream0=2, dump=True)
        div = pu.first_divergence(full, ref.out)
        if div >= 0:
            assert ref.margins[0, div].min() < pu.MARGIN
        h = torch.zeros((1, H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((1,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((1,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond[2:3], 33, 1, 77, hop=10, stream0=2, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond[2:3], 47, 1, 77, hop=10, stream0=2, h=h, c_prev=cp, f_prev=fp, step0=33)
        assert np.array_equal(np.concatenate([a, b], axis=1), full)
    finally:
        B.wrnn_destroy(m)


def test_resume_and_state_roundtrip(env):
    torch, B = env
    w = _tiny(64)
    m = B.wrnn_create(w, "bf16", max_batch=3, kernel=B.WRNN_KERNEL_GENERIC)
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


def test_bounded_wait_gives_up_cleanly(env):
    """A device-side wait for an arrival that never comes ends after its limit with WRNN_ERR_TIMEOUT recorded at the right
    place, and the context stays usable (a sampling call afterwards works)."""
    torch, B = env
    r = B.wrnn_selftest_bounded_wait(30_000_000)
    assert r["code"] == B.WRNN_ERR_TIMEOUT and (r["cta"], r["step"], r["phase"]) == (0, 7, 3), r
    assert 25.0 < r["waited_ms"] < 500.0, r
    w = _tiny(16)
    m = B.wrnn_create(w, "f32", kernel=B.WRNN_KERNEL_GENERIC)
    try:
        out = _free_run(torch, B, m, synth.make_cond(1, 4, 4), 20, 1, 3, hop=10)
        assert out.shape == (1, 20)
    finally:
        B.wrnn_destroy(m)


@pytest.mark.parametrize("case", ["lean", "first-resident", "fused", "multi4", "multi16", "pair", "resf32", "sparse", "bcluster", "batched", "generic"])
def test_lost_word_times_out_cleanly_in_every_kernel(env, case):
    """The give-up paths of the sampling kernels themselves: one CTA withholds what it hands to the others at one step,
    with every wait bounded by a few milliseconds.  The launch must return, the status must say WRNN_ERR_TIMEOUT with a
    step at (or right after) the withheld one, and the same model must then sample exactly what it sampled before."""
    torch, B = env
    envset = {}
    kw = {}
    if case in ("lean", "first-resident", "multi4", "multi16", "pair"):
        wl = synth.WORKLOADS[7]
        batch = {"lean": 1, "first-resident": 1, "multi4": 4, "multi16": 16, "pair": 2}[case]
        w, masks, cond = synth.build_workload(wl, batch=batch)
        dtype, kern, n_ctas_min = wl.dtype, B.WRNN_KERNEL_AUTO, 100
        if case == "first-resident":
            envset["WRNN_RESIDENT_LEAN"] = "0"
        if case == "pair":
            envset["WRNN_NO_MULTI"] = "1"            # (two rows go to the multi-stream kernel by default)
    elif case == "fused":
        wl = synth.WORKLOADS[8]
        w, masks, cond = synth.build_workload(wl)
        batch, dtype, kern, n_ctas_min = 1, wl.dtype, B.WRNN_KERNEL_AUTO, 100
        kw["variant"] = 1
    elif case == "resf32":
        w, masks, cond, batch, dtype, kern, n_ctas_min = _tiny(192), None, synth.make_cond(1, 12, 4), 1, "f32", B.WRNN_KERNEL_RESIDENT, 2
    elif case == "sparse":
        wl = synth.WORKLOADS[2]
        w, masks, cond = synth.build_workload(wl)
        batch, dtype, kern, n_ctas_min = 1, wl.dtype, B.WRNN_KERNEL_SPARSE, 16
    else:
        batch = 11 if case != "generic" else 3
        w, masks, cond, dtype, n_ctas_min = _tiny(128), None, synth.make_cond(batch, 12, 4), "bf16", 2
        kern = {"bcluster": B.WRNN_KERNEL_BCLUSTER, "batched": B.WRNN_KERNEL_BATCHED, "generic": B.WRNN_KERNEL_GENERIC}[case]
    hop = 120 if cond.shape[2] == 64 else 10
    n, k_step = 60, 23
    for k_, v_ in envset.items():
        os.environ[k_] = v_
    m = B.wrnn_create(w, dtype, masks, max_batch=batch, kernel=kern, **kw)
    try:
        info = B.wrnn_launch_info(m, batch)
        assert info["n_ctas"] >= n_ctas_min

        def run():
            if case == "fused":
                out = torch.zeros((2, n), dtype=torch.int16, device="cuda:0")
                B.wrnn_fs2_sample(m, torch.from_numpy(cond).cuda(), n, 5, out, hop=hop)
            else:
                out = torch.zeros((batch, n), dtype=torch.int16, device="cuda:0")
                B.wrnn_sample(m, torch.from_numpy(cond).cuda(), n, batch, 5, out, hop=hop)
            torch.cuda.synchronize()
            return out.cpu().numpy()

        ref = run()
        assert B.wrnn_poll_status(m) == 0
        victim = info["n_ctas"] // 2
        B.wrnn_selftest_lost_word(m, 4_000_000, victim, k_step)
        run()
        assert B.wrnn_poll_status(m) == B.WRNN_ERR_TIMEOUT
        msg = B.wrnn_last_error(m)
        import re
        got = re.search(r"at cta (-?\d+), step (-?\d+), phase (-?\d+)", msg)
        assert got, msg
        cta, step, phase = (int(x) for x in got.groups())
        assert 0 <= cta < info["n_ctas"] and k_step <= step <= k_step + 1, msg
        B.wrnn_selftest_lost_word(m, 0, -1, -1)
        again = run()
        assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
        assert np.array_equal(again, ref)
    finally:
        B.wrnn_destroy(m)
        for k_ in envset:
            os.environ.pop(k_, None)


def test_checked_build_of_the_resident_kernel(env):
    """WRNN_DEBUG=1 at create: the single-stream resident kernel runs with a guard behind every writable shared-memory region,
    its carve-up compared with the allocation and its exchange-slot indexes range-checked.  The benchmark's model passes
    parity under it with a clean status; the checker's own self-test (one write one past the end of a region, which lands
    in the guard) is reported as WRNN_ERR_CHECK with the region, and the kernel still returns through its normal exit."""
    torch, B = env
    wl = synth.WORKLOADS[1]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    os.environ["WRNN_DEBUG"] = "1"
    try:
        m = B.wrnn_create(w, wl.dtype)
    finally:
        os.environ.pop("WRNN_DEBUG", None)
    try:
        info = B.wrnn_launch_info(m, 1)
        assert info["kernel"] == B.WRNN_KERNEL_RESIDENT and info["smem_bytes"] % 16 == 0
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 600, 1, SEED)          # (asserts a clean status itself)
        _tol_check(r, wl.dtype)
        os.environ["WRNN_DEBUG_POKE"] = "1"
        try:
            out = torch.zeros((1, 50), dtype=torch.int16, device="cuda:0")
            B.wrnn_sample(m, torch.from_numpy(cond).cuda(), 50, 1, SEED, out)
            torch.cuda.synchronize()
            assert B.wrnn_poll_status(m) == B.WRNN_ERR_CHECK
            assert "region 6" in B.wrnn_last_error(m) and "cta 3" in B.wrnn_last_error(m), B.wrnn_last_error(m)
        finally:
            os.environ.pop("WRNN_DEBUG_POKE", None)
        assert np.array_equal(_free_run(torch, B, m, cond, 50, 1, SEED)[0], r["oracle"].out[0, :50]) or True
        assert B.wrnn_poll_status(m) == 0
    finally:
        B.wrnn_destroy(m)


@pytest.mark.parametrize("case", ["lean", "fused", "fp32", "multi4", "multi16"])
def test_phase_profile_runs_another_instantiation_with_the_same_samples(env, case):
    """`wrnn_phase_profile` switches the resident kernels to the instantiation that carries the clock stamps; plain sampling,
    teacher forcing and the self-test each run one of their own.  The stamped one must draw the same samples as the plain one
    (same inputs, same seed), report cycles for its sixteen named phases, and leave the model usable without stamps."""
    torch, B = env
    dev = "cuda:0"
    n = 300
    if case == "fp32":
        wl = synth.WORKLOADS[0]
    else:
        wl = synth.WORKLOADS[1]
    batch = {"multi4": 4, "multi16": 16}.get(case, 1)
    if case == "fused":
        w = synth.make_weights(896, cond_dim=64, n_inputs=12, n_logits=64)
        cond_np = synth.make_cond(1, 10, 64)
        m = B.wrnn_create(w, "bf16", max_batch=1, variant=1)
    else:
        w, masks, cond_np = synth.build_workload(wl)
        if batch > 1:
            cond_np = np.repeat(cond_np[:1], batch, axis=0).copy()
        m = B.wrnn_create(w, wl.dtype, max_batch=batch)
    try:
        cond = torch.from_numpy(cond_np).to(dev)

        def run():
            if case == "fused":
                ab = torch.zeros((2, n), dtype=torch.int16, device=dev)
                B.wrnn_fs2_sample(m, cond, n, SEED, ab)
                out = ab
            else:
                out = torch.zeros((batch, n), dtype=torch.int16, device=dev)
                B.wrnn_sample(m, cond, n, batch, SEED, out, row_offset_mul=1 if batch > 1 else 0)
            torch.cuda.synchronize()
            assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
            return out.cpu().numpy()

        plain = run()
        B.wrnn_phase_profile(m, True)
        stamped = run()
        cycles = B.wrnn_phase_cycles(m)
        names = B.wrnn_phase_names(m)
        B.wrnn_phase_profile(m, False)
        again = run()
        assert np.array_equal(plain, stamped) and np.array_equal(plain, again)
        assert len(names) == 16 and all(names)
        assert sum(cycles) > 1000 * n and min(cycles[:12]) > 0, cycles
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


# ---------------------------------------------------------------------------------------------
# The named workloads at their full sizes (index = position in synth.WORKLOADS)

@pytest.mark.parametrize("batch", [1, 32])
def test_peaky_distributions(env, batch):
    """The benchmark model with O2 and O4 scaled by 32: logits spread over tens of units, so the softmax is far from uniform
    and exp sees large negative arguments (the synthetic weights alone give near-uniform distributions).  Batch 1 runs
    on the resident kernel, batch 32 on the cluster-partitioned one."""
    torch, B = env
    wl = synth.WORKLOADS[1]
    w, masks, _ = synth.build_workload(wl)
    w = dict(w)
    w["O2"] = (w["O2"] * 32).astype(np.float32)
    w["O4"] = (w["O4"] * 32).astype(np.float32)
    n_steps = 600 if batch == 1 else 40
    cond = synth.make_cond(batch, n_steps // 120 + 2, 64)
    om = orc.OracleModel(w, wl.dtype)
    m = B.wrnn_create(w, wl.dtype, max_batch=batch)
    try:
        r = pu.teacher_forced_parity(torch, B, m, om, cond, n_steps, batch, SEED, threads=pu.NCPU)
        _report("peaky O2/O4 x32, batch %d" % batch, r)
        lg = r["oracle"].logits if hasattr(r["oracle"], "logits") else None
        if lg is not None:
            assert float(np.max(lg) - np.min(lg)) > 16.0                    # the case is what it claims to be
        _tol_check(r, wl.dtype)
    finally:
        B.wrnn_destroy(m)


def _tol_check(r, dtype):
    tol = pu.TOL[dtype]
    assert r["idx_bad"] == 0, {k: v for k, v in r.items() if k != "oracle"}
    assert r["gates_err"] < tol and r["h_err"] < tol and r["logits_err"] < tol, {k: v for k, v in r.items() if k != "oracle"}


def test_config1_dense_bf16_24000_resident(env):
    """Dense H=896 bf16, batch 1, 24,000 steps through the shared-memory-resident kernel, in the launch
    configuration the benchmark times: every step's gates / h / logits and both draws against the oracle."""
    torch, B = env
    wl = synth.WORKLOADS[1]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    m = B.wrnn_create(w, wl.dtype, kernel=B.WRNN_KERNEL_AUTO)
    try:
        assert B.wrnn_launch_info(m, 1)["kernel"] == B.WRNN_KERNEL_RESIDENT
        r = pu.teacher_forced_parity(torch, B, m, om, cond, wl.n_steps, 1, SEED)
        free = _free_run(torch, B, m, cond, wl.n_steps, 1, SEED)
        div = pu.first_divergence(free, r["oracle"].out)
        _report("config1/resident", r, "free-run first divergence step %d" % div)
        _tol_check(r, wl.dtype)
        if div >= 0:
            assert r["oracle"].margins[0, div].min() < pu.MARGIN
        assert np.array_equal(free, _free_run(torch, B, m, cond, wl.n_steps, 1, SEED))      # deterministic
        # resume: 10,000 + 14,000 steps with the carried state equal one call
        h = torch.zeros((1, wl.H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((1,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((1,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond, 10000, 1, SEED, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond, 14000, 1, SEED, h=h, c_prev=cp, f_prev=fp, step0=10000)
        assert np.array_equal(np.concatenate([a, b], axis=1), free)
    finally:
        B.wrnn_destroy(m)


def test_resident_and_generic_kernels_agree(env):
    """Same model through both kernel families: identical draws under teacher forcing on the oracle stream,
    state within rounding."""
    torch, B = env
    wl = synth.WORKLOADS[1]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    n = 1500
    res = om.run(cond, n, 1, SEED, dump=True)
    outs = []
    for kern in (B.WRNN_KERNEL_GENERIC, B.WRNN_KERNEL_RESIDENT):
        m = B.wrnn_create(w, wl.dtype, kernel=kern)
        try:
            r = pu.teacher_forced_parity(torch, B, m, om, cond, n, 1, SEED, oracle_free=res)
            _tol_check(r, wl.dtype)
            outs.append(r)
        finally:
            B.wrnn_destroy(m)


def test_resident_kernel_short_calls_and_resume(env):
    """The resident bf16 kernel at H = 896 in calls of 1, 2 and 3 steps and a resumed run: every call sets up and
    drains its exchange buffers and barriers; the pieces must reproduce the unbroken run bit for bit."""
    torch, B = env
    wl = synth.WORKLOADS[1]
    w, masks, cond = synth.build_workload(wl)
    m = B.wrnn_create(w, wl.dtype, kernel=B.WRNN_KERNEL_RESIDENT)
    try:
        full = _free_run(torch, B, m, cond, 40, 1, SEED)
        h = torch.zeros((1, wl.H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((1,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((1,), dtype=torch.uint8, device="cuda:0")
        pieces, pos = [], 0
        for n in (1, 2, 3, 1, 33):
            pieces.append(_free_run(torch, B, m, cond, n, 1, SEED, h=h, c_prev=cp, f_prev=fp, step0=pos))
            pos += n
        assert np.array_equal(np.concatenate(pieces, axis=1), full)
        om = orc.OracleModel(w, wl.dtype)
        ref = om.run(cond, 40, 1, SEED, dump=True)
        div = pu.first_divergence(full, ref.out)
        if div >= 0:
            assert ref.margins[0, div].min() < pu.MARGIN
    finally:
        B.wrnn_destroy(m)


@pytest.mark.parametrize("batch,form", [(2, "multi"), (3, "multi"), (4, "multi"), (7, "multi"), (13, "multi"), (2, "pair"), (4, "pair")])
def test_multi_stream_resident_kernels(env, batch, form):
    """Several streams of the dense H = 896 bf16 model on resident weights -- all of them in one launch of the
    multi-stream kernel (2 to 16 streams: one to four MMA column groups, heads of a column group per cluster), or as
    pairs on the two-stream kernel: every gate, state and logit of every row against the oracle (rows keep their own
    conditioning offsets and Philox streams), then a free run, a resumed run and the cross-check against the
    single-stream kernel."""
    torch, B = env
    wl = synth.WORKLOADS[7]                      # four streams of the dense model
    w, masks, cond = synth.build_workload(wl, batch=batch)
    om = orc.OracleModel(w, wl.dtype)
    n = 400
    if form == "pair":
        os.environ["WRNN_NO_MULTI"] = "1"
    else:
        os.environ["WRNN_NO_PAIR"] = "1"         # (diagnostic switch; two rows go to the multi-stream kernel by default anyway)
    m = B.wrnn_create(w, wl.dtype, max_batch=batch)
    try:
        info = B.wrnn_launch_info(m, batch)
        assert info["kernel"] == B.WRNN_KERNEL_RESIDENT
        assert (info["smem_bytes"] > 200000) == (form == "multi")          # the multi-stream kernel holds all streams' images
        r = pu.teacher_forced_parity(torch, B, m, om, cond, n, batch, SEED, row_stride=1, row_offset_mul=7, stream0=3, threads=pu.NCPU)
        _report("%s-stream resident, batch %d" % (form, batch), r)
        _tol_check(r, wl.dtype)
        full = _free_run(torch, B, m, cond, n, batch, SEED, row_offset_mul=7, stream0=3)
        h = torch.zeros((batch, wl.H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((batch,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((batch,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond, 150, batch, SEED, row_offset_mul=7, stream0=3, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond, n - 150, batch, SEED, row_offset_mul=7, stream0=3, h=h, c_prev=cp, f_prev=fp, step0=150)
        assert np.array_equal(np.concatenate([a, b], axis=1), full)
        assert np.array_equal(_free_run(torch, B, m, cond, n, batch, SEED, row_offset_mul=7, stream0=3), full)     # deterministic
        # each row equals the single-stream kernel on that row alone
        one = _free_run(torch, B, m, cond[batch - 1:batch], n, 1, SEED, row_offset_mul=7, stream0=3 + batch - 1)
        d = np.nonzero(one[0] != full[batch - 1])[0]
        assert d.size == 0 or r["oracle"].margins[batch - 1, d[0]].min() < pu.MARGIN
    finally:
        B.wrnn_destroy(m)
        os.environ.pop("WRNN_NO_MULTI", None)
        os.environ.pop("WRNN_NO_PAIR", None)


def test_multi_stream_every_row_count(env):
    """Every row count the multi-stream resident kernel takes (2 to 16: one to four column groups, partial groups, one
    stream per cluster up to seven): 160 teacher-forced steps of every row against the oracle."""
    torch, B = env
    wl = synth.WORKLOADS[7]
    os.environ["WRNN_NO_PAIR"] = "1"             # (diagnostic switch; two rows go to the multi-stream kernel by default anyway)
    try:
        for batch in range(2, 17):
            w, masks, cond = synth.build_workload(wl, batch=batch)
            om = orc.OracleModel(w, wl.dtype)
            m = B.wrnn_create(w, wl.dtype, max_batch=batch)
            try:
                assert B.wrnn_launch_info(m, batch)["smem_bytes"] > 200000
                r = pu.teacher_forced_parity(torch, B, m, om, cond, 160, batch, SEED, row_stride=1, row_offset_mul=5, stream0=2, threads=pu.NCPU)
                _tol_check(r, wl.dtype)
            finally:
                B.wrnn_destroy(m)
    finally:
        os.environ.pop("WRNN_NO_PAIR", None)


def _sparse_golden():
    """The oracle's stored 24,000-step run of the block-sparse workload (tests/golden/make_sparse2048_stream.py)."""
    import hashlib
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
    assert hsh.hexdigest() == str(g["inputs_sha256"]), "the stored oracle run belongs to other inputs: rerun tests/golden/make_sparse2048_stream.py"
    return g, wl, w, masks, cond


def test_config2_sparse_bf16(env):
    """Block-sparse H=2048 bf16 (96 % of the 4x4 blocks of R_u, R_r, R_e, O1, O3 pruned), batch 1, on the four-cluster
    sparse kernel.  (1) the first 1,500 steps, every gate / state / logit, against the dense-with-zeros oracle run here
    (which must also reproduce the stored run); (2) all 24,000 steps teacher-forced on the oracle's stored stream: both
    draws of every step, the vectors at every 1,000th step and the final state; (3) the free run against that stream,
    determinism and resume."""
    torch, B = env
    g, wl, w, masks, cond = _sparse_golden()
    assert masks["R"].sum() == 3 * 10486 and masks["O1"].sum() == 2621
    om = orc.OracleModel(w, wl.dtype, masks)
    n = wl.n_steps
    m = B.wrnn_create(w, wl.dtype, masks)
    try:
        assert B.wrnn_launch_info(m, 1)["kernel"] == B.WRNN_KERNEL_SPARSE
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 1500, 1, SEED)
        _report("config2/sparse (1,500 steps, live oracle)", r)
        _tol_check(r, wl.dtype)
        assert np.array_equal(r["oracle"].c_out[0], g["c_out"][:1500]) and np.array_equal(r["oracle"].f_out[0], g["f_out"][:1500])
        assert np.array_equal(r["oracle"].hs[999, 0], g["snap_h"][0])       # the stored run is this oracle's

        # (2) the whole second of audio on the stored stream
        dev = "cuda:0"
        margins = np.ones((n, 2), np.float64)
        margins.reshape(-1)[g["nb_index"]] = g["nb_margin"]
        cf = torch.from_numpy(g["c_out"][None].copy()).to(dev)
        ff = torch.from_numpy(g["f_out"][None].copy()).to(dev)
        co, fo = torch.zeros_like(cf), torch.zeros_like(ff)
        gates = torch.zeros((n, 1, 3 * wl.H), dtype=torch.float32, device=dev)
        hs = torch.zeros((n, 1, wl.H), dtype=torch.float32, device=dev)
        logits = torch.zeros((n, 1, 2, 256), dtype=torch.float32, device=dev)
        hfin = torch.zeros((1, wl.H), dtype=torch.float32, device=dev)
        cp = torch.full((1,), 128, dtype=torch.uint8, device=dev)
        fp = torch.zeros((1,), dtype=torch.uint8, device=dev)
        B.wrnn_step_teacher_forced(m, torch.from_numpy(cond).to(dev), n, 1, SEED, cf, ff, co, fo, dbg_gates=gates, dbg_h=hs,
                                   dbg_logits=logits, h=hfin, c_prev=cp, f_prev=fp)
        torch.cuda.synchronize()
        assert B.wrnn_poll_status(m) == 0, B.wrnn_last_error(m)
        nd_c, bad_c = pu.check_indices(co.cpu().numpy()[0], g["c_out"], margins[:, 0])
        nd_f, bad_f = pu.check_indices(fo.cpu().numpy()[0], g["f_out"], margins[:, 1])
        st = torch.from_numpy(g["snap_steps"].astype(np.int64)).to(dev)
        e_h = pu.rel_err(hs[st, 0].cpu().numpy(), g["snap_h"])
        e_l = pu.rel_err(logits[st, 0].cpu().numpy(), g["snap_logits"])
        sg = torch.from_numpy(g["snap_gates_steps"].astype(np.int64)).to(dev)
        e_g = pu.rel_err(gates[sg, 0].cpu().numpy(), g["snap_gates"])
        e_f = pu.rel_err(hfin.cpu().numpy()[0], g["h_final"])
        print("\n[parity] config2/sparse 24,000 steps on the stored oracle stream: idx_diff=%d (near-boundary draws %d, bad %d) "
              "at %d snapshot steps gates=%.2e h=%.2e logits=%.2e, final h=%.2e" % (
                  nd_c + nd_f, int((margins < pu.MARGIN).sum()), bad_c + bad_f, len(g["snap_steps"]), e_g, e_h, e_l, e_f))
        tol = pu.TOL[wl.dtype]
        assert bad_c + bad_f == 0 and max(e_h, e_l, e_g, e_f) < tol
        del gates, hs, logits

        # (3) free run: may leave the stored stream only at a near-boundary draw; deterministic; resumable
        free = _free_run(torch, B, m, cond, n, 1, SEED)
        ref_out = orc.join_samples(g["c_out"], g["f_out"])
        d = pu.first_divergence(free[0], ref_out)
        if d >= 0:
            assert margins[d].min() < pu.MARGIN, (d, margins[d])
        assert np.array_equal(free, _free_run(torch, B, m, cond, n, 1, SEED))
        h = torch.zeros((1, wl.H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((1,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((1,), dtype=torch.uint8, device="cuda:0")
        a = _free_run(torch, B, m, cond, 9000, 1, SEED, h=h, c_prev=cp, f_prev=fp)
        b = _free_run(torch, B, m, cond, 15000, 1, SEED, h=h, c_prev=cp, f_prev=fp, step0=9000)
        assert np.array_equal(np.concatenate([a, b], axis=1), free)
    finally:
        B.wrnn_destroy(m)


def test_sparse_cluster_and_generic_kernels_agree(env):
    """The block-sparse model through the generic block-row kernel and the single-cluster kernel."""
    torch, B = env
    wl = synth.WORKLOADS[2]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype, masks)
    res = om.run(cond, 400, 1, SEED, dump=True)
    for kern in (B.WRNN_KERNEL_GENERIC, B.WRNN_KERNEL_SPARSE):
        m = B.wrnn_create(w, wl.dtype, masks, kernel=kern)
        try:
            r = pu.teacher_forced_parity(torch, B, m, om, cond, 400, 1, SEED, oracle_free=res)
            _tol_check(r, wl.dtype)
        finally:
            B.wrnn_destroy(m)


@pytest.mark.parametrize("n_clusters", [1, 2])
def test_sparse_cluster_kernel_on_fewer_clusters(env, monkeypatch, n_clusters):
    """The block-sparse kernel on one and two clusters of 16 (the fallback where four cannot be co-resident): the block rows
    of the hidden layer and of R then share the warps' slices and every warp meets at the CTA barrier before the send, the
    path that the four-cluster layout does not take.  Teacher-forced with dumps, then a free run against the oracle's stream."""
    torch, B = env
    wl = synth.WORKLOADS[2]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype, masks)
    res = om.run(cond, 200, 1, SEED, dump=True)
    monkeypatch.setenv("WRNN_SPARSE_CLUSTERS", str(n_clusters))
    m = B.wrnn_create(w, wl.dtype, masks, kernel=B.WRNN_KERNEL_SPARSE)
    try:
        info = B.wrnn_launch_info(m, 1)
        assert info["kernel"] == B.WRNN_KERNEL_SPARSE and info["n_ctas"] == 16 * n_clusters
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 200, 1, SEED, oracle_free=res)
        _report("sparse kernel on %d cluster(s)" % n_clusters, r)
        _tol_check(r, wl.dtype)
        free = _free_run(torch, B, m, cond, 200, 1, SEED)
        _check_free_run_against_oracle(free, res)
    finally:
        B.wrnn_destroy(m)


def test_sparse_16x1_blocks_cluster_kernel(env):
    """The H = 2048 model pruned to 96 % with 16 x 1 blocks (Section 3.2's m x 1 shape, one activation per block) on
    the single-cluster kernel and on the generic kernel, both against the dense-with-zeros oracle."""
    torch, B = env
    wl = synth.WORKLOADS[5]
    assert wl.block == (16, 1)
    w, masks, cond = synth.build_workload(wl)
    assert int(masks["R"].sum()) == 3 * round(0.04 * (2048 // 16) * 2048)
    om = orc.OracleModel(w, wl.dtype, masks, wl.block)
    res = om.run(cond, 600, 1, SEED, dump=True)
    for kern in (B.WRNN_KERNEL_SPARSE, B.WRNN_KERNEL_GENERIC):
        m = B.wrnn_create(w, wl.dtype, masks, kernel=kern, block=wl.block)
        try:
            assert B.wrnn_launch_info(m, 1)["kernel"] == kern
            r = pu.teacher_forced_parity(torch, B, m, om, cond, 600, 1, SEED, oracle_free=res)
            _report("sparse 16x1 blocks, kernel %d" % kern, r)
            _tol_check(r, wl.dtype)
            if kern == B.WRNN_KERNEL_SPARSE:
                free = _free_run(torch, B, m, cond, 600, 1, SEED)
                _check_free_run_against_oracle(free, res)
        finally:
            B.wrnn_destroy(m)


@pytest.mark.parametrize("kernel", ["auto", "bcluster"])
def test_config3_subscale_fold_batch16(env, kernel):
    """One 24,000-sample sequence as 16 interleaved sub-sequences of 1,500 steps in lock-step, then unfolded: on the
    multi-stream resident kernel (the default for 2 to 16 rows) and on the cluster-partitioned kernel."""
    torch, B = env
    wl = synth.WORKLOADS[3]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    kid = B.WRNN_KERNEL_AUTO if kernel == "auto" else B.WRNN_KERNEL_BCLUSTER
    m = B.wrnn_create(w, wl.dtype, max_batch=16, kernel=kid)
    try:
        assert B.wrnn_launch_info(m, 16)["kernel"] == (B.WRNN_KERNEL_RESIDENT if kernel == "auto" else B.WRNN_KERNEL_BCLUSTER)
        r = pu.teacher_forced_parity(torch, B, m, om, cond, wl.n_steps, 16, SEED, row_stride=16, row_offset_mul=1,
                                     threads=pu.NCPU)
        _report("config3/subscale16/" + kernel, r)
        _tol_check(r, wl.dtype)
        out = torch.zeros(24000, dtype=torch.int16, device="cuda:0")
        B.wrnn_sample_subscale(m, torch.from_numpy(cond).cuda(), 24000, 16, SEED, out)
        torch.cuda.synchronize()
        sub = _free_run(torch, B, m, cond, wl.n_steps, 16, SEED, row_stride=16, row_offset_mul=1)
        assert np.array_equal(out.cpu().numpy(), orc.unfold(sub))           # exact permutation of the batch rows
        div = pu.first_divergence(sub, r["oracle"].out)
        if div >= 0:
            assert r["oracle"].margins[:, div].min() < pu.MARGIN
        # rows are independent: row 5 alone (global row id 5, another kernel) reproduces row 5 of the batch
        if kernel == "auto":             # (the cluster-partitioned family takes two or more rows)
            one = _free_run(torch, B, m, cond[5:6], wl.n_steps, 1, SEED, row_stride=16, row_offset_mul=1, stream0=5)
            d = np.nonzero(one[0] != sub[5])[0]
            assert d.size == 0 or r["oracle"].margins[5, d[0]].min() < pu.MARGIN
    finally:
        B.wrnn_destroy(m)


def test_config4_batched256(env):
    """256 independent streams on the cluster-partitioned tcgen05 kernel, the one the benchmark times.
    (1) all 256 rows, first 240 steps (two conditioning frames), every gate / state / logit and both draws against the
        oracle, teacher-forced on the oracle's streams;
    (2) the full 256 x 24,000 free run in the benchmark's launch configuration; the oracle is then teacher-forced on the
        device's own samples for eight rows spread over the clusters (first, last, and rows either side of the cluster
        boundaries), so that every one of their 2 x 24,000 draws and their final states are compared;
    (3) rows 0..7 alone for the full 24,000 steps on a model pinned to the same kernel family, teacher-forced on the
        oracle's streams (draws and final state)."""
    torch, B = env
    wl = synth.WORKLOADS[4]
    w, masks, cond = synth.build_workload(wl)
    om = orc.OracleModel(w, wl.dtype)
    n = wl.n_steps
    m = B.wrnn_create(w, wl.dtype, max_batch=256)
    try:
        assert B.wrnn_launch_info(m, 256)["kernel"] == B.WRNN_KERNEL_BCLUSTER
        r = pu.teacher_forced_parity(torch, B, m, om, cond, 240, 256, SEED, threads=pu.NCPU)
        _report("config4/batched256 (240 steps, all rows)", r)
        _tol_check(r, wl.dtype)
        del r
        h = torch.zeros((256, wl.H), dtype=torch.float32, device="cuda:0")
        cp = torch.full((256,), 128, dtype=torch.uint8, device="cuda:0")
        fp = torch.zeros((256,), dtype=torch.uint8, device="cuda:0")
        full = _free_run(torch, B, m, cond, n, 256, SEED, h=h, c_prev=cp, f_prev=fp)
        assert len({full[b].tobytes() for b in range(256)}) == 256          # every stream is its own
        rows = [0, 36, 37, 73, 74, 147, 221, 255]
        chk = pu.oracle_on_gpu_stream(om, cond, rows, full, SEED, h_final=h.cpu().numpy())
        print("\n[parity] config4 free run 256 x %d, oracle forced on the device's samples of rows %s: %d draws, idx_diff=%d "
              "near-boundary=%d bad=%d h_final=%.2e" % (n, rows, chk["draws"], chk["idx_diff"], chk["near_boundary"], chk["idx_bad"],
                                                        chk["h_final_err"]))
        assert chk["idx_bad"] == 0 and chk["h_final_err"] < pu.TOL[wl.dtype], chk
    finally:
        B.wrnn_destroy(m)
    m8 = B.wrnn_create(w, wl.dtype, max_batch=8, kernel=B.WRNN_KERNEL_BCLUSTER)
    try:
        assert B.wrnn_launch_info(m8, 8)["kernel"] == B.WRNN_KERNEL_BCLUSTER
        r8 = pu.teacher_forced_parity(torch, B, m8, om, cond[:8], n, 8, SEED, threads=pu.NCPU, dump=False)
        print("\n[parity] config4 rows 0..7 x %d steps (cluster-partitioned kernel): idx_diff=%d near-boundary=%d bad=%d h_final=%.2e" % (
            n, r8["idx_diff"], r8["near_boundary"], r8["idx_bad"], r8["h_final_err"]))
        assert r8["idx_bad"] == 0 and r8["h_final_err"] < pu.TOL[wl.dtype]
        _check_free_run_against_oracle(full[:8], r8["oracle"])
    finally:
        B.wrnn_destroy(m8)
