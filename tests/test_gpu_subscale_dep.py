"""GPU parity of subscale generation with dependent rows on the staggered schedule (Sections 4.1, 4.2) against the CPU
oracle: the conditioning kernel element by element on the oracle's history, the staggered schedule against the
row-after-row order (which it must reproduce bit for bit, whatever the chunk and the lag), and the samples against the
oracle's up to the first near-boundary draw."""
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


def _case(H, B_rows, L, F, D=synth.COND_DIM, hop=synth.HOP, scale=1.0):
    w = synth.make_weights(H, cond_dim=D, seed_w=31, seed_b=32)
    if scale != 1.0:
        for k in ("R", "I", "O1", "O2", "O3", "O4", "W_cond"):
            w[k] = (w[k] * scale).astype(np.float32)
    V, b = synth.make_subscale_conv(B_rows, F, D)
    frames = synth.make_cond(B_rows, (B_rows * L) // hop + 2, D)
    return w, V, b, frames


def _gpu_run(torch, Bn, m, frames, V, b, F, chunk, lag, B_rows, L, hop=synth.HOP):
    dev = "cuda:0"
    out = torch.zeros((B_rows * L,), dtype=torch.int16, device=dev)
    Bn.wrnn_sample_subscale_dependent(m, torch.from_numpy(frames).to(dev), torch.from_numpy(V).to(dev), torch.from_numpy(b).to(dev), F, chunk,
                                      lag, B_rows * L, B_rows, SEED, out, hop=hop)
    torch.cuda.synchronize()
    assert Bn.wrnn_poll_status(m) == 0, Bn.wrnn_last_error(m)
    return out.cpu().numpy()


@pytest.mark.parametrize("H,dtype,B_rows,L,F,chunk,kernel", [
    (32, "f32", 4, 90, 6, 3, "generic"), (64, "bf16", 5, 64, 8, 8, "generic"), (896, "bf16", 16, 300, 32, 32, "generic"),
    (896, "bf16", 16, 300, 32, 32, "auto"),      # four or more active rows advance together on the multi-stream resident kernel
    (896, "bf16", 16, 300, 32, 32, "bcluster"),  # the same on the cluster-partitioned kernel (lone rows on the any-shape kernel)
])
def test_staggered_schedule_and_oracle(env, H, dtype, B_rows, L, F, chunk, kernel):
    torch, Bn = env
    w, V, b, frames = _case(H, B_rows, L, F, scale=2.0 if H < 100 else 1.0)
    om = orc.OracleModel(w, dtype)
    ref, cond_ref, margins = orc.subscale_dependent_run(om, frames, V, b, B_rows, L, synth.HOP, SEED)
    dev = "cuda:0"
    # the conditioning kernel on the oracle's history
    hist = torch.from_numpy(ref).to(dev)
    fr_d, V_d, b_d = torch.from_numpy(frames).to(dev), torch.from_numpy(V).to(dev), torch.from_numpy(b).to(dev)
    for row in range(B_rows):
        v = torch.zeros((L, synth.COND_DIM), dtype=torch.float32, device=dev)
        Bn.wrnn_subscale_conditioning(hist, fr_d, V_d, b_d, F, row, v)
        torch.cuda.synchronize()
        assert pu.rel_err(v.cpu().numpy(), cond_ref[row]) < 1e-5, row
    m = Bn.wrnn_create(w, dtype, max_batch=B_rows, kernel={"generic": Bn.WRNN_KERNEL_GENERIC, "auto": Bn.WRNN_KERNEL_AUTO,
                                                           "bcluster": Bn.WRNN_KERNEL_BCLUSTER}[kernel])
    try:
        if kernel != "generic":
            assert Bn.wrnn_launch_info(m, B_rows)["kernel"] == (Bn.WRNN_KERNEL_RESIDENT if kernel == "auto" else Bn.WRNN_KERNEL_BCLUSTER)
        lag = F + chunk if (F + chunk) % chunk == 0 else ((F + chunk + chunk - 1) // chunk) * chunk
        stag = _gpu_run(torch, Bn, m, frames, V, b, F, chunk, lag, B_rows, L)
        # row after row: a lag beyond the row length leaves one row active at a time
        seq_lag = ((L + F + chunk) // chunk + 1) * chunk
        seq = _gpu_run(torch, Bn, m, frames, V, b, F, chunk, seq_lag, B_rows, L)
        if kernel == "generic":      # one kernel family: the schedule cannot change a bit
            assert np.array_equal(stag, seq)
            # another chunk / lag: same samples
            if chunk % 2 == 0 and F % (chunk // 2) == 0:
                other = _gpu_run(torch, Bn, m, frames, V, b, F, chunk // 2, 2 * (F + chunk // 2), B_rows, L)
                assert np.array_equal(other, stag)
        # against the oracle, every row and every draw: the oracle generates in the order of Eq. 4 conditioned on the
        # DEVICE's samples (earlier rows through the conditioning network, the row's own past by teacher forcing) and
        # reports what it would have drawn; only near-boundary draws may differ, in any row
        got = orc.fold(stag, B_rows)
        want, _, mg = orc.subscale_dependent_run(om, frames, V, b, B_rows, L, synth.HOP, SEED, forced=got, teacher=True)
        gc, gf = pu._split(got)
        wc, wf = pu._split(want)
        nd_c, bad_c = pu.check_indices(gc, wc, mg[:, :, 0])
        nd_f, bad_f = pu.check_indices(gf, wf, mg[:, :, 1])
        print("\n[parity] dependent subscale H=%d %s: %d rows x %d positions, oracle forced on the device's samples: idx_diff=%d "
              "(near-boundary draws %d, bad %d)" % (H, kernel, B_rows, L, nd_c + nd_f, int((mg < pu.MARGIN).sum()), bad_c + bad_f))
        assert bad_c + bad_f == 0
        # and the free comparison with the oracle's own generation: the first difference, if any, at a near-boundary draw
        for row in range(B_rows):
            d = np.nonzero(got[row] != ref[row])[0]
            if d.size:
                assert margins[row, d[0]].min() < pu.MARGIN, (row, int(d[0]))
                break
    finally:
        Bn.wrnn_destroy(m)


def test_argument_errors(env):
    torch, Bn = env
    w, V, b, frames = _case(32, 4, 40, 4)
    m = Bn.wrnn_create(w, "f32", max_batch=4)
    dev = "cuda:0"
    out = torch.zeros((160,), dtype=torch.int16, device=dev)
    fr_d, V_d, b_d = torch.from_numpy(frames).to(dev), torch.from_numpy(V).to(dev), torch.from_numpy(b).to(dev)
    try:
        for (chunk, lag, B_rows) in ((4, 7, 4), (4, 6, 4), (4, 8, 5)):      # lag not a multiple / too small, B > max_batch
            with pytest.raises(Bn.WrnnError) as e:
                Bn.wrnn_sample_subscale_dependent(m, fr_d, V_d, b_d, 4, chunk, lag, 160 if B_rows == 4 else 200, B_rows, SEED, out)
            assert e.value.code == 1
    finally:
        Bn.wrnn_destroy(m)


def test_edge_shapes(env):
    """One sub-tensor (no earlier row: an ordinary stream), a row shorter than a chunk, and an empty request."""
    torch, Bn = env
    dev = "cuda:0"
    w, V, b, frames = _case(64, 1, 50, 4)
    om = orc.OracleModel(w, "f32")
    m = Bn.wrnn_create(w, "f32", max_batch=4)
    try:
        one = _gpu_run(torch, Bn, m, frames, V, b, 4, 8, 16, 1, 50)
        ref, _, margins = orc.subscale_dependent_run(om, frames, V, b, 1, 50, synth.HOP, SEED)
        d = np.nonzero(one != ref[0])[0]
        assert d.size == 0 or margins[0, d[0]].min() < pu.MARGIN
        # rows of 5 positions with chunks of 8: every call is a short one
        w3, V3, b3, fr3 = _case(64, 3, 5, 2)
        m3 = Bn.wrnn_create(w3, "f32", max_batch=3)
        try:
            got = orc.fold(_gpu_run(torch, Bn, m3, fr3, V3, b3, 2, 8, 16, 3, 5), 3)
            ref3, _, mg3 = orc.subscale_dependent_run(orc.OracleModel(w3, "f32"), fr3, V3, b3, 3, 5, synth.HOP, SEED)
            for row in range(3):
                d = np.nonzero(got[row] != ref3[row])[0]
                if d.size:
                    assert mg3[row, d[0]].min() < pu.MARGIN
                    break
        finally:
            Bn.wrnn_destroy(m3)
        out = torch.zeros((4,), dtype=torch.int16, device=dev)
        Bn.wrnn_sample_subscale_dependent(m, torch.from_numpy(frames).to(dev), torch.from_numpy(V).to(dev), torch.from_numpy(b).to(dev), 4, 8, 16,
                                          0, 1, SEED, out)       # nothing to do
    finally:
        Bn.wrnn_destroy(m)
