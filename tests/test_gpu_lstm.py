"""Recurrent use of one pivoted gate layer (LSTM cell) against the fp64 oracle recurrence.

Binding check, teacher-forced: every tested step starts from the oracle's own (h, c), so the bound
is local: with d_g = 2e-3 * (|W| |z|) + 1e-4 on each pre-activation (the fp16-weight tolerance),
sig' <= 1/4 and tanh' <= 1 give
    d_c <= d_f |c_prev| / 4 + d_i / 4 + d_g + 1e-6 (1 + |c|),
    d_h <= d_o / 4 + d_c + 2^-10 |h| + 1e-6        (h is stored as fp16 on both sides).
The free-running 256-step comparison is reported and only loosely bounded: the paper does not pin it."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def pb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1712_01084_b200 import binding
    binding.lib()
    return binding


def _dense(lay):
    return po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)


def _step_bounds(a, c_prev, c, h, H):
    d = 2e-3 * a + 1e-4
    di, df, dg, do = d[0:H], d[H:2 * H], d[2 * H:3 * H], d[3 * H:4 * H]
    dc = 0.25 * df * np.abs(c_prev) + 0.25 * di + dg + 1e-6 * (1 + np.abs(c))
    dh = 0.25 * do + dc + 2.0 ** -10 * np.abs(h) + 1e-6
    return dc, dh


@pytest.fixture(params=[1, 0], ids=["persistent", "per-step"])
def cell_mode(pb, request):
    """Both ways pp_lstm_forward can run a qualifying fp16 layer: one cooperative kernel with the
    weights resident in shared memory, or two kernels per step."""
    pb.pp_set_tuning(11, request.param)
    yield request.param
    pb.pp_set_tuning(11, 1)


@pytest.mark.parametrize("scale", [1 / 16, 1.0])
def test_lstm_teacher_forced_steps(pb, scale, cell_mode):
    steps = 12 if scale < 1 else 6
    wl = synth.config4(steps=steps, scale=scale)
    lay, H, I = wl.layers[0], wl.extra["H"], wl.extra["I"]
    W = _dense(lay)
    L = pb.Layer.from_synth(lay)
    cell = pb.Lstm(L, I, H, max_steps=4)
    x_seq = wl.x
    h = np.zeros(H); c = np.zeros(H)
    for t in range(steps):
        _, a, c_new, h_new = po.lstm_step(W, x_seq[t].astype(np.float64), h, c, threads=8)
        h_dev = torch.from_numpy(h.astype(np.float16)).cuda()
        c_dev = torch.from_numpy(c.astype(np.float32)).cuda()
        pb.pp_lstm_forward(cell, torch.from_numpy(x_seq[t:t + 1]).cuda(), h_dev, c_dev)
        dc, dh = _step_bounds(a, c, c_new, h_new, H)
        # c was handed over rounded to fp32: |sig(f)| <= 1 times that rounding
        dc = dc + np.abs(c) * 2.0 ** -23
        dh = dh + np.abs(c) * 2.0 ** -23
        ec = np.abs(c_dev.cpu().numpy().astype(np.float64) - c_new)
        eh = np.abs(h_dev.cpu().numpy().astype(np.float64) - h_new)
        assert np.max(ec / dc) <= 1.0, f"step {t}: c error/bound {np.max(ec / dc):.3f}"
        assert np.max(eh / dh) <= 1.0, f"step {t}: h error/bound {np.max(eh / dh):.3f}"
        h = h_new.astype(np.float16).astype(np.float64)      # the recurrence stores h as fp16
        c = c_new
    cell.close(); L.close()


def test_lstm_free_running_256_steps(pb, cell_mode):
    wl = synth.config4(steps=256)
    lay, H, I = wl.layers[0], wl.extra["H"], wl.extra["I"]
    L = pb.Layer.from_synth(lay)
    cell = pb.Lstm(L, I, H, max_steps=256)
    h = torch.zeros(H, dtype=torch.float16, device="cuda")
    c = torch.zeros(H, dtype=torch.float32, device="cuda")
    pb.pp_lstm_forward(cell, torch.from_numpy(wl.x).cuda(), h, c)
    h_ref, c_ref, _ = po.lstm_forward(_dense(lay), wl.x.astype(np.float64), H, h_round="f16", threads=8)
    dh = np.max(np.abs(h.cpu().numpy().astype(np.float64) - h_ref))
    dc = np.max(np.abs(c.cpu().numpy().astype(np.float64) - c_ref))
    print(f"free-running drift after 256 steps: max |dh| = {dh:.3e}, max |dc| = {dc:.3e}")
    # No bound follows from the paper (the cell is the workload's).  Both sides round h_t to binary16 after every
    # step, so the outputs differ by what the fp32 gate arithmetic and the hardware exponential leave (measured
    # 6.1e-5 on h, 1.4e-6 on c) unless a value lands on the other side of a rounding boundary: one binary16
    # step below 1 is 4.9e-4.  Limits: that one step for h (8 x the measured drift), 14 x the measured drift for c.
    assert dh < 5e-4 and dc < 2e-5
    # run it again from zero: identical bits (deterministic kernels, scratch left clean)
    h2 = torch.zeros_like(h); c2 = torch.zeros_like(c)
    pb.pp_lstm_forward(cell, torch.from_numpy(wl.x).cuda(), h2, c2)
    assert torch.equal(h, h2) and torch.equal(c, c2)
    assert cell.status() == 0
    cell.close(); L.close()


@pytest.mark.parametrize("H,I,B,density", [(40, 56, 16, 1.0), (604, 420, 32, 0.4), (1208, 200, 64, 0.3)])
def test_lstm_ragged_strip_counts_and_bias(pb, H, I, B, density, cell_mode):
    """Strip counts that do not divide by the strips a CTA of the persistent cell holds (151 strips
    dealt out in twos, 302 in fours), block-rows of unequal length, and a layer bias inside g."""
    lay, rng = synth.make_layer(4100 + H, 4 * H, I + H, B, wdtype="f16", tiles="uniform", density=density,
                                bias_std=0.3)
    L = pb.Layer.from_synth(lay)
    steps = 7
    cell = pb.Lstm(L, I, H, max_steps=steps)
    x_seq = rng.uniform(-1, 1, (steps, I)).astype(np.float16)
    h0 = rng.uniform(-1, 1, H).astype(np.float16)
    c0 = rng.uniform(-1, 1, H).astype(np.float32)
    h = torch.from_numpy(h0).cuda(); c = torch.from_numpy(c0).cuda()
    pb.pp_lstm_forward(cell, torch.from_numpy(x_seq).cuda(), h, c)
    hr, cr, _ = po.lstm_forward(_dense(lay), x_seq.astype(np.float64), H, h_round="f16", threads=4,
                                h0=h0, c0=c0, bias=lay.bias.astype(np.float64))
    eh = np.max(np.abs(h.cpu().numpy().astype(np.float64) - hr))
    ec = np.max(np.abs(c.cpu().numpy().astype(np.float64) - cr))
    print(f"ragged cell H={H}: max |dh| = {eh:.3e}, max |dc| = {ec:.3e}")
    assert eh < 4e-3 and ec < 4e-3
    assert cell.status() == 0
    cell.close(); L.close()


def test_lstm_fp32_layer_and_bad_arguments(pb):
    H, I, B = 48, 80, 16
    lay, rng = synth.make_layer(77, 4 * H, I + H, B, wdtype="f32", tiles="uniform", density=0.5)
    L = pb.Layer.from_synth(lay)
    cell = pb.Lstm(L, I, H, max_steps=5)
    x_seq = rng.uniform(-1, 1, (5, I)).astype(np.float32)
    h = torch.zeros(H, device="cuda"); c = torch.zeros(H, device="cuda")
    pb.pp_lstm_forward(cell, torch.from_numpy(x_seq).cuda(), h, c)
    h_ref, c_ref, _ = po.lstm_forward(_dense(lay), x_seq.astype(np.float64), H, h_round="f32")
    assert np.max(np.abs(h.cpu().numpy() - h_ref)) < 1e-4 and np.max(np.abs(c.cpu().numpy() - c_ref)) < 1e-4
    with pytest.raises(pb.PPError):
        pb.pp_lstm_forward(cell, torch.zeros((6, I), device="cuda"), h, c)          # more steps than allocated
    with pytest.raises(pb.PPError):
        pb.Lstm(L, I + 1, H, 4)                                                     # shape mismatch
    cell.close(); L.close()
