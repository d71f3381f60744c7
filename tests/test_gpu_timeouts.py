"""The time-out paths of the kernels, exercised without hanging or faulting anything.

Every device-side wait in this library is bounded.  Tuning key 15 shortens the bound to a given number of polls
that return at once, so that a wait runs out while the data it waits for is still on its way: the kernel must
raise its status word, let its own copies land, give back tensor memory and END BY ITSELF; the host reads
PP_ERR_TIMEOUT.  With the default bound restored the same handle must work again and match the oracle."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

PP_ERR_TIMEOUT = 7


@pytest.fixture(scope="module")
def pb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1712_01084_b200 import binding
    binding.lib()
    return binding


@pytest.fixture
def one_poll(pb):
    def set_polls(n):
        pb.pp_set_tuning(15, n)
    yield set_polls
    pb.pp_set_tuning(15, 0)


def _close(y, y_ref, a, rtol=2e-3, atol=1e-4):
    return np.all(np.abs(y.astype(np.float64) - y_ref) <= rtol * a + atol)


def test_persistent_kernel_x_wait_runs_out(pb, one_poll):
    wl = synth.config5(k=16, batch=1, scale=0.25)
    lay = wl.layers[0]
    L = pb.Layer.from_synth(lay)
    x = torch.from_numpy(wl.x).cuda()
    y_ref, _, a = po.layer_forward(lay, wl.x.astype(np.float64))
    assert L.launch_info(1)["kernel"] == "stream"
    one_poll(1)
    pb.pp_forward(L, x, lay.act)
    assert L.status() == PP_ERR_TIMEOUT          # synchronises: the kernel came back by itself
    assert L.status() == 0                       # the flag is cleared by the read
    one_poll(0)
    y = pb.pp_forward(L, x, lay.act).cpu().numpy()
    assert L.status() == 0 and _close(y, y_ref, a)
    L.close()


@pytest.mark.parametrize("tile_kernel", [0, 2, 3], ids=["one_block_row", "clustered", "persistent"])
def test_tile_kernels_stage_wait_runs_out(pb, one_poll, tile_kernel):
    wl = synth.config5(k=128, batch=40, scale=0.125)      # 1024 x 1024, every tile kept
    lay = wl.layers[0]
    x = torch.from_numpy(wl.x).cuda()
    y_ref, _, a = po.layer_forward(lay, wl.x.astype(np.float64))
    pb.pp_set_tuning(12, tile_kernel)                 # before the layer exists: the persistent kernel's plan is built at creation
    try:
        L = pb.Layer.from_synth(lay)
        assert L.launch_info(40)["kernel"] == {0: "tile", 2: "tile_cluster", 3: "tile_persist"}[tile_kernel]
        one_poll(1)
        pb.pp_forward(L, x, lay.act)
        assert L.status() == PP_ERR_TIMEOUT
        one_poll(0)
        y = pb.pp_forward(L, x, lay.act).cpu().numpy()
        assert L.status() == 0 and _close(y, y_ref, a)
    finally:
        pb.pp_set_tuning(12, 1)
    L.close()


def test_chain_kernel_boundary_wait_runs_out(pb, one_poll):
    wl = synth.config3(batch=2, scale=0.25)
    layers = [pb.Layer.from_synth(l) for l in wl.layers]
    pb.pp_set_tuning(14, 1)
    try:
        chain = pb.Chain(layers, [l.act for l in wl.layers], max_batch=4)
        x = torch.from_numpy(wl.x).cuda()
        res = po.chain_forward(wl.layers, wl.x.astype(np.float64), round_intermediate="f16")
        good = pb.pp_chain_forward(chain, x).cpu().numpy()
        assert chain.status() == 0
        one_poll(1)
        pb.pp_chain_forward(chain, x)
        assert chain.status() == PP_ERR_TIMEOUT      # also clears the arrival counter the launch left behind
        one_poll(0)
        y = pb.pp_chain_forward(chain, x).cpu().numpy()
        assert chain.status() == 0 and np.array_equal(y, good)
        assert np.max(np.abs(y - res[-1][1])) < 0.05     # coarse: the bit-level checks live in test_gpu_parity.py
    finally:
        pb.pp_set_tuning(14, 0)
    chain.close()
    for l in layers:
        l.close()


def test_lstm_cell_packet_wait_runs_out(pb, one_poll):
    wl = synth.config4(steps=4, scale=0.25)
    lay, H, I = wl.layers[0], wl.extra["H"], wl.extra["I"]
    L = pb.Layer.from_synth(lay)
    cell = pb.Lstm(L, I, H, max_steps=4)
    xs = torch.from_numpy(wl.x).cuda()

    def run():
        h = torch.zeros(H, dtype=torch.float16, device="cuda")
        c = torch.zeros(H, dtype=torch.float32, device="cuda")
        pb.pp_lstm_forward(cell, xs, h, c)
        return h, c

    h_good, c_good = run()
    assert cell.status() == 0
    one_poll(1)
    run()
    assert cell.status() == PP_ERR_TIMEOUT
    one_poll(0)
    h, c = run()
    assert cell.status() == 0 and torch.equal(h, h_good) and torch.equal(c, c_good)
    cell.close(); L.close()
