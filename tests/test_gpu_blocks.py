"""Irregular block structure (Section 4.1.5) on the GPU: layers whose W_piv holds rectangles of any size
and position, created through pp_layer_create_blocks, against the fp64 oracle's block form of Eq. 1.
Tolerances as everywhere: fp32 1e-5 / 1e-6, fp16 weights 2e-3 / 1e-4 on (|W| |x|)_i; integer data bit for bit."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

TOL = {"f32": (1e-5, 1e-6), "f16": (2e-3, 1e-4)}


@pytest.fixture(scope="module")
def pb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1712_01084_b200 import binding
    binding.lib()
    return binding


def _reference(lay, x, act):
    W = po.reconstruct_blocks(lay.M, lay.N, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values)
    return po.dense_forward(W, lay.bias, x.astype(np.float64), act, threads=8)


def _run(pb, wl, act, exact=False):
    lay = wl.layers[0]
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, torch.from_numpy(wl.x).cuda(), act).cpu().numpy()
    L.close()
    y_ref, _, a = _reference(lay, wl.x, act)
    if exact:
        assert np.array_equal(y.astype(np.float64), y_ref), wl.name
    else:
        rtol, atol = TOL[lay.wdtype]
        worst = np.max(np.abs(y.astype(np.float64) - y_ref) / (rtol * a + atol))
        assert worst <= 1.0, f"{wl.name}: worst error/bound = {worst:.3f}"


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("batch", [1, 5, 33])
def test_mixed_rectangles(pb, dtype, B, batch):
    """Blocks of different heights and widths at positions off the tile grid, several per row, ragged M and N."""
    wl = synth.irregular_blocks(500 + B + batch, 9 * B - 11, 13 * B - 5, B, wdtype=dtype, n_row_cuts=5,
                                n_col_cuts=7, keep=0.45, batch=batch, bias_std=0.1)
    for act in (0, 1):
        _run(pb, wl, act)


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("B", [16, 64])
def test_mixed_rectangles_bit_exact(pb, dtype, B):
    """Small integers: every partial sum is exact, so placement of every block element is checked bit for bit."""
    wl = synth.irregular_blocks(600 + B, 7 * B - 3, 6 * B - 1, B, wdtype=dtype, n_row_cuts=6, n_col_cuts=4,
                                keep=0.5, batch=3, bias_std=1.0, integer_values=True)
    _run(pb, wl, 0, exact=True)
    _run(pb, wl, 1, exact=True)


@pytest.mark.parametrize("size,blocks_per_side,B,dtype", [
    (512, 16, 32, "f32"),      # the example of Section 5: 16 blocks of 32 x 32
    (1024, 4, 64, "f32"),      # 25 % fill-in: 4 blocks of 256 x 256
    (2048, 8, 64, "f16"),      # 12.5 %
    (256, 32, 16, "f32"),      # 3.125 %: blocks of 8 x 8, smaller than the grid
    (4096, 4, 64, "f32"),      # the largest block of the paper's sweep: 1024 x 1024
])
def test_paper_geometry(pb, size, blocks_per_side, B, dtype):
    wl = synth.paper_square(size, blocks_per_side, B, wdtype=dtype)
    _run(pb, wl, 0)
    wl = synth.paper_square(size, blocks_per_side, B, wdtype=dtype, integer_values=True)
    _run(pb, wl, 0, exact=True)


def test_block_layer_in_a_chain(pb):
    """A layer made from blocks is a layer like any other: it folds into a chain (Section 4.2.1)."""
    w0 = synth.irregular_blocks(71, 300, 500, 32, wdtype="f16", n_row_cuts=4, n_col_cuts=6, keep=0.5,
                                batch=2, bias_std=0.1, act=synth.ACT_RELU)
    l0 = w0.layers[0]
    l1, _ = synth.make_layer(72, 200, 300, 32, wdtype="f16", tiles="uniform", density=0.4, bias_std=0.1)
    L0, L1 = pb.Layer.from_synth(l0), pb.Layer.from_synth(l1)
    ch = pb.Chain([L0, L1], [synth.ACT_RELU, synth.ACT_IDENTITY], max_batch=2)
    y = pb.pp_chain_forward(ch, torch.from_numpy(w0.x).cuda()).cpu().numpy()
    y0, _, a0 = _reference(l0, w0.x, synth.ACT_RELU)
    h = y0.astype(np.float16).astype(np.float64)
    W1 = po.reconstruct(l1.M, l1.N, l1.B, l1.row_perm, l1.col_perm, l1.tile_list, l1.tile_values)
    y1, _, a1 = po.dense_forward(W1, l1.bias, h, 0)
    # error of the first layer (its bound + rounding to fp16) carried through |W1|, plus the second layer's own bound
    e0 = 2e-3 * a0 + 1e-4 + np.abs(y0) * 2.0 ** -11
    bound = e0 @ np.abs(W1).T + 2e-3 * a1 + 1e-4
    assert np.all(np.abs(y.astype(np.float64) - y1) <= bound)
    ch.close(); L0.close(); L1.close()


# ------------------------------------------------ layout study (Section 4.1.1): three layouts x two thread mappings
@pytest.mark.parametrize("mapping", [0, 1], ids=["rows_per_lane", "lanes_along_k"])
@pytest.mark.parametrize("layout", [0, 1, 2], ids=["brc", "bcr", "cbr"])
@pytest.mark.parametrize("size,blocks_per_side", [(512, 16), (1024, 4), (96, 8), (4096, 2), (60, 5), (2600, 2)])
def test_layout_study_kernels(pb, layout, mapping, size, blocks_per_side):
    """Every layout with every mapping gives the oracle's numbers (block edges from 12 to 2048: below a warp,
    ragged against the 128-row and 32-row CTA shapes, and longer than one staged chunk of 1024 columns)."""
    for integer in (False, True):
        wl = synth.paper_square(size, blocks_per_side, 1, wdtype="f32", integer_values=integer)
        lay = wl.layers[0]
        K = pb.LayoutStudy(size, blocks_per_side, layout, mapping, lay.row_perm, lay.col_perm, lay.block_values)
        y = K.forward(torch.from_numpy(wl.x[0]).cuda()).cpu().numpy()
        K.close()
        y_ref, _, a = _reference(lay, wl.x, 0)
        if integer:
            assert np.array_equal(y.astype(np.float64), y_ref[0])
        else:
            assert np.all(np.abs(y.astype(np.float64) - y_ref[0]) <= 1e-5 * a[0] + 1e-6)


def test_layout_study_rejects_bad_arguments(pb):
    rp = np.arange(64, dtype=np.int32)
    v = np.zeros(4 * 16 * 16, dtype=np.float32)
    with pytest.raises(pb.PPError) as e:
        pb.LayoutStudy(64, 4, 0, 0, rp * 0, rp, v)                 # not a permutation
    assert e.value.status == 2
    for layout, mapping in ((3, 0), (0, 2)):
        with pytest.raises(pb.PPError) as e:
            pb.LayoutStudy(64, 4, layout, mapping, rp, rp, v)
        assert e.value.status == 1


def test_feed_back_search_to_layer(pb):
    """Section 3.2 end to end: search the index arrays on |W| of a dense matrix with a hidden block structure,
    keep the diagonal blocks, run the pruned layer, compare with the dense product of the pruned matrix."""
    rng = np.random.default_rng(321)
    M = N = 256
    levels = 3
    W = (rng.standard_normal((M, N)) * 0.01).astype(np.float32)
    pr, pc = rng.permutation(M), rng.permutation(N)
    e = M >> levels
    for k in range(1 << levels):                       # heavy entries on hidden diagonal blocks
        W[np.ix_(pr[k * e:(k + 1) * e], pc[k * e:(k + 1) * e])] += rng.standard_normal((e, e)).astype(np.float32)
    rp, cp, bl, kept = pb.pp_pivot_find(np.abs(W), levels, 32, rng.permutation(M), rng.permutation(N))
    assert kept > 0.9 * np.abs(W).sum()
    vals = np.concatenate([W[np.ix_(rp[r0:r0 + h], cp[c0:c0 + w])].ravel() for r0, c0, h, w in bl]).astype(np.float32)
    L = pb.Layer.from_blocks(M, N, 32, rp, cp, bl, vals)
    x = rng.uniform(-1, 1, (2, N)).astype(np.float32)
    y = pb.pp_forward(L, torch.from_numpy(x).cuda(), 0).cpu().numpy()
    L.close()
    Wp = po.reconstruct_blocks(M, N, rp, cp, bl, vals)
    y_ref, _, a = po.dense_forward(Wp, None, x.astype(np.float64), 0)
    assert np.all(np.abs(y - y_ref) <= 1e-5 * a + 1e-6)
    mask = Wp != 0                                      # the pruned matrix is W on the kept entries, zero elsewhere
    assert np.array_equal(Wp[mask], W.astype(np.float64)[mask])
