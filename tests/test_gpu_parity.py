"""Parity of the CUDA library (through its C interface) against the fp64 oracle.

Tolerances (|y - y_ref| <= rtol * (|W| |x|)_i + atol, the magnitude computed by
the oracle): fp32 weights 1e-5 / 1e-6; fp16 weights with fp32 accumulation
2e-3 / 1e-4.  Index and permutation handling is checked bit for bit with small
integer data, for which every partial sum is exact in fp16 / fp32 / fp64."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

TOL = {np.dtype(np.float32): (1e-5, 1e-6), np.dtype(np.float16): (2e-3, 1e-4)}


@pytest.fixture(scope="module")
def pb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1712_01084_b200 import binding
    binding.lib()                     # fails loudly if the library is not built
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _rand_layer(seed, M, N, B, dtype, density=0.4, bias=True, integer=False, empty_rows=()):
    rng = np.random.default_rng(seed)
    Mb, Nb = -(-M // B), -(-N // B)
    grid = [(br, bc) for br in range(Mb) for bc in range(Nb) if br not in empty_rows]
    T = max(1, int(density * len(grid)))
    sel = rng.permutation(len(grid))[:T]
    tl = np.array([grid[s] for s in sel], dtype=np.int32).reshape(-1, 2)
    if integer:
        tv = rng.integers(-4, 5, size=(T, B, B)).astype(dtype)
        b = rng.integers(-8, 9, size=M).astype(np.float32) if bias else None
    else:
        tv = (rng.standard_normal((T, B, B)) / np.sqrt(N)).astype(dtype)
        b = (rng.standard_normal(M) * 0.1).astype(np.float32) if bias else None
    return synth.Layer(M, N, B, rng.permutation(Mb * B).astype(np.int32),
                       rng.permutation(Nb * B).astype(np.int32), tl, tv, b)


def _check(y_gpu, y_ref, a_ref, dtype, what=""):
    rtol, atol = TOL[np.dtype(dtype)]
    err = np.abs(y_gpu.astype(np.float64) - y_ref)
    bound = rtol * a_ref + atol
    worst = np.max(err / bound)
    assert worst <= 1.0, f"{what}: worst error/bound = {worst:.3f}"


def _run_and_check(pb, lay, x, act, what=""):
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, _dev(x), act).cpu().numpy()
    y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=act, threads=8)
    _check(y, y_ref, a, lay.tile_values.dtype, what)
    L.close()
    return y


# ------------------------------------------------------------------ small sweeps
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("batch", [1, 2, 3, 8, 9, 17, 33])
@pytest.mark.parametrize("persistent", [1, 0])
def test_small_layers(pb, dtype, B, batch, persistent):
    """Ragged M and N, unbalanced block-rows, one block-row without tiles, several tiles and a ragged tail;
    through the persistent kernel (in groups of 8 columns) and through the chunked kernel (the tensor-core
    path, which fp16 B = 64 layers would take from batch 9 on, is switched off here and tested further down)."""
    pb.pp_set_tuning(5, persistent)
    pb.pp_set_tuning(9, 0)
    try:
        lay = _rand_layer(100 + B + batch, 5 * B - 3, 9 * B - 7, B, dtype, density=0.45, empty_rows=(2,))
        x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(dtype)
        for act in (0, 1):
            _run_and_check(pb, lay, x, act, f"{dtype.__name__} B={B} batch={batch} act={act}")
    finally:
        pb.pp_set_tuning(5, 1)
        pb.pp_set_tuning(9, 9)


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("direct,depth", [(0, 4), (1, 8), (0, 8)])
def test_persistent_kernel_batch1_variants(pb, dtype, B, direct, depth):
    """Batch 1 with x permuted in shared memory first (direct=0) or read through the index array in
    the multiply loop (direct=1, the default), and with 4 or 8 weight copies in flight per warp."""
    pb.pp_set_tuning(7, direct); pb.pp_set_tuning(6, depth)
    try:
        lay = _rand_layer(70 + B, 7 * B - 3, 11 * B - 9, B, dtype, density=0.5, empty_rows=(1,))
        x = np.random.default_rng(B).uniform(-1, 1, (1, lay.N)).astype(dtype)
        for act in (0, 1):
            _run_and_check(pb, lay, x, act, f"direct={direct} depth={depth} B={B}")
    finally:
        pb.pp_set_tuning(7, 2); pb.pp_set_tuning(6, 0)


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("ctas,min_frags,snap", [(296, 1, 0), (5, 1, 0), (37, 4, 50), (2000, 1, 25)])
def test_persistent_kernel_partitions(pb, dtype, ctas, min_frags, snap):
    """CTA ranges that cut strips in the middle (cross-CTA partial sums), that snap to strip
    boundaries, fewer CTAs than strips and more CTAs than SMs can hold at once."""
    pb.pp_set_tuning(2, ctas); pb.pp_set_tuning(3, min_frags); pb.pp_set_tuning(4, snap)
    try:
        for B in (16, 64):
            lay = _rand_layer(11 + B, 9 * B - 3, 20 * B - 7, B, dtype, density=0.5, empty_rows=(0, 4))
            for batch in (1, 3, 8):
                x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(dtype)
                _run_and_check(pb, lay, x, 1, f"ctas={ctas} B={B} batch={batch}")
    finally:
        pb.pp_set_tuning(2, 296); pb.pp_set_tuning(3, 128); pb.pp_set_tuning(4, -1)


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("target_kib", [1, 4, 64])
def test_split_block_rows(pb, dtype, target_kib):
    """Block-rows cut into many work items (cross-CTA reduction) and into one."""
    pb.pp_set_tuning(0, target_kib)
    try:
        lay = _rand_layer(7, 200, 1500, 32, dtype, density=0.6)
        for batch in (1, 5):
            x = np.random.default_rng(3).uniform(-1, 1, (batch, lay.N)).astype(dtype)
            _run_and_check(pb, lay, x, 1, f"target {target_kib} KiB batch {batch}")
    finally:
        pb.pp_set_tuning(0, 32)


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("persistent", [1, 0])
def test_integer_data_is_bit_exact(pb, dtype, B, persistent):
    """Small-integer weights, inputs and bias: all sums exact, so any index or
    permutation slip shows up as a bit difference."""
    pb.pp_set_tuning(0, 2); pb.pp_set_tuning(5, persistent); pb.pp_set_tuning(2, 23); pb.pp_set_tuning(3, 1)
    try:
        lay = _rand_layer(50 + B, 4 * B - 1, 6 * B - 5, B, dtype, density=0.5, integer=True)
        for batch in (1, 4, 11):
            x = np.random.default_rng(5).integers(-2, 3, (batch, lay.N)).astype(dtype)
            L = pb.Layer.from_synth(lay)
            for act in (0, 1):
                y = pb.pp_forward(L, _dev(x), act).cpu().numpy()
                y_ref, _, _ = po.layer_forward(lay, x.astype(np.float64), act=act)
                assert np.array_equal(y.astype(np.float64), y_ref)
            L.close()
    finally:
        pb.pp_set_tuning(0, 32); pb.pp_set_tuning(5, 1); pb.pp_set_tuning(2, 296); pb.pp_set_tuning(3, 128)


def test_identity_perms_density_one(pb):
    lay, rng = synth.make_layer(1, 256, 384, 64, wdtype="f32", tiles="balanced", k=6, identity_perms=True)
    x = synth.draw_x(rng, 2, 384, -1, 1, "f32")
    y = _run_and_check(pb, lay, x, 0, "dense identity")
    Wd = np.block([[lay.tile_values[br * 6 + bc] for bc in range(6)] for br in range(4)]).astype(np.float64)
    ref = x.astype(np.float64) @ Wd.T
    assert np.max(np.abs(y - ref)) < 1e-5


@pytest.mark.parametrize("persistent", [1, 0])
def test_deterministic_and_canaries(pb, persistent):
    """Same inputs twice -> identical bits; memory around y is untouched."""
    pb.pp_set_tuning(0, 2); pb.pp_set_tuning(5, persistent); pb.pp_set_tuning(4, 0)
    try:
        lay = _rand_layer(9, 777, 1111, 32, np.float16, density=0.5)
        L = pb.Layer.from_synth(lay)
    finally:
        pb.pp_set_tuning(0, 32); pb.pp_set_tuning(4, -1)
    x = _dev(np.random.default_rng(1).uniform(-1, 1, (3, lay.N)).astype(np.float16))
    pad = 64
    buf = torch.full((3 * lay.M + 2 * pad,), 12345.0, dtype=torch.float32, device="cuda")
    out = buf[pad:pad + 3 * lay.M].view(3, lay.M)
    y1 = pb.pp_forward(L, x, 1, out=out).clone()
    assert torch.all(buf[:pad] == 12345.0) and torch.all(buf[-pad:] == 12345.0)
    try:
        for _ in range(5):
            y2 = pb.pp_forward(L, x, 1)
            assert torch.equal(y1, y2)
    finally:
        pb.pp_set_tuning(5, 1)
    L.close()


def test_argument_errors(pb):
    lay = _rand_layer(10, 64, 64, 32, np.float32)
    L = pb.Layer.from_synth(lay)
    x = torch.zeros(4096, device="cuda")
    assert pb.lib().pp_forward(L._h, x.data_ptr() + 4, x.data_ptr() + 2048, 1, 0, None) == 1   # misaligned x
    assert pb.lib().pp_forward(L._h, x.data_ptr(), x.data_ptr(), 1, 0, None) == 1     # aliasing
    assert pb.lib().pp_forward(L._h, x.data_ptr(), x.data_ptr() + 2048, 0, 0, None) == 1  # batch 0
    with pytest.raises(TypeError):
        pb.pp_forward(L, torch.zeros(1, 64, device="cuda", dtype=torch.float16))
    L.close()


# ------------------------------------------------------------------ the five workloads
def test_config1_full(pb):
    wl = synth.config1()
    _run_and_check(pb, wl.layers[0], wl.x, wl.layers[0].act, "config 1")


def test_config2_full(pb):
    wl = synth.config2()
    _run_and_check(pb, wl.layers[0], wl.x, wl.layers[0].act, "config 2")


def _chain_bound(layers, res, dtype_tol):
    """Propagated end-to-end bound: e_{l} <= |W_l| e_{l-1} + tol_l (+ fp16 rounding of the stored output)."""
    rtol, atol = dtype_tol
    e = None
    for li, lay in enumerate(layers):
        xin, y, a = res[li]
        tol = rtol * a + atol
        if e is not None:
            W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
            prop, _, _ = po.dense_forward(np.abs(W), None, e, 0, threads=8)
            tol = tol + prop
        if li + 1 < len(layers):
            tol = tol + np.abs(y) * 2.0 ** -10 + 2.0 ** -24     # stored as fp16 (both sides round)
        e = tol
    return e


@pytest.fixture(params=[1, 0], ids=["one_kernel", "kernel_per_layer"])
def chain_mode(request, pb):
    """Chains of fp16 layers run as one cooperative kernel (tuning key 14 = 1) or one launch per layer (default)."""
    pb.pp_set_tuning(14, request.param)
    yield request.param
    pb.pp_set_tuning(14, 0)


@pytest.mark.parametrize("batch", [1, 8])
def test_config3_chain_full(pb, batch, chain_mode):
    wl = synth.config3(batch=batch)
    layers = [pb.Layer.from_synth(l) for l in wl.layers]
    chain = pb.Chain(layers, [l.act for l in wl.layers], max_batch=8)
    y = pb.pp_chain_forward(chain, _dev(wl.x)).cpu().numpy().astype(np.float64)
    assert chain.status() == 0
    res = po.chain_forward(wl.layers, wl.x.astype(np.float64), round_intermediate="f16", threads=8)
    bound = _chain_bound(wl.layers, res, TOL[np.dtype(np.float16)])
    worst = np.max(np.abs(y - res[-1][1]) / bound)
    assert worst <= 1.0, f"chain end-to-end worst error/bound {worst:.3f}"
    # teacher-forced per-layer check: every layer alone, fed the oracle's (rounded) input
    for li, lay in enumerate(wl.layers):
        xin = res[li][0].astype(np.float16)
        yl = pb.pp_forward(layers[li], _dev(xin), lay.act).cpu().numpy()
        _check(yl, res[li][1], res[li][2], np.float16, f"config 3 layer {li}")
    chain.close()
    for l in layers:
        l.close()


@pytest.mark.parametrize("B,dims", [(16, [200, 150, 90, 33]), (32, [700, 333, 64, 129, 10]), (64, [256, 1000, 70])])
@pytest.mark.parametrize("batch", [1, 3, 8])
def test_chain_one_kernel_equals_kernel_per_layer(pb, B, dims, batch):
    """fp16 chains: the cooperative one-kernel execution, the launch-per-layer execution and the oracle give the
    same bits on integer data (ragged sizes, empty block-rows, layers whose plans have different CTA counts,
    twice in a row: the boundary counter must be left clean)."""
    lays = []
    for l in range(len(dims) - 1):
        lay = _rand_layer(900 + 10 * B + l, dims[l + 1], dims[l], B, np.float16, density=0.5, integer=True,
                          empty_rows=(1,) if l == 1 else ())
        lay.tile_values = (np.sign(lay.tile_values) * (np.abs(lay.tile_values) > 3)).astype(np.float16)   # entries in {-1,0,1}
        lay.bias = np.sign(lay.bias).astype(np.float32)
        lay.act = 1 if l + 2 < len(dims) else 0
        lays.append(lay)
    x = np.random.default_rng(B + batch).integers(-1, 2, (batch, dims[0])).astype(np.float16)
    L = [pb.Layer.from_synth(l) for l in lays]
    outs = []
    try:
        pb.pp_set_tuning(14, 1)                         # read when the chain is created and at every call
        chain = pb.Chain(L, [l.act for l in lays], max_batch=8)
        for mode in (1, 1, 0):
            pb.pp_set_tuning(14, mode)
            outs.append(pb.pp_chain_forward(chain, _dev(x)).cpu().numpy())
            assert chain.status() == 0
    finally:
        pb.pp_set_tuning(14, 0)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    res = po.chain_forward(lays, x.astype(np.float64), round_intermediate="f16")
    assert np.array_equal(outs[0].astype(np.float64), res[-1][1])
    chain.close()
    for l in L:
        l.close()


def test_chain_matches_layer_by_layer_bits(pb):
    """Folded chain (pivoted intermediates) == unfolded evaluation with the same
    kernels, bit for bit, on integer data; fp32 chain against the oracle."""
    dims = [200, 150, 90, 33]
    lays = []
    for l in range(3):
        lay = _rand_layer(300 + l, dims[l + 1], dims[l], 16, np.float32, density=0.5, integer=True)
        lay.tile_values = np.sign(lay.tile_values) * (np.abs(lay.tile_values) > 3)   # entries in {-1,0,1}
        lay.act = 1 if l < 2 else 0
        lays.append(lay)
    x = np.random.default_rng(2).integers(-1, 2, (3, dims[0])).astype(np.float32)
    L = [pb.Layer.from_synth(l) for l in lays]
    chain = pb.Chain(L, [l.act for l in lays], max_batch=4)
    y = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
    cur = _dev(x)
    for lay, Ld in zip(lays, L):
        cur = pb.pp_forward(Ld, cur, lay.act)
    assert np.array_equal(y, cur.cpu().numpy())
    res = po.chain_forward(lays, x.astype(np.float64))
    assert np.array_equal(y.astype(np.float64), res[-1][1])
    chain.close()


@pytest.mark.parametrize("k", [128, 64, 32, 16, 8])
def test_config5_batch1_full(pb, k):
    wl = synth.config5(k=k, batch=1)
    _run_and_check(pb, wl.layers[0], wl.x, 0, f"config 5 k={k}")


@pytest.mark.parametrize("k,batch", [(128, 16), (128, 128), (64, 128), (32, 16), (8, 128), (8, 16)])
def test_config5_batched_full(pb, k, batch):
    """Full size, every output row of every input vector against the fp64 product, with the kernel choice left
    on automatic: the launch configurations the benchmark times (density 1 takes the clustered tensor-core
    kernel, sparse layers the one-block-row kernel)."""
    import os
    wl = synth.config5(k=k, batch=batch)
    lay = wl.layers[0]
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, _dev(wl.x), 0).cpu().numpy()
    assert L.status() == 0
    y_ref, _, a = po.layer_forward(lay, wl.x.astype(np.float64), act=0, threads=os.cpu_count() or 1)
    _check(y, y_ref, a, np.float16, f"config 5 k={k} batch {batch}, all rows")
    L.close()


@pytest.mark.parametrize("batch", [2, 4, 8, 16])
def test_config5_small_batch_sampled_rows(pb, batch):
    """Full size; the oracle evaluates a sample of output rows.  Batch 2..8 runs the persistent kernel with x read
    through the index array (one CTA per SM from batch 3 on: two waves of the 296-CTA plan), 16 the tile path."""
    wl = synth.config5(k=32, batch=batch)
    lay = wl.layers[0]
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, _dev(wl.x), 0).cpu().numpy()
    W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    rows = np.random.default_rng(0).choice(lay.M, 256, replace=False).astype(np.int32)
    y_ref, a = po.dense_forward_rows(W, None, wl.x.astype(np.float64), 0, rows)
    _check(y[:, rows], y_ref, a, np.float16, f"config 5 batch {batch} sampled")
    L.close()


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("prepass", [0, 2])
def test_input_permutation_prepass(pb, dtype, prepass):
    """Multi-column inputs permuted by the pre-pass kernel (forced) or inside the layer kernels, for the
    persistent kernel (batch <= 8), the chunked kernel (batch 20, fp16) and a folded chain."""
    pb.pp_set_tuning(10, prepass)
    try:
        lay = _rand_layer(31, 6 * 32 - 5, 10 * 32 - 3, 32, dtype, density=0.5, empty_rows=(3,))
        for batch in (2, 8, 20):
            x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(dtype)
            _run_and_check(pb, lay, x, 1, f"prepass={prepass} batch={batch}")
        dims = [150, 100, 70]
        lays = []
        for l in range(2):
            ll = _rand_layer(400 + l, dims[l + 1], dims[l], 16, dtype, density=0.6, integer=True)
            ll.tile_values = (np.sign(ll.tile_values) * (np.abs(ll.tile_values) > 3)).astype(dtype)
            ll.act = 1 if l == 0 else 0
            lays.append(ll)
        x = np.random.default_rng(2).integers(-1, 2, (5, dims[0])).astype(dtype)
        L = [pb.Layer.from_synth(l) for l in lays]
        chain = pb.Chain(L, [l.act for l in lays], max_batch=8)
        y = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
        res = po.chain_forward(lays, x.astype(np.float64))
        assert np.array_equal(y.astype(np.float64), res[-1][1])
        chain.close()
    finally:
        pb.pp_set_tuning(10, 1)


# ------------------------------------------------------------------ tensor-core tile path (batch >= 64)
@pytest.fixture(params=[2, 0, 3, 1], ids=["clustered", "row-per-cta", "persistent", "auto"])
def tile_kernel(pb, request):
    """The tensor-core kernels: a cluster of 4 CTAs per 4 block-rows, one CTA per block-row, or one persistent CTA
    per SM over an equal share of the layer's steps."""
    pb.pp_set_tuning(12, request.param)
    yield request.param
    pb.pp_set_tuning(12, 1)


@pytest.mark.parametrize("batch", [9, 31, 64, 100, 128, 129, 300])
def test_tile_path_small_layer(pb, batch, tile_kernel):
    """fp16, B = 64: ragged sizes, unbalanced block-rows, one block-row without tiles, batch chunks of 128
    with a ragged last chunk; compared element by element, and bit for bit on integer data."""
    lay = _rand_layer(900 + batch, 5 * 64 - 3, 9 * 64 - 7, 64, np.float16, density=0.45, empty_rows=(2,))
    x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(np.float16)
    L = pb.Layer.from_synth(lay)
    want = {0: "tile", 2: "tile_cluster", 3: "tile_persist"}.get(tile_kernel)
    assert want is None or L.launch_info(batch)["kernel"] == want
    for act in (0, 1):
        y = pb.pp_forward(L, _dev(x), act).cpu().numpy()
        assert L.status() == 0
        y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=act, threads=8)
        _check(y, y_ref, a, np.float16, f"tile path batch={batch} act={act}")
    L.close()
    lay = _rand_layer(950 + batch, 4 * 64 - 1, 6 * 64 - 5, 64, np.float16, density=0.5, integer=True)
    x = np.random.default_rng(5).integers(-2, 3, (batch, lay.N)).astype(np.float16)
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, _dev(x), 1).cpu().numpy()
    y_ref, _, _ = po.layer_forward(lay, x.astype(np.float64), act=1, threads=8)
    assert np.array_equal(y.astype(np.float64), y_ref)
    # the same batch through the matrix-vector kernels gives the same integers
    pb.pp_set_tuning(9, 0)
    try:
        y2 = pb.pp_forward(L, _dev(x), 1).cpu().numpy()
    finally:
        pb.pp_set_tuning(9, 9)
    assert np.array_equal(y, y2)
    L.close()


def test_tile_path_both_kernels_same_bits_and_repeatable(pb):
    """Unbalanced groups (a group with an empty block-row, a last group of 2 block-rows, a block-row
    whose tiles all fall into one CTA's quarter): repeated calls give identical bits, and on integer
    data the clustered kernel and the one-block-row kernel agree exactly."""
    lay = _rand_layer(977, 10 * 64 - 9, 23 * 64 - 1, 64, np.float16, density=0.3, empty_rows=(5,), integer=True)
    x = np.random.default_rng(3).integers(-2, 3, (128, lay.N)).astype(np.float16)
    try:
        pb.pp_set_tuning(12, 3)                       # the persistent kernel's plan is built when the layer is created
        L = pb.Layer.from_synth(lay)
        assert L.launch_info(128)["kernel"] == "tile_persist"
        pb.pp_set_tuning(12, 2)
        y1 = pb.pp_forward(L, _dev(x), 0).cpu().numpy()
        y1b = pb.pp_forward(L, _dev(x), 0).cpu().numpy()
        pb.pp_set_tuning(12, 0)
        y0 = pb.pp_forward(L, _dev(x), 0).cpu().numpy()
        pb.pp_set_tuning(12, 3)
        y3 = pb.pp_forward(L, _dev(x), 0).cpu().numpy()
        y3b = pb.pp_forward(L, _dev(x), 0).cpu().numpy()
    finally:
        pb.pp_set_tuning(12, 1)
    assert L.status() == 0
    assert np.array_equal(y1, y1b) and np.array_equal(y1, y0) and np.array_equal(y1, y3) and np.array_equal(y3, y3b)
    y_ref, _, _ = po.layer_forward(lay, x.astype(np.float64), act=0, threads=8)
    assert np.array_equal(y1.astype(np.float64), y_ref)
    L.close()
    lay = _rand_layer(978, 7 * 64, 12 * 64, 64, np.float16, density=0.6)
    x = np.random.default_rng(4).uniform(-1, 1, (96, lay.N)).astype(np.float16)
    L = pb.Layer.from_synth(lay)
    try:
        pb.pp_set_tuning(12, 2)
        ya = pb.pp_forward(L, _dev(x), 1).cpu().numpy()
        yb = pb.pp_forward(L, _dev(x), 1).cpu().numpy()
    finally:
        pb.pp_set_tuning(12, 1)
    assert np.array_equal(ya, yb)
    L.close()


def test_layer_created_without_tile_copy(pb):
    """A layer created while tuning key 9 is 0 keeps no second copy of its tiles: every batch runs the
    matrix-vector kernels, also after the key is back at its default, and clones inherit that."""
    lay = _rand_layer(77, 4 * 64, 6 * 64, 64, np.float16, density=0.6)
    x = np.random.default_rng(5).uniform(-1, 1, (40, lay.N)).astype(np.float16)
    pb.pp_set_tuning(9, 0)
    try:
        L = pb.Layer.from_synth(lay)
    finally:
        pb.pp_set_tuning(9, 9)
    C = L.clone()
    assert L.launch_info(40)["kernel"] in ("gemv", "stream") and C.launch_info(40)["kernel"] in ("gemv", "stream")
    y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=1)
    for layer in (L, C):
        _check(pb.pp_forward(layer, _dev(x), 1).cpu().numpy(), y_ref, a, np.float16, "no tile copy")
    full = pb.Layer.from_synth(lay)
    assert full.launch_info(40)["kernel"] in ("tile", "tile_cluster", "tile_persist")
    L.close(); C.close(); full.close()


def test_config5_batch128_tile_path_sampled_rows(pb, tile_kernel):
    """Full size (8192 x 8192, density 25 %), batch 128, in the launch configuration the bench times;
    the oracle evaluates a sample of output rows."""
    wl = synth.config5(k=32, batch=128)
    lay = wl.layers[0]
    L = pb.Layer.from_synth(lay)
    y = pb.pp_forward(L, _dev(wl.x), 0).cpu().numpy()
    assert L.status() == 0
    W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    rows = np.random.default_rng(0).choice(lay.M, 96, replace=False).astype(np.int32)
    y_ref, a = po.dense_forward_rows(W, None, wl.x.astype(np.float64), 0, rows)
    _check(y[:, rows], y_ref, a, np.float16, "config 5 batch 128 sampled")
    L.close()


# ------------------------------------------------------------------ permutation elimination (Sections 4.2.2, 4.2.3)
def _check_pivoted(y_piv, y_ref, a_ref, omap, dtype, what):
    real = omap >= 0
    assert np.all(y_piv[:, ~real] == 0.0), f"{what}: padding positions must hold 0"
    _check(y_piv[:, real], y_ref[:, omap[real]], a_ref[:, omap[real]], dtype, what)


@pytest.mark.parametrize("dtype,B", [(np.float32, 32), (np.float16, 16), (np.float16, 64)])
@pytest.mark.parametrize("batch", [1, 5, 40, 130])
def test_forward_pivoted_output(pb, dtype, B, batch):
    """Output permutation elimination (Section 4.2.2): the result left in pivoted row order, relabelled by
    the map the layer hands out, equals the oracle's; batch 130 with fp16, B = 64 runs the tensor-core
    kernels.  On integer data the relabelled result has the bits of the ordinary call."""
    lay = _rand_layer(1200 + B + batch, 5 * B - 3, 9 * B - 7, B, dtype, density=0.45, empty_rows=(2,))
    x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(dtype)
    L = pb.Layer.from_synth(lay)
    omap = L.output_map()
    assert omap.shape == (5 * B,) and sorted(omap[omap >= 0].tolist()) == list(range(lay.M))
    assert np.array_equal(omap, np.where(lay.row_perm < lay.M, lay.row_perm, -1))
    for kern in ((2, 0) if (dtype == np.float16 and B == 64 and batch >= 64) else (1,)):
        pb.pp_set_tuning(12, kern)
        try:
            for act in (0, 1):
                y_piv = pb.pp_forward_pivoted(L, _dev(x), act).cpu().numpy()
                y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=act, threads=8)
                _check_pivoted(y_piv, y_ref, a, omap, dtype, f"pivoted {dtype.__name__} B={B} batch={batch} act={act}")
        finally:
            pb.pp_set_tuning(12, 1)
    L.close()
    lay = _rand_layer(1300 + B + batch, 4 * B - 1, 6 * B - 5, B, dtype, density=0.5, integer=True)
    x = np.random.default_rng(5).integers(-2, 3, (batch, lay.N)).astype(dtype)
    L = pb.Layer.from_synth(lay)
    omap = L.output_map()
    y = pb.pp_forward(L, _dev(x), 1).cpu().numpy()
    y_piv = pb.pp_forward_pivoted(L, _dev(x), 1).cpu().numpy()
    assert np.array_equal(y_piv[:, omap >= 0], y[:, omap[omap >= 0]])
    assert L.status() == 0
    L.close()


@pytest.mark.parametrize("dtype,B", [(np.float32, 32), (np.float16, 64)])
def test_chain_identity_links_and_pivoted_output(pb, dtype, B):
    """Cross-layer permutation elimination (Section 4.2.3): when the consumer's column permutation equals
    the producer's row permutation the link is detected as the identity and stored without an index
    array; same bits as the mapped store, oracle parity, and the final output may stay pivoted
    (Section 4.2.2).  Link 1 is an identity, link 2 is not (different permutations), link 3 is not
    (different padded lengths would be needed: here it has an unequal permutation too)."""
    dims = [7 * B - 5, 6 * B, 5 * B, 4 * B - 3]          # M of layers 0 and 1 are multiples of B: no padding rows
    lays = []
    for l in range(3):
        ll = _rand_layer(1400 + l + B, dims[l + 1], dims[l], B, dtype, density=0.6)
        ll.act = 1 if l < 2 else 0
        lays.append(ll)
    lays[1].col_perm = lays[0].row_perm.copy()           # P^{AB} = I for link 0 -> 1
    x = np.random.default_rng(9).uniform(-1, 1, (6, dims[0])).astype(dtype)
    L = [pb.Layer.from_synth(l) for l in lays]
    chain = pb.Chain(L, [l.act for l in lays], max_batch=8)
    assert chain.link_info().tolist() == [0, 1, 0]
    res = po.chain_forward(lays, x.astype(np.float64), round_intermediate="f16" if dtype == np.float16 else "f32",
                           threads=4)
    y1 = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
    pb.pp_set_tuning(13, 0)
    try:
        y0 = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
    finally:
        pb.pp_set_tuning(13, 1)
    assert np.array_equal(y1, y0)
    bound = _chain_bound(lays, res, TOL[np.dtype(dtype)])
    worst = np.max(np.abs(y1.astype(np.float64) - res[-1][1]) / bound)
    assert worst <= 1.0, f"chain with an identity link: worst error/bound {worst:.3f}"
    chain.set_output_pivoted(True)
    omap = chain.output_map()
    yp = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
    assert yp.shape == (6, 4 * B)
    assert np.array_equal(yp[:, omap >= 0], y1[:, omap[omap >= 0]]) and np.all(yp[:, omap < 0] == 0)
    chain.set_output_pivoted(False)
    assert np.array_equal(pb.pp_chain_forward(chain, _dev(x)).cpu().numpy(), y1)
    chain.close()
    for l in L:
        l.close()


def test_chain_identity_link_with_padding_rows(pb):
    """An identity link whose producer has padding rows (M not a multiple of B): the padding rows hold
    act(0) = 0 and land on the consumer's padding columns."""
    B, dtype = 16, np.float32
    dims = [5 * B - 2, 4 * B - 5, 3 * B]
    lays = [_rand_layer(1500 + l, dims[l + 1], dims[l], B, dtype, density=0.7, integer=True) for l in range(2)]
    lays[0].act, lays[1].act = 1, 0
    lays[1].col_perm = lays[0].row_perm.copy()
    x = np.random.default_rng(2).integers(-2, 3, (3, dims[0])).astype(dtype)
    L = [pb.Layer.from_synth(l) for l in lays]
    chain = pb.Chain(L, [1, 0], max_batch=4)
    assert chain.link_info().tolist() == [0, 1]
    y = pb.pp_chain_forward(chain, _dev(x)).cpu().numpy()
    res = po.chain_forward(lays, x.astype(np.float64))
    assert np.array_equal(y.astype(np.float64), res[-1][1])
    chain.close()
    for l in L:
        l.close()


def test_forward_host_matches_device_call(pb):
    """pp_forward_host (host buffers in, host buffers out) gives the bits of pp_forward, also when a second
    call brings a larger batch (the staging buffers grow); pageable buffers (copy-engine transfers), page-locked
    ones (moved by the library's own kernels, with lengths and addresses that are no multiples of 16 bytes) and
    page-locked ones with tuning key 16 = 0."""
    lay = _rand_layer(4242, 300, 500, 32, np.float16, density=0.4)
    L = pb.Layer.from_synth(lay)
    try:
        for batch, pin, key16, offset in ((1, True, 1, 0), (5, False, 1, 0), (3, True, 1, 0), (40, True, 1, 0),
                                          (2, True, 0, 0), (1, True, 1, 1), (7, True, 1, 3)):
            pb.pp_set_tuning(16, key16)
            x = np.random.default_rng(batch).uniform(-1, 1, (batch, lay.N)).astype(np.float16)
            if pin:                         # views into page-locked buffers, optionally off the 16-byte grid
                xbuf = torch.empty(batch * lay.N + 8, dtype=torch.float16).pin_memory()
                ybuf = torch.full((batch * lay.M + 8,), float("nan"), dtype=torch.float32).pin_memory()
                xh = xbuf[offset:offset + batch * lay.N].view(batch, lay.N)
                xh.copy_(torch.from_numpy(x))
                out = ybuf[offset:offset + batch * lay.M].view(batch, lay.M)
                yh = pb.pp_forward_host(L, xh, 1, out=out)
                assert torch.isnan(ybuf[:offset]).all() and torch.isnan(ybuf[offset + batch * lay.M:]).all()
            else:
                yh = pb.pp_forward_host(L, torch.from_numpy(x), 1)
            yd = pb.pp_forward(L, _dev(x), 1).cpu()
            assert torch.equal(yh, yd), (batch, pin, key16, offset)
            y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=1, threads=4)
            _check(yh.numpy(), y_ref, a, np.float16, f"host call batch {batch}")
    finally:
        pb.pp_set_tuning(16, 1)
    L.close()


@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("batch", [2, 3, 5, 8])
@pytest.mark.parametrize("key7", [2, 1])
def test_several_vectors_through_the_index_array(pb, B, batch, key7):
    """fp16, 2..8 input vectors: read through the column index array inside the multiply loop (tuning key 7 = 2,
    the default: no pivoted copy of x, no pre-pass) or permuted in shared memory first (key 7 = 1); ragged N,
    padding columns, a block-row without tiles; real values within tolerance and small integers bit for bit."""
    pb.pp_set_tuning(7, key7)
    try:
        for integer in (False, True):
            lay = _rand_layer(900 + B + batch, 6 * B - 5, 10 * B - 3, B, np.float16, density=0.5, empty_rows=(1,),
                              integer=integer)
            rng = np.random.default_rng(batch)
            x = (rng.integers(-2, 3, (batch, lay.N)) if integer else rng.uniform(-1, 1, (batch, lay.N))).astype(np.float16)
            for act in (0, 1):
                y = _run_and_check(pb, lay, x, act, f"direct multi B={B} batch={batch}")
                if integer:
                    y_ref, _, _ = po.layer_forward(lay, x.astype(np.float64), act=act)
                    assert np.array_equal(y.astype(np.float64), y_ref)
    finally:
        pb.pp_set_tuning(7, 2)


@pytest.mark.parametrize("tile_kernel,pdl", [(1, 1), (0, 1), (2, 0), (3, 1)])
def test_interleaved_calls_of_several_layers_without_synchronising(pb, tile_kernel, pdl):
    """Calls of different layers, batches and kernel families are enqueued back to back (each launch may begin
    while the previous one is still running: dependent launches) and only checked at the end."""
    rng = np.random.default_rng(100 + tile_kernel)
    specs = [(700, 900, 64, np.float16, 1.0), (333, 200, 16, np.float32, 0.3), (2100, 1500, 64, np.float16, 0.5),
             (650, 480, 32, np.float16, 0.2)]
    pb.pp_set_tuning(12, tile_kernel)
    pb.pp_set_tuning(8, pdl)
    try:
        lays = [_rand_layer(50 + i, M, N, B, dt, density=d) for i, (M, N, B, dt, d) in enumerate(specs)]
        Ls = [pb.Layer.from_synth(l) for l in lays]
        plan = []
        for batch in (1, 130, 9, 1, 40, 2, 128, 16, 1, 31, 8, 64):
            for i in rng.permutation(len(lays))[:3]:
                x = rng.uniform(-1, 1, (batch, lays[i].N)).astype(lays[i].tile_values.dtype)
                plan.append((int(i), x, int(rng.integers(0, 2))))
        xs = [_dev(x) for _, x, _ in plan]
        torch.cuda.synchronize()
        outs = [pb.pp_forward(Ls[i], xd, act) for (i, _, act), xd in zip(plan, xs)]
        torch.cuda.synchronize()
        kernels = {Ls[i].launch_info(x.shape[0])["kernel"] for i, x, _ in plan}
        assert {"stream", "gemv"} <= kernels and any(k.startswith("tile") for k in kernels)
        for (i, x, act), yd in zip(plan, outs):
            y_ref, _, a = po.layer_forward(lays[i], x.astype(np.float64), act=act, threads=8)
            _check(yd.cpu().numpy(), y_ref, a, lays[i].tile_values.dtype, f"layer {i} batch {x.shape[0]}")
        for L in Ls:
            assert L.status() == 0
            L.close()
    finally:
        pb.pp_set_tuning(12, 1)
        pb.pp_set_tuning(8, 1)


@pytest.mark.parametrize("dtype,B", [(np.float16, 64), (np.float16, 16), (np.float32, 32)])
def test_inputs_ready_before_the_stream(pb, dtype, B):
    """Tuning key 17: inputs that were complete before the calls were enqueued are fetched ahead of the dependency
    wait; only the writes wait for the previous kernel.  Many calls of the same layers back to back (so consecutive
    kernels share exchange slots, counters and shared strips) must give the bits of the ordinary calls."""
    rng = np.random.default_rng(1700 + B)
    lays = [_rand_layer(170 + B, 1100, 1300, B, dtype, density=0.5, integer=True),
            _rand_layer(171 + B, 260, 200, B, dtype, density=0.7, integer=True)]
    Ls = [pb.Layer.from_synth(l) for l in lays]
    plan = [(int(rng.integers(0, 2)), int(b)) for b in (1, 1, 3, 1, 8, 1, 2, 1, 1, 5, 1, 1) for _ in range(3)]
    xs = [rng.integers(-3, 4, (b, lays[i].N)).astype(dtype) for i, b in plan]
    xd = [_dev(x) for x in xs]
    torch.cuda.synchronize()                         # every input is complete before the first call is enqueued
    try:
        pb.pp_set_tuning(17, 1)
        outs = [pb.pp_forward(Ls[i], x, 1) for (i, _), x in zip(plan, xd)]
        torch.cuda.synchronize()
    finally:
        pb.pp_set_tuning(17, 0)
    assert all(Ls[i].launch_info(b)["kernel"] == "stream" for i, b in plan)
    for (i, b), x, yd in zip(plan, xs, outs):
        y_ref, _, _ = po.layer_forward(lays[i], x.astype(np.float64), act=1, threads=8)
        assert np.array_equal(yd.cpu().numpy().astype(np.float64), y_ref), f"layer {i} batch {b}"
    for L in Ls:
        assert L.status() == 0
        L.close()
    with pytest.raises(pb.PPError):
        pb.pp_set_tuning(17, 2)


@pytest.mark.parametrize("k", [128, 16])
def test_inputs_ready_full_size(pb, k):
    """Tuning key 17 on the full-size layer, the launch configuration the bench times: three calls back to back on one
    layer (shared exchange slots and counters), each against the fp64 product."""
    wl = synth.config5(k=k, batch=1)
    lay = wl.layers[0]
    rng = np.random.default_rng(171 + k)
    xs = [wl.x] + [rng.uniform(-1, 1, wl.x.shape).astype(wl.x.dtype) for _ in range(2)]
    xd = [_dev(x) for x in xs]
    L = pb.Layer.from_synth(lay)
    torch.cuda.synchronize()
    try:
        pb.pp_set_tuning(17, 1)
        outs = [pb.pp_forward(L, x, lay.act) for x in xd]
        torch.cuda.synchronize()
    finally:
        pb.pp_set_tuning(17, 0)
    assert L.launch_info(1)["kernel"] == "stream"
    for i, (x, yd) in enumerate(zip(xs, outs)):
        y_ref, _, a = po.layer_forward(lay, x.astype(np.float64), act=lay.act, threads=8)
        _check(yd.cpu().numpy(), y_ref, a, lay.tile_values.dtype, f"k={k} call {i}")
    assert L.status() == 0
    L.close()
