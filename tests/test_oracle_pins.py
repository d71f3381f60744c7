"""Pins for the CPU oracle: every check compares it with something other than
itself -- hand-worked values, the paper's index-array example, explicit
permutation-matrix products, library matmuls and closed forms."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth


def _layer_from_golden(g):
    M, N, B = int(g["M"][0]), int(g["N"][0]), int(g["B"][0])
    return dict(M=M, N=N, B=B,
                row_perm=np.array(g["row_perm"], dtype=np.int32),
                col_perm=np.array(g["col_perm"], dtype=np.int32),
                tile_list=np.array(g["tile_list"], dtype=np.int32).reshape(-1, 2),
                tile_values=np.array(g["tile_values"]).reshape(-1, B, B))


# ---------------------------------------------------------------- hand example
def test_hand_4x4_reconstruct(hand4):
    L = _layer_from_golden(hand4)
    W = po.reconstruct(**L)
    assert np.array_equal(W, np.array(hand4["W"]).reshape(4, 4))


def test_hand_4x4_forward(hand4):
    L = _layer_from_golden(hand4)
    W = po.reconstruct(**L)
    x = np.array(hand4["x"])
    y, s, a = po.dense_forward(W, np.array(hand4["bias"]), x, act=1)
    assert np.array_equal(s[0], hand4["pre_act"])
    assert np.array_equal(a[0], hand4["absW_absx"])
    assert np.array_equal(y[0], hand4["y_relu"])
    y0, s0, _ = po.dense_forward(W, None, x, act=0)
    assert np.array_equal(y0[0], hand4["Wx"])
    ys = po.structured_forward(bias=np.array(hand4["bias"]), x=x, act=1, **L)
    assert np.array_equal(ys[0], hand4["y_relu"])


def test_hand_4x4_chain(hand4):
    lay = synth.hand_example()
    lay2 = synth.hand_example()
    lay2.act = synth.ACT_IDENTITY
    res = po.chain_forward([lay, lay2], np.array(hand4["x"]))
    assert np.array_equal(res[0][1][0], hand4["y_relu"])
    assert np.array_equal(res[1][1][0], hand4["chain_y"])


def test_hand_example_matches_fixture(hand4):
    """The in-code copy of the example used by other tests is the fixture."""
    lay = synth.hand_example()
    assert list(lay.row_perm) == hand4["row_perm"]
    assert list(lay.col_perm) == hand4["col_perm"]
    assert list(lay.tile_list.ravel()) == hand4["tile_list"]
    assert list(lay.tile_values.ravel()) == hand4["tile_values"]
    assert list(lay.bias) == hand4["bias"]


# ------------------------------------------------------- index-array convention
def test_cab_convention():
    """Section 4.1.4: the index array of "cab" relative to "abc" is [2,0,1],
    i.e. out[k] = in[idx[k]].  With an identity tile and identity row_perm the
    layer output is exactly the gathered input."""
    x = np.array([ord("a"), ord("b"), ord("c")], dtype=np.float64)
    y = po.structured_forward(3, 3, 3, [0, 1, 2], [2, 0, 1], [[0, 0]], np.eye(3), None, x, 0)
    assert "".join(chr(int(v)) for v in y[0]) == "cab"
    W = po.reconstruct(3, 3, 3, [0, 1, 2], [2, 0, 1], [[0, 0]], np.eye(3))
    y2, _, _ = po.dense_forward(W, None, x, 0)
    assert "".join(chr(int(v)) for v in y2[0]) == "cab"


def test_row_scatter_convention():
    """Listing 1's last step stores acc[i] to a_out[P_row[i]]: with an identity
    tile and identity col_perm, y[row_perm[i]] = x[i]."""
    x = np.array([10.0, 20.0, 30.0])
    y = po.structured_forward(3, 3, 3, [2, 0, 1], [0, 1, 2], [[0, 0]], np.eye(3), None, x, 0)
    assert list(y[0]) == [20.0, 30.0, 10.0]
    W = po.reconstruct(3, 3, 3, [2, 0, 1], [0, 1, 2], [[0, 0]], np.eye(3))
    assert list(po.dense_forward(W, None, x, 0)[0][0]) == [20.0, 30.0, 10.0]


# ------------------------------------------------------------------ brute force
def _brute_W(M, N, B, row_perm, col_perm, tile_list, tile_values):
    """P_r^T W_piv P_c with explicit 0/1 matrices and numpy matmul, cropped to M x N."""
    Mb, Nb = -(-M // B), -(-N // B)
    Wp = np.zeros((Mb * B, Nb * B))
    for t, (br, bc) in enumerate(tile_list):
        Wp[br * B:(br + 1) * B, bc * B:(bc + 1) * B] = tile_values[t]
    Pr = np.zeros((Mb * B, Mb * B)); Pc = np.zeros((Nb * B, Nb * B))
    Pr[np.arange(Mb * B), row_perm] = 1.0      # (P x)[k] = x[perm[k]]
    Pc[np.arange(Nb * B), col_perm] = 1.0
    return (Pr.T @ Wp @ Pc)[:M, :N]


@pytest.mark.parametrize("seed", range(40))
def test_brute_force_tiny(seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 5))
    M = int(rng.integers(1, 13)); N = int(rng.integers(1, 13))
    Mb, Nb = -(-M // B), -(-N // B)
    T = int(rng.integers(0, Mb * Nb + 1))
    flat = rng.choice(Mb * Nb, size=T, replace=False)
    tl = np.stack([flat // Nb, flat % Nb], axis=1).astype(np.int32).reshape(-1, 2)
    tv = rng.standard_normal((T, B, B))
    rp = rng.permutation(Mb * B).astype(np.int32); cp = rng.permutation(Nb * B).astype(np.int32)
    bias = rng.standard_normal(M)
    x = rng.standard_normal((3, N))
    Wb = _brute_W(M, N, B, rp, cp, tl, tv)
    W = po.reconstruct(M, N, B, rp, cp, tl, tv)
    assert np.array_equal(W, Wb)
    for act in (0, 1):
        ref = x @ Wb.T + bias
        if act:
            ref = np.maximum(ref, 0.0)
        y, s, a = po.dense_forward(W, bias, x, act)
        np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)
        np.testing.assert_allclose(a, np.abs(x) @ np.abs(Wb).T, rtol=0, atol=1e-12)
        ys = po.structured_forward(M, N, B, rp, cp, tl, tv, bias, x, act)
        np.testing.assert_allclose(ys, ref, rtol=0, atol=1e-12)


# ------------------------------------------- row-sampled product (used at full size)
def test_rows_variant_hand_4x4(hand4):
    """The row-sampled product on the hand-worked example: rows in a shuffled order, one of them twice."""
    L = _layer_from_golden(hand4)
    W = po.reconstruct(**L)
    x = np.array(hand4["x"])
    rows = [3, 0, 3, 2, 1]
    y, a = po.dense_forward_rows(W, np.array(hand4["bias"]), x, 1, rows)
    assert list(y[0]) == [hand4["y_relu"][r] for r in rows]
    assert list(a[0]) == [hand4["absW_absx"][r] for r in rows]
    y0, _ = po.dense_forward_rows(W, None, x, 0, rows)
    assert list(y0[0]) == [hand4["Wx"][r] for r in rows]


@pytest.mark.parametrize("act", [0, 1])
def test_rows_variant_against_library_matmul(act):
    """Ragged layer with a bias, three input vectors: the sampled rows (shuffled, one repeated, the last
    row of W included) must equal the same columns of a numpy matrix product and of the full oracle
    product, for the values and for the magnitudes |W||x|."""
    rng = np.random.default_rng(77)
    M, N, B = 37, 53, 8
    Mb, Nb = -(-M // B), -(-N // B)
    T = 17
    flat = rng.choice(Mb * Nb, size=T, replace=False)
    tl = np.stack([flat // Nb, flat % Nb], axis=1).astype(np.int32)
    tv = rng.standard_normal((T, B, B))
    rp = rng.permutation(Mb * B).astype(np.int32); cp = rng.permutation(Nb * B).astype(np.int32)
    bias = rng.standard_normal(M)
    x = rng.standard_normal((3, N))
    Wb = _brute_W(M, N, B, rp, cp, tl, tv)
    W = po.reconstruct(M, N, B, rp, cp, tl, tv)
    rows = np.concatenate([rng.permutation(M)[:20], [M - 1, 0, M - 1]]).astype(np.int32)
    y, a = po.dense_forward_rows(W, bias, x, act, rows)
    assert y.shape == (3, rows.size) and a.shape == (3, rows.size)
    ref = x @ Wb.T + bias
    if act:
        ref = np.maximum(ref, 0.0)
    np.testing.assert_allclose(y, ref[:, rows], rtol=0, atol=1e-12)
    np.testing.assert_allclose(a, (np.abs(x) @ np.abs(Wb).T)[:, rows], rtol=0, atol=1e-12)
    yf, _, af = po.dense_forward(W, bias, x, act)
    assert np.array_equal(y, yf[:, rows]) and np.array_equal(a, af[:, rows])
    # no rows at all is a valid request
    y_e, a_e = po.dense_forward_rows(W, bias, x, act, np.zeros(0, dtype=np.int32))
    assert y_e.shape == (3, 0) and a_e.shape == (3, 0)


# -------------------------------------------------------------------- invariants
def test_identity_perms_density_one_is_plain_gemv():
    rng = np.random.default_rng(7)
    M, N, B = 24, 40, 8
    Wd = rng.standard_normal((M, N))
    tl = np.array([(br, bc) for br in range(M // B) for bc in range(N // B)], dtype=np.int32)
    tv = np.stack([Wd[br * B:(br + 1) * B, bc * B:(bc + 1) * B] for br, bc in tl])
    W = po.reconstruct(M, N, B, np.arange(M), np.arange(N), tl, tv)
    assert np.array_equal(W, Wd)
    x = rng.standard_normal((2, N)); b = rng.standard_normal(M)
    y, _, _ = po.dense_forward(W, b, x, 0)
    np.testing.assert_allclose(y, x @ Wd.T + b, rtol=0, atol=1e-12)


def test_B1_is_elementwise_coo():
    rng = np.random.default_rng(8)
    M, N = 9, 11
    T = 30
    flat = rng.choice(M * N, size=T, replace=False)
    tl = np.stack([flat // N, flat % N], axis=1).astype(np.int32)
    tv = rng.standard_normal((T, 1, 1))
    rp = rng.permutation(M); cp = rng.permutation(N)
    x = rng.standard_normal(N)
    ref = np.zeros(M)
    for (i, j), v in zip(tl, tv.ravel()):
        ref[rp[i]] += v * x[cp[j]]
    y, _, _ = po.layer_forward(synth.Layer(M, N, 1, rp, cp, tl, tv, None), x)
    np.testing.assert_allclose(y[0], ref, rtol=0, atol=1e-13)


def test_structured_equals_dense_on_config_shapes():
    wl = synth.config3(batch=2, scale=1 / 16)
    for lay in wl.layers:
        x = np.random.default_rng(3).uniform(0, 1, size=(2, lay.N))
        y, _, a = po.layer_forward(lay, x)
        ys = po.structured_forward(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list,
                                   lay.tile_values, lay.bias, x, lay.act)
        assert np.all(np.abs(y - ys) <= 1e-12 * (a + 1.0))


def test_tile_order_and_relabelling_invariance():
    wl = synth.config1(scale=0.25)
    lay = wl.layers[0]
    W = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    rng = np.random.default_rng(5)
    o = rng.permutation(lay.T)
    W2 = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list[o], lay.tile_values[o])
    assert np.array_equal(W, W2)
    # relabel rows inside every block-row: row_perm o pi with the tile rows moved the same way
    B = lay.B
    pi = rng.permutation(B)
    rp2 = lay.row_perm.reshape(-1, B)[:, pi].ravel()
    W3 = po.reconstruct(lay.M, lay.N, B, rp2, lay.col_perm, lay.tile_list, lay.tile_values[:, pi, :])
    assert np.array_equal(W, W3)


def test_padding_and_empty_block_rows():
    """M, N not multiples of B; block-row 1 has no tile, so y = act(bias) there."""
    M, N, B = 5, 7, 4
    rp = np.array([4, 0, 7, 1, 2, 6, 3, 5], dtype=np.int32)     # 5,6,7 are phantom rows
    cp = np.array([7, 6, 5, 4, 3, 2, 1, 0], dtype=np.int32)     # 7 is a phantom column
    tl = np.array([[0, 0], [0, 1]], dtype=np.int32)
    tv = np.arange(32, dtype=np.float64).reshape(2, 4, 4) + 1
    bias = np.array([1.0, -2.0, 3.0, -4.0, 5.0])
    x = np.arange(1, 8, dtype=np.float64)
    W = po.reconstruct(M, N, B, rp, cp, tl, tv)
    assert np.array_equal(W, _brute_W(M, N, B, rp, cp, tl, tv))
    y, _, _ = po.dense_forward(W, bias, x, 1)
    # rows fed by pivoted rows 4..7 (block-row 1) see no tile: originals 2 and 3 (6, 5 are phantom)
    assert y[0][2] == 3.0 and y[0][3] == 0.0
    ys = po.structured_forward(M, N, B, rp, cp, tl, tv, bias, x, 1)
    np.testing.assert_allclose(ys, y, atol=1e-12)


def test_errors():
    with pytest.raises(po.OracleError):
        po.reconstruct(4, 4, 2, [0, 1, 2, 2], [0, 1, 2, 3], [[0, 0]], np.zeros((1, 2, 2)))
    with pytest.raises(po.OracleError):
        po.reconstruct(4, 4, 2, [0, 1, 2, 3], [0, 1, 2, 3], [[0, 0], [0, 0]], np.zeros((2, 2, 2)))
    with pytest.raises(po.OracleError):
        po.reconstruct(4, 4, 2, [0, 1, 2, 3], [0, 1, 2, 3], [[2, 0]], np.zeros((1, 2, 2)))


# ------------------------------------------------------------------ observations
def test_observation_1_pointwise_ops_commute_with_permutations():
    rng = np.random.default_rng(11)
    v = rng.standard_normal(64); p = rng.permutation(64)
    assert np.array_equal(np.maximum(v, 0)[p], np.maximum(v[p], 0))
    sm = lambda u: np.exp(u - u.max()) / np.exp(u - u.max()).sum()
    np.testing.assert_allclose(sm(v)[p], sm(v[p]), rtol=1e-15)


def test_chain_equals_manual_composition():
    wl = synth.config3(batch=3, scale=1 / 16)
    res = po.chain_forward(wl.layers, wl.x, round_intermediate=None)
    cur = wl.x.astype(np.float64)
    for lay in wl.layers:
        W = _brute_W(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list,
                     lay.tile_values.astype(np.float64))
        cur = cur @ W.T + lay.bias
        if lay.act:
            cur = np.maximum(cur, 0)
    np.testing.assert_allclose(res[-1][1], cur, rtol=1e-12, atol=1e-12)


def test_chain_rounding_points():
    """With fp16 rounding of intermediates, layer l+1 sees exactly fp16 values."""
    wl = synth.config3(batch=1, scale=1 / 16)
    res = po.chain_forward(wl.layers, wl.x, round_intermediate="f16")
    for li in (1, 2):
        xin = res[li][0]
        assert np.array_equal(xin, xin.astype(np.float16).astype(np.float64))
    assert res[0][0].dtype == np.float64


# ------------------------------------------------------------------------- LSTM
def _lstm_W(H, wi, wf, wg, wo):
    """I = 1: every gate row reads only the scalar input x_t with the given weight."""
    W = np.zeros((4 * H, 1 + H))
    for k, w in enumerate((wi, wf, wg, wo)):
        W[k * H:(k + 1) * H, 0] = w
    return W


@pytest.mark.parametrize("wi,wf,wg,wo,c_expect,h_expect", [
    (50, -50, 50, 50, 1.0, np.tanh(1.0)),          # input open, forget closed: c = tanh(g) = 1
    (-50, 50, 50, 50, 0.3, np.tanh(0.3)),          # input closed, forget open: c = c0
    (50, 50, -50, 50, 0.3 - 1.0, np.tanh(-0.7)),   # candidate -1 added to c0
    (50, 50, 50, -50, 1.3, 0.0),                   # output closed: h = 0
])
def test_lstm_saturated_gates(wi, wf, wg, wo, c_expect, h_expect):
    H = 3
    W = _lstm_W(H, wi, wf, wg, wo)
    h, c, _ = po.lstm_forward(W, np.ones((1, 1)), H, c0=np.full(H, 0.3))
    np.testing.assert_allclose(c, c_expect, atol=1e-12)
    np.testing.assert_allclose(h, h_expect, atol=1e-12)


def test_lstm_counter_closed_form():
    """All gates saturated open: c_t = t, h_t = tanh(t)."""
    H = 2
    W = _lstm_W(H, 50, 50, 50, 50)
    h, c, hs = po.lstm_forward(W, np.ones((5, 1)), H)
    np.testing.assert_allclose(c, 5.0, atol=1e-10)
    np.testing.assert_allclose(hs[:, 0], np.tanh(np.arange(1, 6)), atol=1e-10)


def test_lstm_zero_weights_and_recurrence_wiring():
    H = 4
    h, c, _ = po.lstm_forward(np.zeros((4 * H, 2 + H)), np.ones((7, 2)), H)
    assert np.all(h == 0) and np.all(c == 0)
    # h feeds back through columns [I, I+H): gate g of unit 0 reads h_{t-1} of unit 1 only
    W = np.zeros((4 * H, 1 + H))
    W[0:H, 0] = 50; W[H:2 * H, 0] = -50; W[3 * H:4 * H, 0] = 50       # i open, f closed, o open
    W[2 * H + 1, 0] = 0.5                                             # unit 1 candidate from x
    W[2 * H + 0, 1 + 1] = 2.0                                         # unit 0 candidate from h[1]
    _, _, hs = po.lstm_forward(W, np.ones((2, 1)), H)
    h1_unit1 = np.tanh(np.tanh(0.5))
    np.testing.assert_allclose(hs[0, 1], h1_unit1, atol=1e-12)
    np.testing.assert_allclose(hs[1, 0], np.tanh(np.tanh(2.0 * h1_unit1)), atol=1e-12)


# ------------------------------------------------ irregular block structure (Section 4.1.5)
def test_hand_blocks_4x4(hand_blocks4):
    g = hand_blocks4
    rp = np.array(g["row_perm"], dtype=np.int32)
    cp = np.array(g["col_perm"], dtype=np.int32)
    W = po.reconstruct_blocks(4, 4, rp, cp, np.array(g["blocks"], dtype=np.int32).reshape(-1, 4), g["block_values"])
    assert np.array_equal(W, np.array(g["W"]).reshape(4, 4))
    y, s, a = po.dense_forward(W, None, np.array(g["x"]), act=0)
    assert np.array_equal(y[0], g["Wx"])
    assert np.array_equal(a[0], g["absW_absx"])


def _dense_from_blocks(Mp, Np, blocks, values):
    """W_piv assembled by array slicing (not by the oracle's element loop)."""
    Wp = np.zeros((Mp, Np))
    cover = np.zeros((Mp, Np), dtype=np.int64)
    off = 0
    for r0, c0, h, w in blocks:
        Wp[r0:r0 + h, c0:c0 + w] = np.asarray(values[off:off + h * w], dtype=np.float64).reshape(h, w)
        cover[r0:r0 + h, c0:c0 + w] += 1
        off += h * w
    return Wp, cover


@pytest.mark.parametrize("seed", range(6))
def test_blocks_against_permutation_matrices(seed):
    """Random rectangles (unaligned, several per row): Eq. 1 with explicit 0/1 matrices, W = P_r^T W_piv P_c."""
    rng = np.random.default_rng(seed)
    B = int(rng.choice([1, 2, 3, 4]))
    M, N = int(rng.integers(3, 13)), int(rng.integers(3, 13))
    wl = synth.irregular_blocks(900 + seed, M, N, B, wdtype="f32", n_row_cuts=3, n_col_cuts=3, keep=0.5,
                                integer_values=True)
    lay = wl.layers[0]
    Mp, Np = lay.row_perm.size, lay.col_perm.size
    Wp, cover = _dense_from_blocks(Mp, Np, lay.blocks, lay.block_values)
    assert cover.max() == 1
    Pr = np.zeros((Mp, Mp)); Pr[np.arange(Mp), lay.row_perm] = 1.0
    Pc = np.zeros((Np, Np)); Pc[np.arange(Np), lay.col_perm] = 1.0
    W_full = Pr.T @ Wp @ Pc
    W = po.reconstruct_blocks(M, N, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values)
    assert np.array_equal(W, W_full[:M, :N])


def test_blocks_equal_tiles_when_uniform():
    """Blocks that are exactly the tiles of a uniform layer give the same W as the tile form."""
    lay = synth.config1(scale=0.25).layers[0]
    B = lay.B
    blocks = np.array([[br * B, bc * B, B, B] for br, bc in lay.tile_list], dtype=np.int32)
    W_b = po.reconstruct_blocks(lay.M, lay.N, lay.row_perm, lay.col_perm, blocks, lay.tile_values.reshape(-1))
    W_t = po.reconstruct(lay.M, lay.N, B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values)
    assert np.array_equal(W_b, W_t)


def test_blocks_split_and_order_invariance():
    """Cutting a block in two, or listing the blocks in another order, changes nothing."""
    wl = synth.irregular_blocks(77, 40, 56, 8, wdtype="f32", n_row_cuts=4, n_col_cuts=5, keep=0.6)
    lay = wl.layers[0]
    W = po.reconstruct_blocks(lay.M, lay.N, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values)
    blocks2, vals2 = [], []
    offs = np.concatenate([[0], np.cumsum(lay.blocks[:, 2].astype(np.int64) * lay.blocks[:, 3])])
    for k in range(len(lay.blocks) - 1, -1, -1):
        r0, c0, h, w = (int(v) for v in lay.blocks[k])
        v = lay.block_values[offs[k]:offs[k + 1]].reshape(h, w)
        if w >= 2:
            blocks2 += [[r0, c0, h, w // 2], [r0, c0 + w // 2, h, w - w // 2]]
            vals2 += [v[:, :w // 2].ravel(), v[:, w // 2:].ravel()]
        else:
            blocks2.append([r0, c0, h, w]); vals2.append(v.ravel())
    W2 = po.reconstruct_blocks(lay.M, lay.N, lay.row_perm, lay.col_perm, np.array(blocks2, dtype=np.int32),
                               np.concatenate(vals2))
    assert np.array_equal(W, W2)


def test_blocks_rejects_overlap_and_range():
    rp = np.arange(8, dtype=np.int32)
    with pytest.raises(po.OracleError):
        po.reconstruct_blocks(8, 8, rp, rp, [[0, 0, 4, 4], [3, 3, 2, 2]], np.zeros(20))
    with pytest.raises(po.OracleError):
        po.reconstruct_blocks(8, 8, rp, rp, [[6, 0, 4, 4]], np.zeros(16))


def test_paper_square_geometry():
    """Section 5's example: size 512 at fill-in 6.25 % is 16 identical 32 x 32 blocks, one per block-row."""
    lay = synth.paper_square(512, 16, 32).layers[0]
    assert lay.blocks.shape == (16, 4)
    assert np.all(lay.blocks[:, 2] == 32) and np.all(lay.blocks[:, 3] == 32)
    assert len(set(lay.blocks[:, 0])) == 16 and len(set(lay.blocks[:, 1])) == 16
    W = po.reconstruct_blocks(512, 512, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values)
    assert np.count_nonzero(W) == 16 * 32 * 32
    assert np.all(np.count_nonzero(W, axis=1) == 32) and np.all(np.count_nonzero(W, axis=0) == 32)
