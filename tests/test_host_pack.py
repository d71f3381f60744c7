"""Host-side logic of the C library, exercised without a GPU: symbol export,
packer round trip, index arrays, fragment layout, work list, permutation
folding and error codes.  The last test walks the packed arrays with the same
address arithmetic the kernels use and compares with the oracle, so every index
the kernels form is checked for range on the CPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import binding as pb
from paper_1712_01084_b200 import build as pbuild
from paper_1712_01084_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()


def test_library_exports_every_declared_symbol():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(pp_[a-z0-9_]+)\s*\(", src))
    assert {"pp_layer_create", "pp_forward", "pp_chain_forward", "pp_pack_create"} <= names
    L = ctypes.CDLL(pb.LIB_PATH)
    for n in sorted(names):
        assert hasattr(L, n), f"{n} declared in include/ but not exported"


def test_per_device_bookkeeping_selfcheck():
    """Kernel attributes are set once per device; the table that remembers them keeps devices apart."""
    assert pb.lib().pp_selftest_host() == 0


def _random_layer(seed, M, N, B, dtype, density=0.4, bias=True):
    rng = np.random.default_rng(seed)
    Mb, Nb = -(-M // B), -(-N // B)
    T = max(1, int(density * Mb * Nb))
    flat = rng.permutation(Mb * Nb)[:T]          # deliberately unsorted
    tl = np.stack([flat // Nb, flat % Nb], axis=1).astype(np.int32)
    tv = rng.standard_normal((T, B, B)).astype(dtype)
    return synth.Layer(M, N, B, rng.permutation(Mb * B).astype(np.int32), rng.permutation(Nb * B).astype(np.int32),
                       tl, tv, rng.standard_normal(M).astype(np.float32) if bias else None)


def _pack(lay):
    return pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("B", [16, 32, 64])
def test_round_trip_bit_exact(dtype, B):
    lay = _random_layer(B + (dtype == np.float16), 5 * B - 3, 7 * B - 1, B, dtype)
    pk = _pack(lay)
    tl, tv = pk.unpack()
    order = np.lexsort((lay.tile_list[:, 1], lay.tile_list[:, 0]))
    assert np.array_equal(tl, lay.tile_list[order])
    # entries on padding rows / columns are not part of W: they come back as zero, all others bit for bit
    want = lay.tile_values[order].copy()
    for t, (br, bc) in enumerate(tl):
        want[t][lay.row_perm[br * B:(br + 1) * B] >= lay.M, :] = 0
        want[t][:, lay.col_perm[bc * B:(bc + 1) * B] >= lay.N] = 0
    assert np.any(want != lay.tile_values[order])                     # the case has padding inside kept tiles
    assert np.array_equal(tv.view(np.uint8), want.view(np.uint8))


def test_index_arrays():
    lay = _random_layer(3, 100, 200, 16, np.float16)
    pk = _pack(lay)
    row_ptr, col_ptr, tile_col = pk.get("row_ptr"), pk.get("col_ptr"), pk.get("tile_col")
    assert row_ptr[0] == 0 and row_ptr[-1] == lay.T and col_ptr[0] == 0
    order = np.lexsort((lay.tile_list[:, 1], lay.tile_list[:, 0]))
    st = lay.tile_list[order]
    for br in range(pk.Mb):
        k = row_ptr[br + 1] - row_ptr[br]
        seg = tile_col[col_ptr[br]:col_ptr[br + 1]]
        assert len(seg) % 4 == 0 and len(seg) == -(-k // 4) * 4          # 16-byte aligned runs
        assert np.array_equal(seg[:k], st[row_ptr[br]:row_ptr[br + 1], 1])
        assert np.all(seg[k:] == -1)
        assert np.all(np.diff(seg[:k]) > 0)
    g = pk.get("gather_idx"); s = pk.get("scatter_idx"); b = pk.get("bias_piv")
    assert np.array_equal(g, np.where(lay.col_perm < lay.N, lay.col_perm, -1))
    assert np.array_equal(s, np.where(lay.row_perm < lay.M, lay.row_perm, -1))
    real = lay.row_perm < lay.M
    assert np.array_equal(b[real], lay.bias[lay.row_perm[real]]) and np.all(b[~real] == 0)
    inv = pk.get("inv_row_perm")
    assert np.array_equal(inv[lay.row_perm], np.arange(pk.Mb * 16))


def test_fragment_layout_fp32_lane_is_row():
    """fp32, B=32: fragment f of a tile holds columns 4f..4f+3, lane = row."""
    lay = _random_layer(4, 64, 64, 32, np.float32, density=1.0)
    pk = _pack(lay)
    vals = pk.get("values").view(np.float32).reshape(-1, 32, 4)      # [frag][lane][q]
    tl, tv = pk.unpack()
    row_ptr = pk.get("row_ptr")
    for br in range(pk.Mb):
        k = row_ptr[br + 1] - row_ptr[br]
        for j in range(k):
            tile = tv[row_ptr[br] + j]
            for f in range(8):
                frag = row_ptr[br] * 8 + j * 8 + f
                assert np.array_equal(vals[frag], tile[:, 4 * f:4 * f + 4])


def test_fragment_layout_fp16_is_mma_operand():
    """fp16: each 512-byte fragment is a 16x16 block in the register order of the
    m16n8k16 A operand: lane = 4*(row%8) + (col%8)//2, slots (r,c),(r,c+1),(r+8,c),(r+8,c+1),(r,c+8),..."""
    lay = _random_layer(5, 64, 128, 64, np.float16, density=1.0)
    pk = _pack(lay)
    vals = pk.get("values").view(np.float16).reshape(-1, 32, 8)
    tl, tv = pk.unpack()
    row_ptr = pk.get("row_ptr")
    for br in range(pk.Mb):
        k = row_ptr[br + 1] - row_ptr[br]
        for j in range(k):
            tile = tv[row_ptr[br] + j]
            for rg in range(4):
                for f in range(4):
                    frag = row_ptr[br] * 16 + (rg * k + j) * 4 + f
                    blk = tile[16 * rg:16 * rg + 16, 16 * f:16 * f + 16]
                    for lane in range(32):
                        g, t = lane // 4, lane % 4
                        want = [blk[g, 2 * t], blk[g, 2 * t + 1], blk[g + 8, 2 * t], blk[g + 8, 2 * t + 1],
                                blk[g, 2 * t + 8], blk[g, 2 * t + 9], blk[g + 8, 2 * t + 8], blk[g + 8, 2 * t + 9]]
                        assert list(vals[frag, lane]) == want


def test_work_items_cover_every_tile_once():
    for target in (1, 8, 32, 1024):
        pb.pp_set_tuning(0, target)
        try:
            lay = _random_layer(6, 300, 500, 32, np.float16, density=0.3)
            pk = _pack(lay)
            items, row_ptr, col_ptr = pk.get("items"), pk.get("row_ptr"), pk.get("col_ptr")
            seen = np.zeros(lay.T, dtype=int)
            per_br = {}
            for it in items:
                frag_base, rg_stride, nf, col_off, ntiles, br, pn, slot_base = [int(v) for v in it]
                part, nparts = pn & 0xffff, pn >> 16
                k = row_ptr[br + 1] - row_ptr[br]
                j0 = col_off - col_ptr[br]
                assert 0 <= j0 and j0 + ntiles <= max(k, 0) and nf == ntiles * 2 and rg_stride == k * 2
                assert frag_base == row_ptr[br] * 4 + j0 * 2
                seen[row_ptr[br] + j0: row_ptr[br] + j0 + ntiles] += 1
                per_br.setdefault(br, []).append((part, nparts, slot_base))
                assert ntiles * 32 <= 2048
            assert np.all(seen == 1)
            assert sorted(per_br) == list(range(pk.Mb))              # empty block-rows still get an item
            slots = 0
            for br, parts in per_br.items():
                assert [p for p, _, _ in parts] == list(range(parts[0][1]))
                if parts[0][1] > 1:
                    slots += parts[0][1]
            assert slots == pk.n_slots
        finally:
            pb.pp_set_tuning(0, 32)


def test_fold_perm_hand_example(hand4):
    rp = np.array(hand4["row_perm"], dtype=np.int32); cp = np.array(hand4["col_perm"], dtype=np.int32)
    q = pb.pp_fold_perm(rp, 4, cp, 4)
    assert list(q) == hand4["folded_q"]
    # layer-2 pivoted input gathered from layer-1 pivoted output
    y1_piv = np.array(hand4["layer1_piv_act"])
    assert list(y1_piv[q]) == hand4["layer2_x_piv"]


def test_fold_perm_property_with_padding():
    """Gathering the producer's pivoted output through q equals scattering it to
    original order and gathering through the consumer's col_perm (Section 4.2.1)."""
    rng = np.random.default_rng(9)
    M, BA, BB = 1000, 32, 16
    MpA, NpB = -(-M // BA) * BA, -(-M // BB) * BB
    rpA = rng.permutation(MpA).astype(np.int32); cpB = rng.permutation(NpB).astype(np.int32)
    q = pb.pp_fold_perm(rpA, M, cpB, M)
    y_piv = rng.standard_normal(MpA)
    y = np.zeros(M)
    real = rpA < M
    y[rpA[real]] = y_piv[real]
    want = np.where(cpB < M, y[np.minimum(cpB, M - 1)], 0.0)
    got = np.where(q >= 0, y_piv[np.maximum(q, 0)], 0.0)
    assert np.array_equal(got, want)
    # identical permutations fold to the identity (cross-layer permutation elimination)
    assert np.array_equal(pb.pp_fold_perm(rpA, MpA, rpA, MpA), np.arange(MpA))


def test_error_codes():
    lay = _random_layer(7, 64, 64, 32, np.float32)
    bad = lay.row_perm.copy(); bad[0] = bad[1]
    with pytest.raises(pb.PPError) as e:
        pb.Packed(lay.M, lay.N, lay.B, bad, lay.col_perm, lay.tile_list, lay.tile_values)
    assert e.value.status == 2
    tl = np.concatenate([lay.tile_list, lay.tile_list[:1]]); tv = np.concatenate([lay.tile_values, lay.tile_values[:1]])
    with pytest.raises(pb.PPError) as e:
        pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, tl, tv)
    assert e.value.status == 3
    tl = lay.tile_list.copy(); tl[0, 1] = 99
    with pytest.raises(pb.PPError) as e:
        pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, tl, lay.tile_values)
    assert e.value.status == 3
    with pytest.raises(pb.PPError) as e:
        pb.Packed(48, 48, 24, np.arange(48), np.arange(48), np.zeros((1, 2), np.int32), np.zeros((1, 24, 24), np.float32))
    assert e.value.status == 6
    L = pb.lib()
    assert L.pp_pack_create(None, 1, 1, 16, None, None, None, 0, None, 0, None) == 1
    assert L.pp_forward(None, None, None, 1, 0, None) == 1
    assert L.pp_chain_forward(None, None, None, 1, None) == 1
    assert b"permutation" in L.pp_status_string(2)


# ------------------------------------------------ walk the packed arrays like a kernel
def _emulate(pk, x, act, dtype):
    """y from the packed arrays only, forming every index the way the kernels do."""
    B = pk.B
    f16 = dtype == np.float16
    rg_rows = 16 if f16 else min(B, 32)
    kf = 16 if f16 else 128 // rg_rows
    n_rg = B // rg_rows
    vals = pk.get("values").view(dtype)
    n_frag = vals.size * vals.itemsize // 512
    per_lane = 8 if f16 else 4
    vals = vals.reshape(n_frag, 32, per_lane)
    items, tile_col = pk.get("items"), pk.get("tile_col")
    gather, scatter, bias = pk.get("gather_idx"), pk.get("scatter_idx"), pk.get("bias_piv")
    y = np.full(pk.M, np.nan)
    acc = np.zeros(pk.Mb * B)
    for it in items:
        frag_base, rg_stride, nf, col_off, ntiles, br, pn, _ = [int(v) for v in it]
        xs = np.zeros(ntiles * B)
        for c in range(ntiles * B):
            col = tile_col[col_off + c // B]
            assert 0 <= col < pk.Nb
            idx = gather[col * B + c % B]
            assert -1 <= idx < pk.N
            xs[c] = x[idx] if idx >= 0 else 0.0
        for rg in range(n_rg):
            for i in range(nf):
                frag = frag_base + rg * rg_stride + i
                assert 0 <= frag < n_frag
                for lane in range(32):
                    if f16:
                        g, t = lane // 4, lane % 4
                        w = vals[frag, lane].astype(np.float64)
                        k0 = i * 16 + 2 * t
                        acc[br * B + rg * 16 + g] += w[0] * xs[k0] + w[1] * xs[k0 + 1] + w[4] * xs[k0 + 8] + w[5] * xs[k0 + 9]
                        acc[br * B + rg * 16 + g + 8] += w[2] * xs[k0] + w[3] * xs[k0 + 1] + w[6] * xs[k0 + 8] + w[7] * xs[k0 + 9]
                    else:
                        row = lane % rg_rows
                        k0 = i * kf + (lane // rg_rows) * 4
                        acc[br * B + rg * rg_rows + row] += float(np.dot(vals[frag, lane].astype(np.float64), xs[k0:k0 + 4]))
    for i in range(pk.Mb * B):
        if scatter[i] >= 0:
            v = acc[i] + bias[i]
            y[scatter[i]] = max(v, 0.0) if act else v
    return y


@pytest.mark.parametrize("dtype,B", [(np.float32, 16), (np.float32, 32), (np.float32, 64),
                                     (np.float16, 16), (np.float16, 32), (np.float16, 64)])
def test_packed_walk_matches_oracle(dtype, B):
    pb.pp_set_tuning(0, 4)          # small runs so block-rows are split into several items
    try:
        lay = _random_layer(20 + B, 3 * B - 5, 4 * B - 2, B, dtype, density=0.5)
        pk = _pack(lay)
    finally:
        pb.pp_set_tuning(0, 32)
    x = np.random.default_rng(1).uniform(-1, 1, lay.N).astype(dtype)
    got = _emulate(pk, x.astype(np.float64), 1, dtype)
    y, _, a = po.layer_forward(lay, x.astype(np.float64), act=1)
    assert not np.any(np.isnan(got))
    assert np.all(np.abs(got - y[0]) <= 1e-12 * (a[0] + 1))


# ------------------------------------------------ persistent kernel's plan, walked like the kernel
def _emulate_stream(pk, x, act, dtype):
    """Follow the persistent kernel: per-CTA fragment ranges, 16 warps with equal shares, partial
    sums parked per (strip, warp), per-strip sums in warp order, cross-CTA sums in CTA order."""
    NW, MAXS = 16, 48
    B = pk.B
    f16 = dtype == np.float16
    RG = 16 if f16 else min(B, 32)
    vals = pk.get("values").view(dtype)
    F = pk.n_frags
    vals = vals.reshape(F, 32, 8 if f16 else 4)
    xoff, sstart = pk.get("xoff"), pk.get("strip_start")
    ctas, sinfo = pk.get("cta_desc"), pk.get("strip_info")
    gather, scatter, bias = pk.get("gather_idx"), pk.get("scatter_idx"), pk.get("bias_piv")
    xs = np.where(gather >= 0, x[np.maximum(gather, 0)], 0.0)
    S = pk.n_strips
    assert sstart[S] == F and S == pk.Mb * (B // RG)
    covered = np.zeros(F, dtype=int)
    gpart = {}
    y_piv = np.full(S * RG, np.nan)
    listed = np.zeros(S, dtype=int)
    for c, (pb_, pe, s_first, s_count) in enumerate(ctas):
        assert 1 <= s_count <= MAXS and 0 <= s_first and s_first + s_count <= S and pb_ <= pe
        n = pe - pb_
        wb = [pb_ + (n * w) // NW for w in range(NW + 1)]
        loc = sstart[s_first:s_first + s_count + 1]
        park = {}
        for w in range(NW):
            if wb[w] >= wb[w + 1]:
                continue
            ls = 0
            while ls + 1 < s_count and loc[ls + 1] <= wb[w]:
                ls += 1
            seg_end = min(wb[w + 1], loc[ls + 1])
            acc = np.zeros(RG)
            for p in range(wb[w], wb[w + 1]):
                if p == seg_end:
                    assert ls + w not in park
                    park[ls + w] = acc
                    acc = np.zeros(RG)
                    ls += 1
                    while loc[ls + 1] <= p:
                        ls += 1
                    seg_end = min(wb[w + 1], loc[ls + 1])
                assert loc[ls] <= p < loc[ls + 1]
                covered[p] += 1
                xo = xoff[p]
                assert 0 <= xo and xo + (16 if f16 else (8 if RG == 16 else 4)) <= pk.Nb * B
                for lane in range(32):
                    wv = vals[p, lane].astype(np.float64)
                    if f16:
                        g, t = lane // 4, lane % 4
                        k0 = xo + 2 * t
                        acc[g] += wv[0] * xs[k0] + wv[1] * xs[k0 + 1] + wv[4] * xs[k0 + 8] + wv[5] * xs[k0 + 9]
                        acc[g + 8] += wv[2] * xs[k0] + wv[3] * xs[k0 + 1] + wv[6] * xs[k0 + 8] + wv[7] * xs[k0 + 9]
                    else:
                        k0 = xo + (lane // RG) * 4
                        acc[lane % RG] += float(np.dot(wv, xs[k0:k0 + 4]))
            assert ls + w not in park and ls + w < MAXS + NW
            park[ls + w] = acc
        for ls in range(s_count):
            s = s_first + ls
            listed[s] += 1
            lo, hi = max(loc[ls], pb_), min(loc[ls + 1], pe)
            v = np.zeros(RG)
            if lo < hi:
                w_lo = max(w for w in range(NW) if wb[w] <= lo)
                w_hi = max(w for w in range(NW) if wb[w] <= hi - 1)
                for w in range(w_lo, w_hi + 1):
                    if wb[w] < wb[w + 1]:
                        v = v + park.pop(ls + w)
            first_cta, nparts, slot_base, _ = sinfo[s]
            if nparts == 1:
                y_piv[s * RG:(s + 1) * RG] = v
            else:
                assert ls in (0, s_count - 1) and first_cta <= c < first_cta + nparts
                gpart[slot_base + c - first_cta] = v
        assert not park
    assert np.all(covered == 1)
    assert np.array_equal(listed, sinfo[:, 1])
    for s in range(S):
        first_cta, nparts, slot_base, _ = sinfo[s]
        if nparts > 1:
            y_piv[s * RG:(s + 1) * RG] = sum(gpart.pop(slot_base + q) for q in range(nparts))
    assert not gpart
    y = np.full(pk.M, np.nan)
    for i in range(S * RG):
        if scatter[i] >= 0:
            v = y_piv[i] + bias[i]
            y[scatter[i]] = max(v, 0.0) if act else v
    return y


@pytest.mark.parametrize("dtype,B", [(np.float32, 16), (np.float32, 32), (np.float32, 64),
                                     (np.float16, 16), (np.float16, 32), (np.float16, 64)])
@pytest.mark.parametrize("ctas,min_frags,snap", [(296, 128, 25), (7, 1, 0), (3, 1, 50), (1000, 1, 10)])
def test_stream_plan_walk_matches_oracle(dtype, B, ctas, min_frags, snap):
    pb.pp_set_tuning(2, ctas); pb.pp_set_tuning(3, min_frags); pb.pp_set_tuning(4, snap)
    try:
        lay = _random_layer(40 + B, 5 * B - 5, 6 * B - 2, B, dtype, density=0.5)
        lay.tile_list = lay.tile_list[lay.tile_list[:, 0] != 1]          # block-row 1 has no tile
        lay.tile_values = lay.tile_values[:len(lay.tile_list)]
        pk = _pack(lay)
    finally:
        pb.pp_set_tuning(2, 296); pb.pp_set_tuning(3, 128); pb.pp_set_tuning(4, -1)
    x = np.random.default_rng(1).uniform(-1, 1, lay.N).astype(dtype)
    got = _emulate_stream(pk, x.astype(np.float64), 1, dtype)
    y, _, a = po.layer_forward(lay, x.astype(np.float64), act=1)
    assert not np.any(np.isnan(got))
    assert np.all(np.abs(got - y[0]) <= 1e-12 * (a[0] + 1))


def test_stream_plan_many_empty_strips_and_no_tiles():
    """More strips than one CTA may list, most of them empty; and a layer without any tile."""
    rng = np.random.default_rng(3)
    M, N, B = 16 * 300, 64, 16
    tl = np.array([[5, 1], [150, 0], [151, 3], [299, 2]], dtype=np.int32)
    lay = synth.Layer(M, N, B, rng.permutation(M).astype(np.int32), rng.permutation(N).astype(np.int32), tl,
                      rng.standard_normal((4, B, B)).astype(np.float16), rng.standard_normal(M).astype(np.float32))
    for T in (4, 0):
        lay.tile_list, lay.tile_values = tl[:T], lay.tile_values[:T]
        pk = _pack(lay)
        assert np.all(pk.get("cta_desc")[:, 3] <= 48)
        x = rng.uniform(-1, 1, N).astype(np.float16)
        got = _emulate_stream(pk, x.astype(np.float64), 0, np.float16)
        y, _, a = po.layer_forward(lay, x.astype(np.float64), act=0)
        assert np.all(np.abs(got - y[0]) <= 1e-12 * (a[0] + 1))


def test_clustered_tile_plan_covers_every_tile_once():
    """Plan of the clustered tensor-core kernel (fp16, B = 64): per group of 4 block-rows one step per
    distinct tile-column in ascending order, every kept tile in exactly one step slot of its own
    block-row, and four contiguous parts per group that cover the group's steps."""
    for seed, Mb, Nb, density in ((1, 10, 23, 0.3), (2, 4, 4, 1.0), (3, 3, 7, 0.5), (4, 9, 16, 0.1)):
        lay, _ = synth.make_layer(seed, Mb * 64 - 5, Nb * 64 - 3, 64, wdtype="f16", tiles="uniform", density=density)
        pk = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)
        steps, parts = pk.get("tile_steps"), pk.get("tile_parts")
        row_ptr, col_ptr, tile_col = pk.get("row_ptr"), pk.get("col_ptr"), pk.get("tile_col")
        G = -(-Mb // 4)
        assert parts.shape == (G, 5)
        seen = np.zeros(pk.T, dtype=np.int64)
        nxt = 0
        for g in range(G):
            assert parts[g, 0] == nxt and np.all(np.diff(parts[g]) >= 0)
            nxt = parts[g, 4]
            grp = steps[parts[g, 0]:parts[g, 4]]
            assert np.all(np.diff(grp[:, 0]) > 0)                        # tile-columns ascending, distinct
            want_cols = set()
            for j in range(4):
                br = g * 4 + j
                k = row_ptr[br + 1] - row_ptr[br] if br < Mb else 0
                cols = tile_col[col_ptr[br]:col_ptr[br] + k] if br < Mb else []
                want_cols |= set(int(c) for c in cols)
                col_of_tile = {int(row_ptr[br] + t): int(cols[t]) for t in range(k)}
                for st in grp:
                    if st[1 + j] >= 0:
                        assert col_of_tile[int(st[1 + j])] == st[0]
                        seen[st[1 + j]] += 1
            assert set(int(c) for c in grp[:, 0]) == want_cols
            assert np.array_equal(grp[:, 5], (grp[:, 1:5] >= 0).sum(axis=1))
            # parts balanced by bytes: no part exceeds its share by more than one step's worth
            cost = 2 + grp[:, 5]
            if len(grp):
                share = cost.sum() / 4
                for r in range(4):
                    assert cost[parts[g, r] - parts[g, 0]:parts[g, r + 1] - parts[g, 0]].sum() <= share + 6
        assert nxt == len(steps)
        assert np.all(seen == 1)
        # step-ordered tile images: the tiles of a step lie next to each other, block-rows ascending,
        # and the steps follow each other without a gap
        tile_pos = pk.get("tile_pos")
        assert sorted(tile_pos.tolist()) == list(range(pk.T))
        nxt = 0
        for st in steps:
            assert st[6] == nxt
            for j in range(4):
                if st[1 + j] >= 0:
                    assert tile_pos[st[1 + j]] == nxt
                    nxt += 1
        assert nxt == pk.T
        pk.close()


# ------------------------------------------------ irregular block structure (Section 4.1.5)
def _numpy_tiles(Mp, Np, B, blocks, values):
    """The tile form of a set of blocks by array slicing: dense W_piv, then the tiles any block touches."""
    Wp = np.zeros((Mp, Np), dtype=values.dtype)
    touched = np.zeros((Mp // B, Np // B), dtype=bool)
    off = 0
    for r0, c0, h, w in blocks:
        Wp[r0:r0 + h, c0:c0 + w] = values[off:off + h * w].reshape(h, w)
        touched[r0 // B:(r0 + h - 1) // B + 1, c0 // B:(c0 + w - 1) // B + 1] = True
        off += h * w
    tl = np.argwhere(touched).astype(np.int32)
    tv = np.stack([Wp[br * B:(br + 1) * B, bc * B:(bc + 1) * B] for br, bc in tl]) if len(tl) else \
        np.zeros((0, B, B), dtype=values.dtype)
    return tl, tv


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("B,aligned", [(16, False), (32, False), (64, True), (16, True)])
def test_blocks_to_tiles_bit_exact(dtype, B, aligned):
    wl = synth.irregular_blocks(300 + B, 5 * B - 5, 7 * B - 9, B, wdtype=dtype, n_row_cuts=4, n_col_cuts=5,
                                keep=0.5, aligned=aligned)
    lay = wl.layers[0]
    tl, tv = pb.pp_blocks_to_tiles(lay.M, lay.N, B, lay.blocks, lay.block_values)
    tl_ref, tv_ref = _numpy_tiles(lay.row_perm.size, lay.col_perm.size, B, lay.blocks, lay.block_values)
    assert np.array_equal(tl, tl_ref)
    assert tv.tobytes() == tv_ref.tobytes()
    if aligned:      # blocks on the grid cost exactly their own bytes
        assert tv.size == lay.block_values.size


def test_blocks_pack_equals_tile_pack():
    """pp_pack_create_blocks is pp_blocks_to_tiles followed by pp_pack_create."""
    wl = synth.irregular_blocks(41, 200, 330, 32, wdtype="f16", n_row_cuts=3, n_col_cuts=6, keep=0.6, bias_std=0.1)
    lay = wl.layers[0]
    tl, tv = pb.pp_blocks_to_tiles(lay.M, lay.N, lay.B, lay.blocks, lay.block_values)
    a = pb.Packed.from_blocks(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values, lay.bias)
    b = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, tl, tv, lay.bias)
    for which in ("row_ptr", "tile_col", "values", "bias_piv", "gather_idx", "scatter_idx"):
        assert np.array_equal(a.get(which), b.get(which)), which
    # and the tile form reconstructs the same W as the block form (oracle on both)
    W_t = po.reconstruct(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, tl, tv)
    W_b = po.reconstruct_blocks(lay.M, lay.N, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values)
    assert np.array_equal(W_t, W_b)


def test_blocks_error_codes():
    rp = np.arange(64, dtype=np.int32)
    v = np.zeros(64 * 64, dtype=np.float32)
    def status(blocks, vals):
        try:
            pb.Packed.from_blocks(64, 64, 16, rp, rp, np.array(blocks, dtype=np.int32), vals)
        except pb.PPError as e:
            return e.status
        return 0
    assert status([[0, 0, 16, 16]], v[:256]) == 0
    assert status([[0, 0, 16, 16], [15, 15, 2, 2]], v[:260]) == 3      # overlap in one element
    assert status([[0, 0, 16, 16], [16, 16, 2, 2]], v[:260]) == 0                       # touching corners is fine
    assert status([[60, 0, 8, 4]], v[:32]) == 3                         # leaves the padded matrix
    assert status([[0, 0, 0, 4]], v[:0]) == 3                           # empty block
    assert status([[-1, 0, 2, 2]], v[:4]) == 3


@pytest.mark.parametrize("n_ctas", [1, 7, 148, 500])
@pytest.mark.parametrize("density,empty_rows", [(1.0, ()), (0.4, ()), (0.1, (0, 1, 2, 3, 9)), (0.02, ())])
def test_persistent_tile_plan_covers_every_step_once(n_ctas, density, empty_rows):
    """Plan of the persistent tensor-core kernel: every step of every group falls into exactly one unit, a group
    without tiles still has a (step-less) unit, a group's units are numbered in order and know their count and
    first index, a CTA's units are consecutive, and the CTAs' shares of the cost differ by at most one step."""
    rng = np.random.default_rng(17)
    M, N, B = 13 * 64 - 5, 11 * 64, 64
    Mb, Nb = -(-M // B), N // B
    grid = [(br, bc) for br in range(Mb) for bc in range(Nb) if br not in empty_rows]
    sel = rng.permutation(len(grid))[:max(1, int(density * len(grid)))]
    tl = np.array([grid[i] for i in sel], dtype=np.int32)
    tv = rng.standard_normal((tl.shape[0], B, B)).astype(np.float16)
    pk = pb.Packed(M, N, B, rng.permutation(Mb * B).astype(np.int32), rng.permutation(N).astype(np.int32), tl, tv)
    steps, parts = pk.get("tile_steps"), pk.get("tile_parts")
    units, cta_unit = pk.tile_units(n_ctas)
    groups = -(-Mb // 4)
    assert cta_unit[0] == 0 and cta_unit[-1] == len(units) and np.all(np.diff(cta_unit) >= 0)
    covered = np.zeros(len(steps), dtype=np.int32)
    seen_groups = []
    for u, (s0, s1, g, part, n_parts, first, _, _) in enumerate(units):
        assert parts[g, 0] <= s0 <= s1 <= parts[g, 4]
        covered[s0:s1] += 1
        assert first <= u < first + n_parts and part == u - first and units[first, 2] == g
        assert (s0 == s1) == (parts[g, 0] == parts[g, 4])           # step-less units only for groups without tiles
        seen_groups.append(g)
    assert np.all(covered == 1)
    assert sorted(set(seen_groups)) == list(range(groups)) and seen_groups == sorted(seen_groups)
    # a CTA's steps are contiguous, and the shares are balanced to within one step's cost
    cost = 2 + steps[:, 5] if len(steps) else np.zeros(0)
    share = []
    for c in range(n_ctas):
        mine = units[cta_unit[c]:cta_unit[c + 1]]
        if len(mine):
            assert np.all(mine[1:, 0] == mine[:-1, 1])
        share.append(sum(int(cost[s0:s1].sum()) for s0, s1 in mine[:, :2]))
    assert sum(share) == int(cost.sum())
    if len(steps):
        assert max(share) - min(share) <= 2 * int(cost.max())


# ------------------------------------------------ physical layouts of the layout study (Section 4.1.1)
@pytest.mark.parametrize("size,nb", [(64, 4), (96, 8), (40, 5)])
def test_layout_study_layouts(size, nb):
    """BRC = block,row,column; BCR = block,column,row; CBR = column,block,row (rightmost axis fastest)."""
    E = size // nb
    v = np.arange(nb * E * E, dtype=np.float32).reshape(nb, E, E)
    assert np.array_equal(pb.pp_layout_pack(size, nb, pb.PP_LAYOUT_BRC, v), v.reshape(-1))
    assert np.array_equal(pb.pp_layout_pack(size, nb, pb.PP_LAYOUT_BCR, v), v.transpose(0, 2, 1).reshape(-1))
    assert np.array_equal(pb.pp_layout_pack(size, nb, pb.PP_LAYOUT_CBR, v), v.transpose(2, 0, 1).reshape(-1))


def test_tuning_keys_reject_values_out_of_range():
    """pp_set_tuning is host code: every key takes its documented values and refuses the others (no GPU needed)."""
    from paper_1712_01084_b200 import binding as pb
    good = {5: (0, 1), 6: (4, 6, 8, 0), 7: (0, 1, 2), 8: (0, 1), 12: (2, 3, 1), 13: (0, 1), 15: (7, 0), 16: (0, 1), 17: (1, 0)}
    bad = {5: 2, 6: 5, 7: 3, 8: -1, 12: 4, 13: 2, 15: -1, 16: 2, 17: 2, 99: 0}
    for key, values in good.items():
        for v in values:                 # the last value of each tuple is the default, which stays set
            pb.pp_set_tuning(key, v)
    for key, v in bad.items():
        with pytest.raises(pb.PPError):
            pb.pp_set_tuning(key, v)
