"""pp_forward_noalloc: the forward call for hosts that may not allocate device memory on the
inference path (fixed arenas, foreign memory pools, no-synchronisation contexts).  The caller
uploads the packed layer image itself; the kernel's reduction scratch is a fixed array inside the
library.  Checked against pp_forward on the same inputs and against the fp64 oracle, twice in a
row, because every call shares (and must re-initialise) that array.  Collected last on purpose."""
import numpy as np
import pytest

from oracle import pp_oracle as po
from paper_1712_01084_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.mark.parametrize("case", ["f16_pairs", "f16_many", "f32_ragged"])
def test_noalloc_matches_pp_forward_twice(case):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_1712_01084_b200 import binding as pb
    pb.lib()
    # the partitions are forced so that strips of rows are shared between CTAs and the fixed
    # scratch array is really used: by two CTAs each (exchange slots) or by several (counters)
    tuning = {"f16_pairs": (300, 1, 0), "f16_many": (310, 1, 0), "f32_ragged": (40, 1, 0)}[case]
    if case == "f16_pairs":
        wl = synth.config5(k=64, batch=1, scale=0.5)          # 4096 x 4096
        rtol, atol = 2e-3, 1e-4
    elif case == "f16_many":
        wl = synth.config5(k=64, batch=4, scale=0.25)         # 2048 x 2048, strips cut in 3+ parts
        rtol, atol = 2e-3, 1e-4
    else:
        wl = synth.config1(batch=3, scale=0.5)
        rtol, atol = 1e-5, 1e-6
    lay = wl.layers[0]
    pb.pp_set_tuning(2, tuning[0]); pb.pp_set_tuning(3, tuning[1]); pb.pp_set_tuning(4, tuning[2])
    try:
        packed = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)
        layer = pb.Layer.from_synth(lay)
    finally:
        pb.pp_set_tuning(2, 296); pb.pp_set_tuning(3, 128); pb.pp_set_tuning(4, -1)
    shared = packed.get("strip_info")[:, 1]
    assert shared.max() >= (3 if case == "f16_many" else 2), "the plan must share strips for this test to mean anything"
    image = torch.from_numpy(packed.device_image()).cuda()        # the caller's own device memory
    x = torch.from_numpy(wl.x).cuda()
    ref = pb.pp_forward(layer, x, lay.act)
    y_ref, _, a = po.layer_forward(lay, wl.x.astype(np.float64), threads=8)
    out = torch.empty_like(ref)
    for call in range(2):
        out.fill_(float("nan"))
        pb.pp_forward_noalloc(packed, image, x, lay.act, out=out)
        torch.cuda.synchronize()
        assert pb.pp_noalloc_status() == 0, f"call {call}: the kernel's bounded wait gave up"
        got = out.cpu().numpy().astype(np.float64)
        err = np.abs(got - ref.cpu().numpy().astype(np.float64))       # against the allocating entry point
        assert np.all(err <= rtol * a + atol), f"call {call}: max err vs pp_forward {err.max()}"
        err = np.abs(got - y_ref)                                      # and against the CPU oracle
        assert np.all(err <= rtol * a + atol), f"call {call}: max err vs oracle {err.max()}"
    # a different layer through the same fixed scratch array, then the first one again
    wl2 = synth.config5(k=16, batch=2, scale=0.25)
    other = wl2.layers[0]
    packed2 = pb.Packed(other.M, other.N, other.B, other.row_perm, other.col_perm, other.tile_list, other.tile_values)
    image2 = torch.from_numpy(packed2.device_image()).cuda()
    x2 = torch.from_numpy(wl2.x).cuda()
    layer2 = pb.Layer.from_synth(other)
    ref2 = pb.pp_forward(layer2, x2, 0)
    out2 = torch.empty_like(ref2)
    pb.pp_forward_noalloc(packed2, image2, x2, 0, out=out2)
    assert torch.equal(out2, ref2)
    pb.pp_forward_noalloc(packed, image, x, lay.act, out=out)
    assert torch.equal(out, ref)
    # sizes beyond the fixed limits are refused, not attempted
    big = torch.zeros((9, lay.N), dtype=x.dtype, device="cuda")
    with pytest.raises(pb.PPError) as e:
        pb.pp_forward_noalloc(packed, image, big, 0, out=torch.empty((9, lay.M), device="cuda"))
    assert e.value.status == 6
    layer.close(); layer2.close()
