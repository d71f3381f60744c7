"""Python binding of libpp_b200.so: argument marshalling only.

Function names mirror the C interface (``include/pp.h``).  Device buffers are
PyTorch CUDA tensors; the binding passes their ``data_ptr()`` and the current
stream's handle.  Nothing here computes: if the compiled library is missing the
import fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpp_b200.so")

PP_OK = 0
PP_F32, PP_F16 = 0, 1
PP_ACT_IDENTITY, PP_ACT_RELU = 0, 1

STATUS_NAMES = {0: "PP_OK", 1: "PP_ERR_INVALID_ARG", 2: "PP_ERR_BAD_PERM", 3: "PP_ERR_BAD_TILE",
                4: "PP_ERR_ALLOC", 5: "PP_ERR_CUDA", 6: "PP_ERR_UNSUPPORTED", 7: "PP_ERR_TIMEOUT"}


class PPError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().pp_status_string(status).decode() if _lib is not None else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the C library (once).  No fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with "
                          f"`python -m paper_1712_01084_b200.build` (needs nvcc, targets sm_100a)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32p, i64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)
    ci, c64 = ctypes.c_int, ctypes.c_int64
    fp = ctypes.POINTER(ctypes.c_float)
    create_args = [ctypes.POINTER(vp), ci, ci, ci, i32p, i32p, i32p, c64, vp, ci, fp]
    sig = {
        "pp_status_string": (ctypes.c_char_p, [ci]),
        "pp_pack_create": (ci, create_args),
        "pp_pack_destroy": (ci, [vp]),
        "pp_blocks_to_tiles": (ci, [ci, ci, ci, i32p, c64, vp, ci, i64p, i32p, vp, c64]),
        "pp_pack_create_blocks": (ci, create_args),
        "pp_layer_create_blocks": (ci, create_args),
        "pp_pack_info": (ci, [vp, i64p]),
        "pp_pack_get": (ci, [vp, ci, vp, c64]),
        "pp_pack_unpack": (ci, [vp, i32p, vp]),
        "pp_pack_tile_units": (ci, [vp, ci, i32p, c64, i64p, i32p]),
        "pp_fold_perm": (ci, [i32p, ci, ci, i32p, ci, ci, i32p]),
        "pp_layer_create": (ci, create_args),
        "pp_layer_destroy": (ci, [vp]),
        "pp_layer_clone": (ci, [ctypes.POINTER(vp), vp]),
        "pp_layer_status": (ci, [vp, ctypes.POINTER(ci)]),
        "pp_layer_launch_info": (ci, [vp, ci, i32p]),
        "pp_forward": (ci, [vp, vp, vp, ci, ci, vp]),
        "pp_forward_host": (ci, [vp, vp, vp, ci, ci, vp]),
        "pp_chain_create": (ci, [ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(ci), ci, ci]),
        "pp_chain_destroy": (ci, [vp]),
        "pp_chain_forward": (ci, [vp, vp, vp, ci, vp]),
        "pp_chain_status": (ci, [vp, ctypes.POINTER(ci)]),
        "pp_chain_set_output_pivoted": (ci, [vp, ci]),
        "pp_chain_output_map": (ci, [vp, i32p]),
        "pp_chain_link_info": (ci, [vp, i32p]),
        "pp_forward_pivoted": (ci, [vp, vp, vp, ci, ci, vp]),
        "pp_layer_output_map": (ci, [vp, i32p]),
        "pp_set_tuning": (ci, [ci, ci]),
        "pp_lstm_create": (ci, [ctypes.POINTER(vp), vp, ci, ci, ci]),
        "pp_lstm_destroy": (ci, [vp]),
        "pp_lstm_forward": (ci, [vp, vp, vp, vp, ci, vp]),
        "pp_lstm_status": (ci, [vp, ctypes.POINTER(ci)]),
        "pp_pivot_find": (ci, [ci, ci, fp, ci, ci, i32p, i32p, i32p, i32p, i32p, ctypes.POINTER(ctypes.c_double)]),
        "pp_layout_pack": (ci, [ci, ci, ci, fp, fp]),
        "pp_layout_create": (ci, [ctypes.POINTER(vp), ci, ci, ci, ci, i32p, i32p, fp]),
        "pp_layout_destroy": (ci, [vp]),
        "pp_layout_forward": (ci, [vp, vp, vp, vp]),
        "pp_pack_device_image_bytes": (ci, [vp, i64p]),
        "pp_pack_device_image": (ci, [vp, vp, c64]),
        "pp_forward_noalloc": (ci, [vp, vp, vp, vp, ci, ci, vp]),
        "pp_noalloc_status": (ci, [ctypes.POINTER(ci)]),
        "pp_selftest_host": (ci, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _lib = L
    return L


def _check(st: int, where: str):
    if st != PP_OK:
        raise PPError(st, where)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _layer_args(M, N, B, row_perm, col_perm, tile_list, tile_values, bias):
    rp, rpp = _i32(row_perm)
    cp, cpp = _i32(col_perm)
    tl, tlp = _i32(np.asarray(tile_list).reshape(-1, 2))
    tv = np.ascontiguousarray(tile_values)
    if tv.dtype == np.float16:
        wd = PP_F16
    elif tv.dtype == np.float32:
        wd = PP_F32
    else:
        raise TypeError("tile_values must be float32 or float16")
    T = tl.shape[0]
    if tv.size != T * B * B:
        raise ValueError("tile_values must hold T*B*B elements")
    if rp.size != -(-M // B) * B or cp.size != -(-N // B) * B:
        raise ValueError("row_perm/col_perm must cover the padded ranges")
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    if b is not None and b.size != M:
        raise ValueError("bias must have M entries")
    bp = None if b is None else b.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    keep = (rp, cp, tl, tv, b)
    return keep, (int(M), int(N), int(B), rpp, cpp, tlp, T, tv.ctypes.data_as(ctypes.c_void_p), wd, bp)


def _block_args(M, N, B, row_perm, col_perm, blocks, block_values, bias):
    rp, rpp = _i32(row_perm)
    cp, cpp = _i32(col_perm)
    bl, blp = _i32(np.asarray(blocks).reshape(-1, 4))
    bv = np.ascontiguousarray(block_values).reshape(-1)
    if bv.dtype == np.float16:
        wd = PP_F16
    elif bv.dtype == np.float32:
        wd = PP_F32
    else:
        raise TypeError("block_values must be float32 or float16")
    if bv.size != int(np.sum(bl[:, 2].astype(np.int64) * bl[:, 3])):
        raise ValueError("block_values must hold sum(height*width) elements")
    if rp.size != -(-M // B) * B or cp.size != -(-N // B) * B:
        raise ValueError("row_perm/col_perm must cover the padded ranges")
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    if b is not None and b.size != M:
        raise ValueError("bias must have M entries")
    bp = None if b is None else b.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    keep = (rp, cp, bl, bv, b)
    return keep, (int(M), int(N), int(B), rpp, cpp, blp, bl.shape[0], bv.ctypes.data_as(ctypes.c_void_p), wd, bp)


def pp_blocks_to_tiles(M, N, B, blocks, block_values):
    """Lay irregular blocks over the B x B tile grid (pp_blocks_to_tiles): (tile_list [T,2], tile_values [T,B,B])."""
    bl, blp = _i32(np.asarray(blocks).reshape(-1, 4))
    bv = np.ascontiguousarray(block_values).reshape(-1)
    wd = PP_F16 if bv.dtype == np.float16 else PP_F32
    if bv.dtype not in (np.float16, np.float32):
        raise TypeError("block_values must be float32 or float16")
    if bv.size != int(np.sum(bl[:, 2].astype(np.int64) * bl[:, 3])):
        raise ValueError("block_values must hold sum(height*width) elements")
    T = ctypes.c_int64(0)
    bvp = bv.ctypes.data_as(ctypes.c_void_p)
    _check(lib().pp_blocks_to_tiles(int(M), int(N), int(B), blp, bl.shape[0], bvp, wd, ctypes.byref(T), None, None, 0),
           "pp_blocks_to_tiles")
    tl = np.zeros((T.value, 2), dtype=np.int32)
    tv = np.zeros((T.value, B, B), dtype=bv.dtype)
    _check(lib().pp_blocks_to_tiles(int(M), int(N), int(B), blp, bl.shape[0], bvp, wd, ctypes.byref(T),
                                    tl.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), tv.ctypes.data_as(ctypes.c_void_p),
                                    T.value), "pp_blocks_to_tiles")
    return tl, tv


# ---------------------------------------------------------------- host packer
class Packed:
    """Host-side packed layer (pp_pack_create); needs no GPU."""

    def __init__(self, M, N, B, row_perm, col_perm, tile_list, tile_values, bias=None):
        keep, args = _layer_args(M, N, B, row_perm, col_perm, tile_list, tile_values, bias)
        self._h = ctypes.c_void_p()
        _check(lib().pp_pack_create(ctypes.byref(self._h), *args), "pp_pack_create")
        self._finish(M, N, B, np.asarray(tile_values).dtype)

    @classmethod
    def from_blocks(cls, M, N, B, row_perm, col_perm, blocks, block_values, bias=None) -> "Packed":
        """Packed layer from irregular blocks (pp_pack_create_blocks)."""
        keep, args = _block_args(M, N, B, row_perm, col_perm, blocks, block_values, bias)
        self = object.__new__(cls)
        self._h = ctypes.c_void_p()
        _check(lib().pp_pack_create_blocks(ctypes.byref(self._h), *args), "pp_pack_create_blocks")
        self._finish(M, N, B, np.asarray(block_values).dtype)
        return self

    def _finish(self, M, N, B, wdtype):
        self.M, self.N, self.B = int(M), int(N), int(B)
        self.wdtype = wdtype
        info = (ctypes.c_int64 * 13)()
        _check(lib().pp_pack_info(self._h, info), "pp_pack_info")
        (self.Mb, self.Nb, self.T, self.n_tile_col, self.n_items, self.value_bytes,
         self.max_item_tiles, self.n_slots, self.n_strips, self.n_frags, self.stream_grid,
         self.stream_slots, self.n_tile_steps) = [int(v) for v in info]

    def get(self, which: str) -> np.ndarray:
        Mpad, Npad = self.Mb * self.B, self.Nb * self.B
        spec = {"row_ptr": (0, np.int32, self.Mb + 1), "col_ptr": (1, np.int32, self.Mb + 1),
                "tile_col": (2, np.int32, self.n_tile_col), "gather_idx": (3, np.int32, Npad),
                "scatter_idx": (4, np.int32, Mpad), "bias_piv": (5, np.float32, Mpad),
                "values": (6, np.uint8, self.value_bytes), "items": (7, np.int32, self.n_items * 8),
                "inv_row_perm": (8, np.int32, Mpad), "strip_start": (9, np.int32, self.n_strips + 1),
                "xoff": (10, np.int32, self.n_frags), "cta_desc": (11, np.int32, self.stream_grid * 4),
                "strip_info": (12, np.int32, self.n_strips * 4),
                "tile_steps": (13, np.int32, self.n_tile_steps * 8),
                "tile_pos": (15, np.int32, self.T if self.n_tile_steps else 0),
                "tile_parts": (14, np.int32, (-(-self.Mb // 4)) * 5 if self.n_tile_steps or
                               (self.B == 64 and self.wdtype == np.float16) else 0)}[which]
        out = np.empty(spec[2], dtype=spec[1])
        _check(lib().pp_pack_get(self._h, spec[0], out.ctypes.data_as(ctypes.c_void_p), out.nbytes), "pp_pack_get")
        if which in ("items", "tile_steps"):
            return out.reshape(-1, 8)
        if which == "tile_parts":
            return out.reshape(-1, 5)
        return out.reshape(-1, 4) if which in ("cta_desc", "strip_info") else out

    def tile_units(self, n_ctas: int):
        """Plan of the persistent tensor-core kernel for n_ctas CTAs (pp_pack_tile_units): (units [n, 8], cta_unit [n_ctas + 1])."""
        n = ctypes.c_int64(0)
        _check(lib().pp_pack_tile_units(self._h, int(n_ctas), None, 0, ctypes.byref(n), None), "pp_pack_tile_units")
        units = np.zeros((n.value, 8), dtype=np.int32)
        cta_unit = np.zeros(int(n_ctas) + 1, dtype=np.int32)
        i32p = ctypes.POINTER(ctypes.c_int32)
        _check(lib().pp_pack_tile_units(self._h, int(n_ctas), units.ctypes.data_as(i32p), n.value, ctypes.byref(n),
                                        cta_unit.ctypes.data_as(i32p)), "pp_pack_tile_units")
        return units, cta_unit

    def unpack(self):
        tl = np.empty((self.T, 2), dtype=np.int32)
        tv = np.empty((self.T, self.B, self.B), dtype=self.wdtype)
        _check(lib().pp_pack_unpack(self._h, tl.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                    tv.ctypes.data_as(ctypes.c_void_p)), "pp_pack_unpack")
        return tl, tv

    def device_image(self) -> np.ndarray:
        """Host copy of the layer image that pp_forward_noalloc reads from device memory."""
        n = ctypes.c_int64()
        _check(lib().pp_pack_device_image_bytes(self._h, ctypes.byref(n)), "pp_pack_device_image_bytes")
        img = np.empty(n.value, dtype=np.uint8)
        _check(lib().pp_pack_device_image(self._h, img.ctypes.data_as(ctypes.c_void_p), n.value),
               "pp_pack_device_image")
        return img

    def close(self):
        if self._h:
            lib().pp_pack_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pp_fold_perm(row_perm_A, M_A: int, col_perm_B, N_B: int) -> np.ndarray:
    ra, rap = _i32(row_perm_A)
    cb, cbp = _i32(col_perm_B)
    q = np.empty(cb.size, dtype=np.int32)
    _check(lib().pp_fold_perm(rap, int(M_A), ra.size, cbp, int(N_B), cb.size,
                              q.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))), "pp_fold_perm")
    return q


def pp_set_tuning(key: int, value: int):
    _check(lib().pp_set_tuning(int(key), int(value)), "pp_set_tuning")


# ------------------------------------------------------------------ device API
def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _require_cuda(t, name):
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")


class Layer:
    """Device-resident pivoted FC layer (pp_layer_create / pp_forward)."""

    def __init__(self, M, N, B, row_perm, col_perm, tile_list, tile_values, bias=None):
        keep, args = _layer_args(M, N, B, row_perm, col_perm, tile_list, tile_values, bias)
        self._h = ctypes.c_void_p()
        _check(lib().pp_layer_create(ctypes.byref(self._h), *args), "pp_layer_create")
        self.M, self.N, self.B = int(M), int(N), int(B)
        self.wdtype = np.asarray(tile_values).dtype

    @classmethod
    def from_synth(cls, lay):
        if hasattr(lay, "blocks"):
            return cls.from_blocks(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.blocks, lay.block_values, lay.bias)
        return cls(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)

    @classmethod
    def from_blocks(cls, M, N, B, row_perm, col_perm, blocks, block_values, bias=None) -> "Layer":
        """Layer whose W_piv holds rectangles of any size and position (pp_layer_create_blocks)."""
        keep, args = _block_args(M, N, B, row_perm, col_perm, blocks, block_values, bias)
        self = object.__new__(cls)
        self._h = ctypes.c_void_p()
        _check(lib().pp_layer_create_blocks(ctypes.byref(self._h), *args), "pp_layer_create_blocks")
        self.M, self.N, self.B = int(M), int(N), int(B)
        self.wdtype = np.asarray(block_values).dtype
        return self

    def clone(self) -> "Layer":
        other = object.__new__(Layer)
        other._h = ctypes.c_void_p()
        _check(lib().pp_layer_clone(ctypes.byref(other._h), self._h), "pp_layer_clone")
        other.M, other.N, other.B, other.wdtype = self.M, self.N, self.B, self.wdtype
        return other

    def forward(self, x, act: int = PP_ACT_IDENTITY, out=None, stream=None):
        return pp_forward(self, x, act, out=out, stream=stream)

    def output_map(self) -> np.ndarray:
        """Original output row of every pivoted position, -1 for padding (pp_layer_output_map)."""
        m = np.empty(-(-self.M // self.B) * self.B, dtype=np.int32)
        _check(lib().pp_layer_output_map(self._h, m.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))), "pp_layer_output_map")
        return m

    def launch_info(self, batch: int = 1) -> dict:
        """Kernel and launch shape a forward call with this batch uses (pp_layer_launch_info)."""
        o = np.zeros(6, dtype=np.int32)
        _check(lib().pp_layer_launch_info(self._h, int(batch), o.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))),
               "pp_layer_launch_info")
        names = {0: "gemv", 1: "stream", 2: "tile", 3: "tile_cluster", 4: "tile_persist"}
        return {"kernel": names[int(o[0])], "ctas": int(o[1]), "ring_depth": int(o[2]), "smem_bytes": int(o[3]),
                "stage_mode": int(o[4]), "pdl": int(o[5])}

    def status(self) -> int:
        """PP_OK, or PP_ERR_TIMEOUT when a kernel's bounded wait gave up (synchronises; clears the flag)."""
        st = ctypes.c_int(0)
        _check(lib().pp_layer_status(self._h, ctypes.byref(st)), "pp_layer_status")
        return st.value

    def close(self):
        if self._h:
            lib().pp_layer_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pp_layer_create(M, N, B, row_perm, col_perm, tile_list, tile_values, bias=None) -> Layer:
    return Layer(M, N, B, row_perm, col_perm, tile_list, tile_values, bias)


def pp_layer_create_blocks(M, N, B, row_perm, col_perm, blocks, block_values, bias=None) -> Layer:
    return Layer.from_blocks(M, N, B, row_perm, col_perm, blocks, block_values, bias)


def _check_x(x, N, wdtype):
    import torch
    _require_cuda(x, "x")
    want = torch.float16 if wdtype == np.float16 else torch.float32
    if x.dtype != want:
        raise TypeError(f"x must be {want}")
    if x.dim() == 1:
        x = x.unsqueeze(0)
    if x.shape[-1] != N:
        raise ValueError(f"x must be [batch][{N}]")
    return x


def pp_forward(layer: Layer, x, act: int = PP_ACT_IDENTITY, out=None, stream=None):
    """y[batch][M] (float32, CUDA) = act(W x + b).  Enqueues on the current stream."""
    import torch
    x2 = _check_x(x, layer.N, layer.wdtype)
    batch = x2.shape[0]
    y = torch.empty((batch, layer.M), dtype=torch.float32, device=x.device) if out is None else out
    _require_cuda(y, "out")
    if y.dtype != torch.float32 or y.numel() != batch * layer.M:
        raise ValueError("out must be float32 [batch][M]")
    _check(lib().pp_forward(layer._h, ctypes.c_void_p(x2.data_ptr()), ctypes.c_void_p(y.data_ptr()),
                            batch, int(act), _stream_ptr(stream)), "pp_forward")
    return y


def pp_forward_host(layer: Layer, x_host, act: int = PP_ACT_IDENTITY, out=None, stream=None):
    """y = act(W x + b) from host tensors (pp_forward_host): x_host and the returned y are CPU tensors
    (pinned memory keeps the copies asynchronous); the call returns once y is valid."""
    import torch
    if x_host.is_cuda or not x_host.is_contiguous():
        raise ValueError("x_host must be a contiguous CPU tensor")
    want = torch.float16 if layer.wdtype == np.float16 else torch.float32
    if x_host.dtype != want or x_host.shape[-1] != layer.N:
        raise ValueError("x_host must have the layer's element type and N columns")
    batch = x_host.numel() // layer.N
    y = torch.empty((batch, layer.M), dtype=torch.float32) if out is None else out
    if y.is_cuda or y.dtype != torch.float32 or y.numel() != batch * layer.M or not y.is_contiguous():
        raise ValueError("out must be a contiguous float32 CPU tensor [batch][M]")
    _check(lib().pp_forward_host(layer._h, x_host.data_ptr(), y.data_ptr(), batch, int(act), _stream_ptr(stream)),
           "pp_forward_host")
    return y


def pp_forward_pivoted(layer: Layer, x, act: int = PP_ACT_IDENTITY, out=None, stream=None):
    """y_piv[batch][M_pad] (float32, CUDA): act(W x + b) left in the layer's pivoted row order
    (pp_forward_pivoted); layer.output_map() relabels the positions."""
    import torch
    x2 = _check_x(x, layer.N, layer.wdtype)
    batch = x2.shape[0]
    m_pad = -(-layer.M // layer.B) * layer.B
    y = torch.empty((batch, m_pad), dtype=torch.float32, device=x.device) if out is None else out
    _require_cuda(y, "out")
    if y.dtype != torch.float32 or y.numel() != batch * m_pad:
        raise ValueError("out must be float32 [batch][M_pad]")
    _check(lib().pp_forward_pivoted(layer._h, ctypes.c_void_p(x2.data_ptr()), ctypes.c_void_p(y.data_ptr()),
                                    batch, int(act), _stream_ptr(stream)), "pp_forward_pivoted")
    return y


def pp_forward_noalloc(packed: Packed, device_image, x, act: int = PP_ACT_IDENTITY, out=None, stream=None):
    """pp_forward for callers that may not allocate: `device_image` is a CUDA uint8 tensor holding
    packed.device_image(); `out` must be given (this function creates no tensor)."""
    import torch
    x2 = _check_x(x, packed.N, packed.wdtype)
    batch = x2.shape[0]
    if out is None:
        raise ValueError("out must be provided: this entry point allocates nothing")
    _require_cuda(out, "out")
    _require_cuda(device_image, "device_image")
    if out.dtype != torch.float32 or out.numel() != batch * packed.M:
        raise ValueError("out must be float32 [batch][M]")
    _check(lib().pp_forward_noalloc(packed._h, ctypes.c_void_p(device_image.data_ptr()),
                                    ctypes.c_void_p(x2.data_ptr()), ctypes.c_void_p(out.data_ptr()),
                                    batch, int(act), _stream_ptr(stream)), "pp_forward_noalloc")
    return out


def pp_noalloc_status() -> int:
    """Time-out flag of the current device's pp_forward_noalloc kernels (PP_OK or PP_ERR_TIMEOUT); cleared by the read."""
    st = ctypes.c_int(0)
    _check(lib().pp_noalloc_status(ctypes.byref(st)), "pp_noalloc_status")
    return st.value


class Chain:
    """Stack of layers with folded permutations (pp_chain_create / pp_chain_forward)."""

    def __init__(self, layers: Sequence[Layer], acts: Sequence[int], max_batch: int = 8):
        self.layers = list(layers)          # keep the layers alive
        n = len(self.layers)
        arr = (ctypes.c_void_p * n)(*[l._h for l in self.layers])
        acts_arr = (ctypes.c_int * n)(*[int(a) for a in acts])
        self._h = ctypes.c_void_p()
        _check(lib().pp_chain_create(ctypes.byref(self._h), arr, acts_arr, n, int(max_batch)), "pp_chain_create")
        self.max_batch = int(max_batch)
        self.output_pivoted = False

    def forward(self, x, out=None, stream=None):
        return pp_chain_forward(self, x, out=out, stream=stream)

    def set_output_pivoted(self, enable: bool = True):
        """Leave the result in the last layer's pivoted row order (pp_chain_set_output_pivoted)."""
        _check(lib().pp_chain_set_output_pivoted(self._h, 1 if enable else 0), "pp_chain_set_output_pivoted")
        self.output_pivoted = bool(enable)

    def output_map(self) -> np.ndarray:
        last = self.layers[-1]
        m = np.empty(-(-last.M // last.B) * last.B, dtype=np.int32)
        _check(lib().pp_chain_output_map(self._h, m.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))), "pp_chain_output_map")
        return m

    def status(self) -> int:
        """PP_OK, or PP_ERR_TIMEOUT when a bounded device-side wait gave up (synchronises; clears the flags)."""
        st = ctypes.c_int(0)
        _check(lib().pp_chain_status(self._h, ctypes.byref(st)), "pp_chain_status")
        return st.value

    def link_info(self) -> np.ndarray:
        """identity[l] = 1 when the link into layer l needs no index array (pp_chain_link_info)."""
        m = np.zeros(len(self.layers), dtype=np.int32)
        _check(lib().pp_chain_link_info(self._h, m.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))), "pp_chain_link_info")
        return m

    def close(self):
        if self._h:
            lib().pp_chain_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pp_chain_create(layers, acts, max_batch: int = 8) -> Chain:
    return Chain(layers, acts, max_batch)


def pp_chain_forward(chain: Chain, x, out=None, stream=None):
    import torch
    first, last = chain.layers[0], chain.layers[-1]
    x2 = _check_x(x, first.N, first.wdtype)
    batch = x2.shape[0]
    width = -(-last.M // last.B) * last.B if chain.output_pivoted else last.M
    y = torch.empty((batch, width), dtype=torch.float32, device=x.device) if out is None else out
    _require_cuda(y, "out")
    if y.dtype != torch.float32 or y.numel() != batch * width:
        raise ValueError("out must be float32 [batch][M] ([batch][M_pad] when the output stays pivoted)")
    _check(lib().pp_chain_forward(chain._h, ctypes.c_void_p(x2.data_ptr()), ctypes.c_void_p(y.data_ptr()),
                                  batch, _stream_ptr(stream)), "pp_chain_forward")
    return y


class Lstm:
    """LSTM cell around one pivoted gate layer (pp_lstm_create / pp_lstm_forward)."""

    def __init__(self, gates: Layer, I: int, H: int, max_steps: int):
        self.gates = gates                  # keep the layer alive
        self.I, self.H, self.max_steps = int(I), int(H), int(max_steps)
        self._h = ctypes.c_void_p()
        _check(lib().pp_lstm_create(ctypes.byref(self._h), gates._h, self.I, self.H, self.max_steps), "pp_lstm_create")

    def forward(self, x_seq, h, c, stream=None):
        return pp_lstm_forward(self, x_seq, h, c, stream=stream)

    def status(self) -> int:
        """0, or the code of a bounded device-side wait that gave up (synchronises; clears the flag)."""
        out = ctypes.c_int(0)
        _check(lib().pp_lstm_status(self._h, ctypes.byref(out)), "pp_lstm_status")
        return out.value

    def close(self):
        if self._h:
            lib().pp_lstm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pp_lstm_forward(lstm: Lstm, x_seq, h, c, stream=None):
    """Runs x_seq.shape[0] steps; h (layer dtype, [H]) and c (float32, [H]) are updated in place."""
    import torch
    for t, name in ((x_seq, "x_seq"), (h, "h"), (c, "c")):
        _require_cuda(t, name)
    want = torch.float16 if lstm.gates.wdtype == np.float16 else torch.float32
    if x_seq.dtype != want or h.dtype != want or c.dtype != torch.float32:
        raise TypeError("x_seq and h must have the layer's element type, c must be float32")
    if x_seq.dim() != 2 or x_seq.shape[1] != lstm.I or h.numel() != lstm.H or c.numel() != lstm.H:
        raise ValueError("x_seq must be [steps][I], h and c [H]")
    _check(lib().pp_lstm_forward(lstm._h, ctypes.c_void_p(x_seq.data_ptr()), ctypes.c_void_p(h.data_ptr()),
                                 ctypes.c_void_p(c.data_ptr()), int(x_seq.shape[0]), _stream_ptr(stream)),
           "pp_lstm_forward")
    return h, c


# ------------------------------------------------- layout study (Section 4.1.1)
PP_LAYOUT_BRC, PP_LAYOUT_BCR, PP_LAYOUT_CBR = 0, 1, 2
PP_MAP_ROWS_PER_LANE, PP_MAP_LANES_ALONG_K = 0, 1


def pp_layout_pack(size, n_blocks, layout, block_values) -> np.ndarray:
    bv = np.ascontiguousarray(block_values, dtype=np.float32).reshape(-1)
    out = np.empty_like(bv)
    fp = ctypes.POINTER(ctypes.c_float)
    _check(lib().pp_layout_pack(int(size), int(n_blocks), int(layout), bv.ctypes.data_as(fp), out.ctypes.data_as(fp)),
           "pp_layout_pack")
    return out


class LayoutStudy:
    """Plain fp32 kernel over one physical layout of the blocks and one thread mapping
    (pp_layout_create / pp_layout_forward): the yardstick of the layout study."""

    def __init__(self, size, n_blocks, layout, mapping, row_perm, col_perm, block_values):
        rp, rpp = _i32(row_perm)
        cp, cpp = _i32(col_perm)
        bv = np.ascontiguousarray(block_values, dtype=np.float32).reshape(-1)
        if size % n_blocks or bv.size != n_blocks * (size // n_blocks) ** 2 or rp.size != size or cp.size != size:
            raise ValueError("sizes do not describe n_blocks square blocks of edge size/n_blocks")
        self._h = ctypes.c_void_p()
        _check(lib().pp_layout_create(ctypes.byref(self._h), int(size), int(n_blocks), int(layout), int(mapping), rpp, cpp,
                                      bv.ctypes.data_as(ctypes.POINTER(ctypes.c_float))), "pp_layout_create")
        self.size = int(size)

    def forward(self, x, out=None, stream=None):
        import torch
        _require_cuda(x, "x")
        if x.dtype != torch.float32 or x.numel() != self.size:
            raise ValueError("x must be float32 with `size` elements")
        y = torch.empty(self.size, dtype=torch.float32, device=x.device) if out is None else out
        _check(lib().pp_layout_forward(self._h, x.data_ptr(), y.data_ptr(), _stream_ptr(stream)), "pp_layout_forward")
        return y

    def close(self):
        if self._h:
            lib().pp_layout_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ------------------------------------------------- feed-back search for index arrays (Section 3.2)
def pp_pivot_find(abs_w, levels: int, max_sweeps: int = 32, row_init=None, col_init=None):
    """(row_perm, col_perm, blocks [2^levels, 4], kept sum) for the absolute weights abs_w [M, N] (pp_pivot_find)."""
    A = np.ascontiguousarray(abs_w, dtype=np.float32)
    M, N = A.shape
    i32p = ctypes.POINTER(ctypes.c_int32)
    ri = None if row_init is None else np.ascontiguousarray(row_init, dtype=np.int32)
    ci_ = None if col_init is None else np.ascontiguousarray(col_init, dtype=np.int32)
    rp, cp = np.empty(M, dtype=np.int32), np.empty(N, dtype=np.int32)
    bl = np.empty((max(1, 2 ** min(int(levels), 20)), 4), dtype=np.int32)
    kept = ctypes.c_double(0.0)
    _check(lib().pp_pivot_find(M, N, A.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), int(levels), int(max_sweeps),
                               None if ri is None else ri.ctypes.data_as(i32p), None if ci_ is None else ci_.ctypes.data_as(i32p),
                               rp.ctypes.data_as(i32p), cp.ctypes.data_as(i32p), bl.ctypes.data_as(i32p), ctypes.byref(kept)),
           "pp_pivot_find")
    return rp, cp, bl, kept.value
