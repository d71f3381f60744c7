"""ctypes front end of the fp64 CPU oracle (``pp_oracle.c``).

TEST INFRASTRUCTURE ONLY.  It is used by the tests, the smoke check and the
CPU-baseline leg of the benchmark; the CUDA library never calls it and it
imports nothing from the CUDA package.

The single-layer functions are thin wrappers over the C file.  The chain and
the LSTM recurrence are plain loops over the dense single-layer product:

* chain (Section 4.2.1 describes the folded form; the oracle deliberately does
  NOT fold anything): layer by layer in original coordinates, each layer's
  activated output optionally rounded to the next layer's storage type.
* LSTM cell (not in the paper; the recurrent workload defines it): with
  z_t = [x_t ; h_{t-1}], g = W z_t and original rows [0,H) i, [H,2H) f,
  [2H,3H) g, [3H,4H) o:  c_t = sig(f) c_{t-1} + sig(i) tanh(g),
  h_t = sig(o) tanh(c_t), h_0 = c_0 = 0, no bias.  Parity unpinned by the
  paper: only the closed-form special cases in the tests pin it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pp_oracle.c")
_LIB = os.path.join(_HERE, "libpp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pp_oracle.c with gcc (plain C, -O2, OpenMP for the row loop)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        _lib.ppo_reconstruct.restype = ctypes.c_int
        _lib.ppo_reconstruct.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, i32p,
                                         ctypes.c_int64, f64p, f64p]
        _lib.ppo_reconstruct_blocks.restype = ctypes.c_int
        _lib.ppo_reconstruct_blocks.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p,
                                                i32p, ctypes.c_int64, f64p, f64p]
        _lib.ppo_dense_forward.restype = None
        _lib.ppo_dense_forward.argtypes = [ctypes.c_int, ctypes.c_int, f64p, f64p, f64p, ctypes.c_int,
                                           ctypes.c_int, f64p, f64p, f64p, ctypes.c_int]
        _lib.ppo_dense_forward_rows.restype = None
        _lib.ppo_dense_forward_rows.argtypes = [ctypes.c_int, ctypes.c_int, f64p, f64p, f64p, ctypes.c_int,
                                                ctypes.c_int, i32p, ctypes.c_int, f64p, f64p]
        _lib.ppo_structured_forward.restype = ctypes.c_int
        _lib.ppo_structured_forward.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, i32p,
                                                ctypes.c_int64, f64p, f64p, f64p, ctypes.c_int,
                                                ctypes.c_int, f64p]
    return _lib


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _f64(a):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


class OracleError(ValueError):
    pass


_ERR = {1: "bad permutation", 2: "bad tile (duplicate or out of range)", 3: "bad argument"}


def reconstruct(M, N, B, row_perm, col_perm, tile_list, tile_values) -> np.ndarray:
    """Dense W of Eq. 1 in fp64."""
    lib = _load()
    rp, rpp = _i32(row_perm)
    cp, cpp = _i32(col_perm)
    tl, tlp = _i32(np.asarray(tile_list).reshape(-1, 2))
    tv, tvp = _f64(np.asarray(tile_values, dtype=np.float64).reshape(-1))
    T = tl.shape[0]
    if tv.size != T * B * B:
        raise OracleError("tile_values has the wrong size")
    W = np.empty((M, N), dtype=np.float64)
    rc = lib.ppo_reconstruct(M, N, B, rpp, cpp, tlp, T, tvp, W.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc:
        raise OracleError(_ERR.get(rc, str(rc)))
    return W


def reconstruct_blocks(M, N, row_perm, col_perm, blocks, block_values) -> np.ndarray:
    """Dense W of Eq. 1 when M_block holds rectangles of any size (Section 4.1.5).
    blocks: [nb][4] = (first pivoted row, first pivoted column, height, width);
    block_values: the blocks' values one after the other, each row-major.
    The pivoted sizes are the lengths of the index arrays."""
    lib = _load()
    rp, rpp = _i32(row_perm)
    cp, cpp = _i32(col_perm)
    bl, blp = _i32(np.asarray(blocks).reshape(-1, 4))
    bv, bvp = _f64(np.asarray(block_values, dtype=np.float64).reshape(-1))
    if bv.size != int(np.sum(bl[:, 2].astype(np.int64) * bl[:, 3])):
        raise OracleError("block_values has the wrong size")
    W = np.empty((M, N), dtype=np.float64)
    rc = lib.ppo_reconstruct_blocks(M, N, rp.size, cp.size, rpp, cpp, blp, bl.shape[0], bvp,
                                    W.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc:
        raise OracleError(_ERR.get(rc, str(rc)))
    return W


def dense_forward(W, bias, x, act: int, threads: int = 1):
    """(y, s, a) = (act(Wx+b), Wx+b, |W||x|), each [batch][M], fp64."""
    lib = _load()
    W, Wp = _f64(W)
    M, N = W.shape
    x = np.asarray(x, dtype=np.float64).reshape(-1, N)
    x, xp = _f64(x)
    b, bp = _f64(bias)
    batch = x.shape[0]
    y = np.empty((batch, M)); s = np.empty((batch, M)); a = np.empty((batch, M))
    dp = lambda v: v.ctypes.data_as(ctypes.POINTER(ctypes.c_double))
    lib.ppo_dense_forward(M, N, Wp, bp, xp, batch, int(act), dp(y), dp(s), dp(a), int(threads))
    return y, s, a


def dense_forward_rows(W, bias, x, act: int, rows):
    """(y, a) on the listed original rows only, each [batch][len(rows)]."""
    lib = _load()
    W, Wp = _f64(W)
    M, N = W.shape
    x = np.asarray(x, dtype=np.float64).reshape(-1, N)
    x, xp = _f64(x)
    b, bp = _f64(bias)
    r, rp = _i32(rows)
    batch = x.shape[0]
    y = np.empty((batch, r.size)); a = np.empty((batch, r.size))
    dp = lambda v: v.ctypes.data_as(ctypes.POINTER(ctypes.c_double))
    lib.ppo_dense_forward_rows(M, N, Wp, bp, xp, batch, int(act), rp, r.size, dp(y), dp(a))
    return y, a


def structured_forward(M, N, B, row_perm, col_perm, tile_list, tile_values, bias, x, act: int):
    """Eq. 2 evaluated as gather -> block product -> scatter."""
    lib = _load()
    rp, rpp = _i32(row_perm)
    cp, cpp = _i32(col_perm)
    tl, tlp = _i32(np.asarray(tile_list).reshape(-1, 2))
    tv, tvp = _f64(np.asarray(tile_values, dtype=np.float64).reshape(-1))
    b, bp = _f64(bias)
    x = np.asarray(x, dtype=np.float64).reshape(-1, N)
    x, xp = _f64(x)
    y = np.zeros((x.shape[0], M))
    rc = lib.ppo_structured_forward(M, N, B, rpp, cpp, tlp, tl.shape[0], tvp, bp, xp, x.shape[0], int(act),
                                    y.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc:
        raise OracleError(_ERR.get(rc, str(rc)))
    return y


def layer_forward(layer, x, act: Optional[int] = None, threads: int = 1):
    """Reconstruct + dense product for an object with the fields
    M, N, B, row_perm, col_perm, tile_list, tile_values, bias, act."""
    W = reconstruct(layer.M, layer.N, layer.B, layer.row_perm, layer.col_perm,
                    layer.tile_list, layer.tile_values)
    return dense_forward(W, layer.bias, x, layer.act if act is None else act, threads)


def _round_to(v: np.ndarray, dtype: Optional[str]) -> np.ndarray:
    if dtype == "f16":
        return v.astype(np.float16).astype(np.float64)      # round-to-nearest-even
    if dtype == "f32":
        return v.astype(np.float32).astype(np.float64)
    return v


def chain_forward(layers: Sequence, x, round_intermediate: Optional[str] = None, threads: int = 1):
    """Layer-by-layer evaluation in original coordinates.  Returns a list with,
    per layer, (input used, y, a).  ``round_intermediate`` ("f16"/"f32"/None)
    rounds every layer's output except the last before it feeds the next layer."""
    out = []
    cur = np.asarray(x, dtype=np.float64)
    for li, lay in enumerate(layers):
        y, _, a = layer_forward(lay, cur, threads=threads)
        out.append((cur, y, a))
        cur = _round_to(y, round_intermediate) if li + 1 < len(layers) else y
    return out


def _sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def lstm_step(W, x_t, h_prev, c_prev, threads: int = 1, bias=None):
    """One cell update; returns (pre-activations g [4H], |W||z| [4H], c_t, h_t).
    A layer bias, when given, is part of g = W z + b like in any other layer (Eq. 2)."""
    H = h_prev.size
    z = np.concatenate([np.asarray(x_t, dtype=np.float64).ravel(), h_prev])
    _, g, a = dense_forward(W, bias, z[None, :], 0, threads)
    g = g[0]
    i, f, gg, o = g[0:H], g[H:2 * H], g[2 * H:3 * H], g[3 * H:4 * H]
    c = _sigmoid(f) * c_prev + _sigmoid(i) * np.tanh(gg)
    h = _sigmoid(o) * np.tanh(c)
    return g, a[0], c, h


def lstm_forward(W, x_seq, H: int, h_round: Optional[str] = None, threads: int = 1,
                 h0=None, c0=None, bias=None):
    """Free-running recurrence over x_seq [steps][I].  ``h_round`` rounds h_t to
    the layer's input storage type after every step (c stays fp64 here; the
    comparison tolerance covers the fp32 cell state of the device path)."""
    h = np.zeros(H) if h0 is None else np.asarray(h0, dtype=np.float64).copy()
    c = np.zeros(H) if c0 is None else np.asarray(c0, dtype=np.float64).copy()
    hs = []
    for t in range(x_seq.shape[0]):
        _, _, c, h = lstm_step(W, x_seq[t], h, c, threads, bias)
        h = _round_to(h, h_round)
        hs.append(h.copy())
    return h, c, np.stack(hs) if hs else np.zeros((0, H))
