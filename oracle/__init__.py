"""CPU oracle for sparse 3D convolution -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``spconv_oracle.cpp`` (std::map location table, OFT,
Algorithm 2 in double precision).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library never does
and shares no code with it.

All functions take and return numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "spconv_oracle.cpp")
_LIB = os.path.join(_DIR, "libspconv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with the host C++ compiler (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        i64p = ctypes.POINTER(ctypes.c_int64)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_kmap_build.restype = ctypes.c_void_p
        lib.oracle_kmap_build.argtypes = [i32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        lib.oracle_inverse_kmap_build.restype = ctypes.c_void_p
        lib.oracle_inverse_kmap_build.argtypes = [i32p, ctypes.c_int64, i32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        for name in ("oracle_kmap_n_out", "oracle_kmap_kvol", "oracle_kmap_total_pairs"):
            getattr(lib, name).restype = ctypes.c_int64
            getattr(lib, name).argtypes = [ctypes.c_void_p]
        lib.oracle_kmap_export.restype = None
        lib.oracle_kmap_export.argtypes = [ctypes.c_void_p, i32p, i32p, i64p, i32p, i32p]
        lib.oracle_kmap_free.restype = None
        lib.oracle_kmap_free.argtypes = [ctypes.c_void_p]
        lib.oracle_forward.restype = None
        lib.oracle_forward.argtypes = [f64p, f64p, i32p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                       ctypes.c_int, f64p]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


class OracleError(ValueError):
    """Bad input: invalid argument (1), negative coordinate (2) or duplicate coordinate (3)."""

    def __init__(self, code: int):
        super().__init__({1: "invalid argument", 2: "negative coordinate", 3: "duplicate coordinate"}.get(code, "?"))
        self.code = code


def _ptr(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def build_kmap(coords, kernel: int, stride: int = 1, dilation: int = 1, submanifold: bool = True) -> dict:
    """Kernel map of one layer.

    Returns ``dict(n_in, n_out, kvol, out_coords [n_out,4] int32, oft [n_out,kvol] int32,
    offset_start [kvol+1] int64, pair_in [P] int32, pair_out [P] int32)``.
    ``oft[o, k]`` is the input row feeding output row ``o`` through offset ``k`` or -1
    (the paper's offset table); the pair lists hold the same relation per offset.
    """
    lib = _load()
    c = np.ascontiguousarray(coords, dtype=np.int32).reshape(-1, 4)
    err = ctypes.c_int(0)
    h = lib.oracle_kmap_build(_ptr(c, ctypes.c_int32), c.shape[0], stride, dilation, kernel,
                              int(bool(submanifold)), ctypes.byref(err))
    if not h:
        raise OracleError(err.value)
    return _export(lib, h, c.shape[0])


def build_inverse_kmap(fine, coarse, kernel: int, stride: int, dilation: int = 1) -> dict:
    """Kernel map of the inverse (transposed) convolution of Sec. III-E.

    ``fine`` are the positions before the strided convolution (the inverse layer's outputs, numbered as
    given), ``coarse`` the positions after it (rows of the inverse layer's input features).  Same dict as
    ``build_kmap`` with ``n_in = len(coarse)``, ``n_out = len(fine)``; ``oft[j, k]`` is the coarse row related
    to fine row ``j`` through offset ``k`` or -1.
    """
    lib = _load()
    f = np.ascontiguousarray(fine, dtype=np.int32).reshape(-1, 4)
    c = np.ascontiguousarray(coarse, dtype=np.int32).reshape(-1, 4)
    err = ctypes.c_int(0)
    h = lib.oracle_inverse_kmap_build(_ptr(f, ctypes.c_int32), f.shape[0], _ptr(c, ctypes.c_int32), c.shape[0],
                                      stride, dilation, kernel, ctypes.byref(err))
    if not h:
        raise OracleError(err.value)
    return _export(lib, h, c.shape[0])


def _export(lib, h, n_in: int) -> dict:
    try:
        n_out = lib.oracle_kmap_n_out(h)
        kvol = lib.oracle_kmap_kvol(h)
        p = lib.oracle_kmap_total_pairs(h)
        out_coords = np.empty((n_out, 4), np.int32)
        oft = np.empty((n_out, kvol), np.int32)
        offset_start = np.empty(kvol + 1, np.int64)
        pair_in = np.empty(p, np.int32)
        pair_out = np.empty(p, np.int32)
        lib.oracle_kmap_export(h, _ptr(out_coords, ctypes.c_int32), _ptr(oft, ctypes.c_int32),
                               _ptr(offset_start, ctypes.c_int64), _ptr(pair_in, ctypes.c_int32),
                               _ptr(pair_out, ctypes.c_int32))
    finally:
        lib.oracle_kmap_free(h)
    return dict(n_in=int(n_in), n_out=int(n_out), kvol=int(kvol), out_coords=out_coords, oft=oft,
                offset_start=offset_start, pair_in=pair_in, pair_out=pair_out)


def forward(feats, w, oft) -> np.ndarray:
    """Algorithm 2 in double: ``out[o] = sum_k feats[oft[o,k]] @ w[k]`` over entries != -1.

    ``feats [n_in, cin]``, ``w [kvol, cin, cout]`` (any float dtype; converted exactly to
    float64), ``oft [n_out, kvol]`` int32.  Returns float64 ``[n_out, cout]``.
    """
    lib = _load()
    x = np.ascontiguousarray(feats, dtype=np.float64)
    ww = np.ascontiguousarray(w, dtype=np.float64)
    t = np.ascontiguousarray(oft, dtype=np.int32)
    n_out, kvol = t.shape
    assert ww.shape[0] == kvol and ww.shape[1] == x.shape[1]
    out = np.zeros((n_out, ww.shape[2]), np.float64)
    lib.oracle_forward(_ptr(x, ctypes.c_double), _ptr(ww, ctypes.c_double), _ptr(t, ctypes.c_int32),
                       n_out, kvol, x.shape[1], ww.shape[2], _ptr(out, ctypes.c_double))
    return out


def num_threads() -> int:
    """Threads the forward loop uses (OpenMP default for this host)."""
    return int(_load().oracle_num_threads())


def voxelize(points, n_feat: int, batch_index: int, origin, voxel_size, grid_shape) -> dict:
    """Voxelisation of raw points, the step the paper assumes upstream of its operators (Sec. II-A: a point cloud is
    "partitioned into voxel grids" before the sparse tensor exists).  Plain definition, one point at a time.

    ``points`` float32 ``[n, >= 3 + n_feat]`` rows ``(x, y, z, features...)``.  The cell of a point is
    ``floor((p - origin) / voxel_size)`` per axis, taken in float32 exactly as written (subtract, divide, floor:
    the decision is an integer, so both sides of a comparison must take it in the same precision); points whose
    cell lies outside ``[0, grid_shape)`` are dropped.  Voxels are numbered in the order of their first point;
    a voxel's features are the mean of its points' features (accumulated in float64).  Returns ``dict(coords int32
    [m, 4] rows (batch_index, x, y, z), feats float64 [m, n_feat], counts int64 [m], voxel_of_point int64 [n] (-1 =
    dropped))``.
    """
    pts = np.ascontiguousarray(points, dtype=np.float32)
    o = np.asarray(origin, dtype=np.float32)
    v = np.asarray(voxel_size, dtype=np.float32)
    g = np.asarray(grid_shape, dtype=np.int64)
    index_of = {}
    coords, sums, counts = [], [], []
    voxel_of_point = np.full(len(pts), -1, np.int64)
    for i in range(len(pts)):
        cell = []
        inside = True
        for a in range(3):
            q = np.floor(np.float32(np.float32(pts[i, a] - o[a]) / v[a]))
            if not (0 <= q < g[a]):
                inside = False
                break
            cell.append(int(q))
        if not inside:
            continue
        key = tuple(cell)
        j = index_of.get(key)
        if j is None:
            j = len(coords)
            index_of[key] = j
            coords.append((batch_index,) + key)
            sums.append(np.zeros(n_feat, np.float64))
            counts.append(0)
        sums[j] += pts[i, 3:3 + n_feat].astype(np.float64)
        counts[j] += 1
        voxel_of_point[i] = j
    m = len(coords)
    feats = np.array([s / c for s, c in zip(sums, counts)], np.float64).reshape(m, n_feat)
    return dict(coords=np.array(coords, np.int32).reshape(m, 4), feats=feats, counts=np.array(counts, np.int64),
                voxel_of_point=voxel_of_point)
