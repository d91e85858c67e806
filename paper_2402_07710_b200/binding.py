"""ctypes binding of the C ABI in ``include/spconv_b200.h``.

Argument marshalling only: every step of the path runs inside ``libspconv_b200.so``.
PyTorch supplies device memory and the CUDA stream, nothing else.  There is no fallback:
if the shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libspconv_b200.so")

F32, F16, BF16 = 0, 1, 2
ALGO = {"auto": 0, "simt": 1, "tcgen05": 2, "tcgen05_single": 3}
ROWS_BY_OFFSET_SET, ROWS_AS_GIVEN = 0, 1
_TORCH_DTYPE = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
DTYPE_BY_NAME = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}

EXPORTS = (
    "spconv_build_kmap", "spconv_build_kmap_ordered", "spconv_build_inverse_kmap", "spconv_build_kmap_dense", "spconv_kmap_info", "spconv_kmap_destroy", "spconv_forward", "spconv_forward_algo",
    "spconv_last_device_status", "spconv_layer", "spconv_layer_host", "spconv_strerror", "spconv_subm_offset_table_noalloc",
    "spconv_kmap_status_words", "spconv_test_hook", "spconv_voxelize",
)
HOOK_TABLE_SLOTS, HOOK_PIPE_WAIT_LIMIT_US = 1, 2
NOALLOC_MAX_VOXELS = 131072


class SpconvError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {strerror(status)} (status {status})")
        self.status = status


class _KmapInfo(ctypes.Structure):
    _fields_ = [
        ("kernel_size", ctypes.c_int32), ("stride", ctypes.c_int32), ("dilation", ctypes.c_int32),
        ("submanifold", ctypes.c_int32), ("kvol", ctypes.c_int32), ("n_tiles", ctypes.c_int32),
        ("n_in", ctypes.c_int64), ("n_out", ctypes.c_int64), ("total_pairs", ctypes.c_int64),
        ("out_coords", ctypes.c_void_p), ("nbr", ctypes.c_void_p), ("pair_in", ctypes.c_void_p),
        ("pair_out", ctypes.c_void_p), ("offset_start", ctypes.POINTER(ctypes.c_int64)),
        ("tile_rows", ctypes.c_void_p), ("tile_blocks", ctypes.c_int64),
        ("inverse", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """Load the CUDA library; raise (never fall back) if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2402_07710_b200.build` "
                "(nvcc, sm_100a).  There is no CPU or PyTorch fallback."
            )
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        lib.spconv_build_kmap.restype = i32
        lib.spconv_build_kmap.argtypes = [vp, i64, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        lib.spconv_build_kmap_ordered.restype = i32
        lib.spconv_build_kmap_ordered.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        lib.spconv_build_inverse_kmap.restype = i32
        lib.spconv_build_inverse_kmap.argtypes = [vp, i64, vp, i64, i32, i32, i32, vp, ctypes.POINTER(vp)]
        lib.spconv_build_kmap_dense.restype = i32
        lib.spconv_build_kmap_dense.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_int32), i32, i32, vp, ctypes.POINTER(vp)]
        lib.spconv_kmap_info.restype = i32
        lib.spconv_kmap_info.argtypes = [vp, ctypes.POINTER(_KmapInfo)]
        lib.spconv_kmap_destroy.restype = None
        lib.spconv_kmap_destroy.argtypes = [vp]
        lib.spconv_forward.restype = i32
        lib.spconv_forward.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        lib.spconv_forward_algo.restype = i32
        lib.spconv_forward_algo.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        lib.spconv_last_device_status.restype = i32
        lib.spconv_last_device_status.argtypes = [vp, vp]
        lib.spconv_layer.restype = i32
        lib.spconv_layer.argtypes = [vp, i64, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, i64, vp, ctypes.POINTER(vp)]
        lib.spconv_layer_host.restype = i32
        lib.spconv_layer_host.argtypes = [vp, i64, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp, i64,
                                          ctypes.POINTER(i64), vp]
        lib.spconv_subm_offset_table_noalloc.restype = i32
        lib.spconv_subm_offset_table_noalloc.argtypes = [vp, i64, i32, i32, vp, vp]
        lib.spconv_kmap_status_words.restype = i32
        lib.spconv_kmap_status_words.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        lib.spconv_voxelize.restype = i32
        lib.spconv_voxelize.argtypes = [vp, i64, i32, i32, i32, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                        ctypes.POINTER(ctypes.c_int32), vp, vp, vp, i64, ctypes.POINTER(i64), vp]
        lib.spconv_test_hook.restype = i32
        lib.spconv_test_hook.argtypes = [i32, ctypes.c_longlong]
        lib.spconv_strerror.restype = ctypes.c_char_p
        lib.spconv_strerror.argtypes = [i32]
        _lib = lib
    return _lib


def strerror(status: int) -> str:
    return load().spconv_strerror(int(status)).decode()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream) -> int:
    """CUDA stream handle: the given torch stream, else the current stream of the current device."""
    if stream is None:
        if _raw_stream is not None:   # same value as torch.cuda.current_stream().cuda_stream, without building a Stream object
            return int(_raw_stream(torch.cuda.current_device()))
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class _DevArray:
    """View of library-owned device memory through the CUDA array interface (no copy)."""

    def __init__(self, ptr: int, shape, typestr: str, owner):
        self.__cuda_array_interface__ = {
            "shape": tuple(int(s) for s in shape), "typestr": typestr, "data": (int(ptr), False), "version": 2,
        }
        self._owner = owner


class Kmap:
    """Kernel map handle (owns device memory inside the library until closed or collected)."""

    def __init__(self, handle: int):
        self._h = ctypes.c_void_p(handle)
        info = _KmapInfo()
        st = load().spconv_kmap_info(self._h, ctypes.byref(info))
        if st != 0:
            raise SpconvError(st, "spconv_kmap_info")
        self._info = info
        for name in ("kernel_size", "stride", "dilation", "submanifold", "kvol", "n_tiles", "n_in", "n_out",
                     "total_pairs", "tile_blocks", "inverse"):
            setattr(self, name, int(getattr(info, name)))
        self._offset_start = None   # converted on first use: the build sits on the latency path of a layer

    @property
    def offset_start(self) -> np.ndarray:
        """[kvol + 1] int64: pairs of offset k are pair_in / pair_out [offset_start[k] : offset_start[k + 1]]."""
        if self._offset_start is None:
            self._offset_start = np.ctypeslib.as_array(self._info.offset_start, shape=(self.kvol + 1,)).astype(np.int64)
        return self._offset_start

    def _view(self, ptr, shape):
        n = int(np.prod(shape))
        if n == 0 or not ptr:
            return torch.empty(tuple(shape), dtype=torch.int32, device="cuda")
        return torch.as_tensor(_DevArray(ptr, shape, "<i4", self), device="cuda")

    @property
    def out_coords(self) -> torch.Tensor:
        return self._view(self._info.out_coords, (self.n_out, 4))

    @property
    def nbr(self) -> torch.Tensor:
        """[kvol, n_out] int32: input row feeding output row o through offset k, or -1."""
        return self._view(self._info.nbr, (self.kvol, self.n_out))

    @property
    def pair_in(self) -> torch.Tensor:
        return self._view(self._info.pair_in, (self.total_pairs,))

    @property
    def pair_out(self) -> torch.Tensor:
        return self._view(self._info.pair_out, (self.total_pairs,))

    @property
    def tile_rows(self) -> torch.Tensor:
        return self._view(self._info.tile_rows, (self.n_tiles, 128))

    def close(self):
        if self._h:
            load().spconv_kmap_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def spconv_build_kmap(coords: torch.Tensor, stride: int = 1, dilation: int = 1, kernel_size: int = 3,
                      submanifold: bool = True, stream=None, row_order: int | None = None) -> Kmap:
    """Build the kernel map of one layer from device coordinates ``int32 [n, 4]`` rows (b, x, y, z).
    ``row_order`` (``ROWS_BY_OFFSET_SET`` / ``ROWS_AS_GIVEN``) goes through ``spconv_build_kmap_ordered``."""
    if not (coords.is_cuda and coords.dtype == torch.int32 and coords.dim() == 2 and coords.shape[1] == 4
            and coords.is_contiguous()):
        raise ValueError("coords must be a contiguous CUDA int32 tensor of shape [n, 4]")
    h = ctypes.c_void_p(None)
    if row_order is not None:
        st = load().spconv_build_kmap_ordered(ctypes.c_void_p(coords.data_ptr() if coords.numel() else 0), coords.shape[0],
                                              int(stride), int(dilation), int(kernel_size), int(bool(submanifold)), int(row_order),
                                              ctypes.c_void_p(_stream_ptr(stream)), ctypes.byref(h))
        if st != 0:
            raise SpconvError(st, "spconv_build_kmap_ordered")
        return Kmap(h.value)
    st = load().spconv_build_kmap(ctypes.c_void_p(coords.data_ptr() if coords.numel() else 0), coords.shape[0],
                                  int(stride), int(dilation), int(kernel_size), int(bool(submanifold)),
                                  ctypes.c_void_p(_stream_ptr(stream)), ctypes.byref(h))
    if st != 0:
        raise SpconvError(st, "spconv_build_kmap")
    return Kmap(h.value)


def spconv_build_kmap_dense(coords: torch.Tensor, grid_shape, dilation: int = 1, kernel_size: int = 3, stream=None) -> Kmap:
    """Submanifold kernel map built through a dense-array location table over ``grid_shape = (B, X, Y, Z)``."""
    if not (coords.is_cuda and coords.dtype == torch.int32 and coords.dim() == 2 and coords.shape[1] == 4
            and coords.is_contiguous()):
        raise ValueError("coords must be a contiguous CUDA int32 tensor of shape [n, 4]")
    shape = (ctypes.c_int32 * 4)(*[int(v) for v in grid_shape])
    h = ctypes.c_void_p(None)
    st = load().spconv_build_kmap_dense(ctypes.c_void_p(coords.data_ptr() if coords.numel() else 0), coords.shape[0], shape,
                                        int(dilation), int(kernel_size), ctypes.c_void_p(_stream_ptr(stream)), ctypes.byref(h))
    if st != 0:
        raise SpconvError(st, "spconv_build_kmap_dense")
    return Kmap(h.value)


def spconv_build_inverse_kmap(fine_coords: torch.Tensor, coarse_coords: torch.Tensor, stride: int, dilation: int = 1,
                              kernel_size: int = 3, stream=None) -> Kmap:
    """Kernel map of the inverse (transposed) convolution: output rows are ``fine_coords`` (positions before the
    strided layer), input rows ``coarse_coords`` (positions after it); both device ``int32 [n, 4]``."""
    for c in (fine_coords, coarse_coords):
        if not (c.is_cuda and c.dtype == torch.int32 and c.dim() == 2 and c.shape[1] == 4 and c.is_contiguous()):
            raise ValueError("coordinates must be contiguous CUDA int32 tensors of shape [n, 4]")
    h = ctypes.c_void_p(None)
    st = load().spconv_build_inverse_kmap(ctypes.c_void_p(fine_coords.data_ptr() if fine_coords.numel() else 0), fine_coords.shape[0],
                                          ctypes.c_void_p(coarse_coords.data_ptr() if coarse_coords.numel() else 0),
                                          coarse_coords.shape[0], int(stride), int(dilation), int(kernel_size),
                                          ctypes.c_void_p(_stream_ptr(stream)), ctypes.byref(h))
    if st != 0:
        raise SpconvError(st, "spconv_build_inverse_kmap")
    return Kmap(h.value)


def spconv_forward(feats: torch.Tensor, weights: torch.Tensor, kmap: Kmap, out: torch.Tensor | None = None,
                   algo: str = "auto", stream=None) -> torch.Tensor:
    """``out[o] = sum_k W_k^T feats[nbr(o, k)]``; ``feats [n_in, cin]``, ``weights [kvol, cin, cout]``."""
    if feats.dtype not in _TORCH_DTYPE or weights.dtype != feats.dtype:
        raise ValueError("feats and weights must share a dtype among float32 / float16 / bfloat16")
    if not (feats.is_cuda and weights.is_cuda and feats.is_contiguous() and weights.is_contiguous()):
        raise ValueError("feats and weights must be contiguous CUDA tensors")
    if feats.dim() != 2 or weights.dim() != 3 or feats.shape[0] != kmap.n_in or weights.shape[0] != kmap.kvol \
            or weights.shape[1] != feats.shape[1]:
        raise ValueError("shape mismatch between feats, weights and the kernel map")
    cin, cout = int(weights.shape[1]), int(weights.shape[2])
    if out is None:
        out = torch.empty((kmap.n_out, cout), dtype=feats.dtype, device=feats.device)
    elif not (out.is_cuda and out.is_contiguous() and out.dtype == feats.dtype and tuple(out.shape) == (kmap.n_out, cout)):
        raise ValueError("out must be a contiguous CUDA tensor [n_out, cout] of the feature dtype")
    st = load().spconv_forward_algo(ctypes.c_void_p(feats.data_ptr() if feats.numel() else 0),
                                    ctypes.c_void_p(weights.data_ptr()), kmap._h,
                                    ctypes.c_void_p(out.data_ptr() if out.numel() else 0), cin, cout,
                                    _TORCH_DTYPE[feats.dtype], ALGO[algo], ctypes.c_void_p(_stream_ptr(stream)))
    if st != 0:
        raise SpconvError(st, "spconv_forward")
    return out


def spconv_layer(coords: torch.Tensor, feats: torch.Tensor, weights: torch.Tensor, stride: int = 1, dilation: int = 1,
                 kernel_size: int = 3, submanifold: bool = True, out: torch.Tensor | None = None, stream=None):
    """Kernel map and forward of one layer with one call (device tensors); returns ``(kmap, out)``.  For a strided
    layer ``out`` must be given with enough rows (its first ``kmap.n_out`` rows are written)."""
    if not (coords.is_cuda and coords.dtype == torch.int32 and coords.dim() == 2 and coords.shape[1] == 4
            and coords.is_contiguous()):
        raise ValueError("coords must be a contiguous CUDA int32 tensor of shape [n, 4]")
    if feats.dtype not in _TORCH_DTYPE or weights.dtype != feats.dtype:
        raise ValueError("feats and weights must share a dtype among float32 / float16 / bfloat16")
    if not (feats.is_cuda and weights.is_cuda and feats.is_contiguous() and weights.is_contiguous()):
        raise ValueError("feats and weights must be contiguous CUDA tensors")
    if feats.dim() != 2 or weights.dim() != 3 or feats.shape[0] != coords.shape[0] or weights.shape[1] != feats.shape[1] \
            or weights.shape[0] != int(kernel_size) ** 3:
        raise ValueError("shape mismatch between coords, feats and weights")
    cin, cout = int(weights.shape[1]), int(weights.shape[2])
    if out is None:
        if not submanifold:
            raise ValueError("a strided layer needs an output tensor with room for its rows")
        out = torch.empty((coords.shape[0], cout), dtype=feats.dtype, device=feats.device)
    elif not (out.is_cuda and out.is_contiguous() and out.dtype == feats.dtype and out.dim() == 2 and out.shape[1] == cout):
        raise ValueError("out must be a contiguous CUDA tensor [rows, cout] of the feature dtype")
    h = ctypes.c_void_p(None)
    st = load().spconv_layer(ctypes.c_void_p(coords.data_ptr() if coords.numel() else 0), coords.shape[0],
                             ctypes.c_void_p(feats.data_ptr() if feats.numel() else 0), ctypes.c_void_p(weights.data_ptr()),
                             int(stride), int(dilation), int(kernel_size), int(bool(submanifold)), cin, cout,
                             _TORCH_DTYPE[feats.dtype], ctypes.c_void_p(out.data_ptr() if out.numel() else 0),
                             int(out.shape[0]), ctypes.c_void_p(_stream_ptr(stream)), ctypes.byref(h))
    if st != 0:
        raise SpconvError(st, "spconv_layer")
    return Kmap(h.value), out


def spconv_last_device_status(kmap: Kmap, stream=None) -> int:
    return int(load().spconv_last_device_status(kmap._h, ctypes.c_void_p(_stream_ptr(stream))))


def spconv_voxelize(points: torch.Tensor, n_feat: int, batch_index: int, origin, voxel_size, grid_shape, capacity: int | None = None,
                    with_counts: bool = False, stream=None):
    """Voxelise device points ``float32 [n, >= 3 + n_feat]``; returns ``(coords int32 [m, 4], feats float32 [m, n_feat])``
    (and ``counts int32 [m]`` with ``with_counts``).  Output tensors are allocated here for ``capacity`` rows (default n)."""
    if not (points.is_cuda and points.dtype == torch.float32 and points.dim() == 2 and points.is_contiguous()):
        raise ValueError("points must be a contiguous CUDA float32 tensor [n, columns]")
    n, stride = int(points.shape[0]), int(points.shape[1])
    cap = n if capacity is None else int(capacity)
    coords = torch.empty((max(cap, 1), 4), dtype=torch.int32, device=points.device)
    feats = torch.empty((max(cap, 1), max(n_feat, 1)), dtype=torch.float32, device=points.device)
    counts = torch.empty((max(cap, 1),), dtype=torch.int32, device=points.device) if with_counts else None
    m = ctypes.c_int64(0)
    st = load().spconv_voxelize(ctypes.c_void_p(points.data_ptr() if n else 0), n, stride, int(n_feat), int(batch_index),
                                (ctypes.c_float * 3)(*[float(v) for v in origin]), (ctypes.c_float * 3)(*[float(v) for v in voxel_size]),
                                (ctypes.c_int32 * 3)(*[int(v) for v in grid_shape]), ctypes.c_void_p(coords.data_ptr()),
                                ctypes.c_void_p(feats.data_ptr() if n_feat else 0), ctypes.c_void_p(counts.data_ptr() if with_counts else 0),
                                cap, ctypes.byref(m), ctypes.c_void_p(_stream_ptr(stream)))
    if st != 0:
        err = SpconvError(st, "spconv_voxelize")
        err.n_voxels = int(m.value)
        raise err
    out = (coords[:m.value], feats[:m.value, :n_feat])
    return out + (counts[:m.value],) if with_counts else out


def spconv_kmap_status_words(kmap: Kmap) -> list:
    """The 16 status words device kernels of this map wrote (diagnostics)."""
    words = (ctypes.c_uint32 * 16)()
    st = load().spconv_kmap_status_words(kmap._h, words)
    if st != 0:
        raise SpconvError(st, "spconv_kmap_status_words")
    return list(words)


def spconv_test_hook(which: int, value: int) -> None:
    """Test hooks of the library (see the header); value 0 restores normal behaviour."""
    st = load().spconv_test_hook(int(which), int(value))
    if st != 0:
        raise SpconvError(st, "spconv_test_hook")


def spconv_layer_host(coords: torch.Tensor, feats: torch.Tensor, weights: torch.Tensor, stride: int, dilation: int,
                      kernel_size: int, submanifold: bool, out: torch.Tensor, out_coords: torch.Tensor | None = None,
                      stream=None) -> int:
    """Whole layer from HOST tensors (ideally pinned); returns n_out.  ``out`` is a host tensor with capacity rows."""
    for t in (coords, feats, weights, out):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("spconv_layer_host takes contiguous host tensors")
    n_out = ctypes.c_int64(0)
    cin, cout = int(weights.shape[1]), int(weights.shape[2])
    st = load().spconv_layer_host(ctypes.c_void_p(coords.data_ptr()), coords.shape[0], ctypes.c_void_p(feats.data_ptr()),
                                  ctypes.c_void_p(weights.data_ptr()), int(stride), int(dilation), int(kernel_size),
                                  int(bool(submanifold)), cin, cout, _TORCH_DTYPE[feats.dtype],
                                  ctypes.c_void_p(out.data_ptr()),
                                  ctypes.c_void_p(out_coords.data_ptr() if out_coords is not None else 0),
                                  out.shape[0], ctypes.byref(n_out), ctypes.c_void_p(_stream_ptr(stream)))
    if st != 0:
        raise SpconvError(st, "spconv_layer_host")
    return int(n_out.value)


def spconv_subm_offset_table_noalloc(coords: torch.Tensor, kernel_size: int, dilation: int, nbr_out: torch.Tensor,
                                     stream=None) -> torch.Tensor:
    """Fill the caller's ``nbr_out`` (int32 ``[kernel_size**3, n]``) with the submanifold offset table.

    For callers that may not allocate device memory (everything this needs beyond the two tensors lives in a
    fixed array inside the library); ``n`` is limited to ``NOALLOC_MAX_VOXELS``.  This wrapper allocates
    nothing either: both tensors come from the caller.
    """
    if not (coords.is_cuda and coords.dtype == torch.int32 and coords.dim() == 2 and coords.shape[1] == 4
            and coords.is_contiguous()):
        raise ValueError("coords must be a contiguous CUDA int32 tensor of shape [n, 4]")
    n = coords.shape[0]
    if not (nbr_out.is_cuda and nbr_out.dtype == torch.int32 and nbr_out.is_contiguous()
            and tuple(nbr_out.shape) == (kernel_size ** 3, n)):
        raise ValueError("nbr_out must be a contiguous CUDA int32 tensor of shape [kernel_size**3, n]")
    st = load().spconv_subm_offset_table_noalloc(ctypes.c_void_p(coords.data_ptr() if n else 0), n, int(kernel_size),
                                                 int(dilation), ctypes.c_void_p(nbr_out.data_ptr() if n else 0),
                                                 ctypes.c_void_p(_stream_ptr(stream)))
    if st != 0:
        raise SpconvError(st, "spconv_subm_offset_table_noalloc")
    return nbr_out
