"""Seeded synthetic workloads: voxel coordinates, features and weights.

This module only *draws inputs*.  It holds none of the sparse-convolution
arithmetic (no neighbour search, no output-coordinate generation, no
accumulation), so that both the CPU oracle's tests and the CUDA path's tests can
take their inputs from it without sharing any of the method itself.

Every generator is a pure function of its seed (``numpy.random.default_rng``).
Coordinates are ``int32 [n, 4]`` rows ``(b, x, y, z)``, unique, non-negative,
sorted lexicographically (an artefact of ``numpy.unique``; nothing depends on
it, and :func:`shuffle_rows` removes it when a test wants unordered input, which
is how the paper describes the index list: "with no order", Sec. III-B).

The five workloads stand in for the kinds of scene the sparse-convolution
literature measures on (an indoor surface scan, one automotive LiDAR sweep, a
batch of sweeps through a detection encoder).  No public dataset is read or
reproduced; all geometry is drawn from the seed.
"""
from __future__ import annotations

import numpy as np

DTYPES = ("f32", "f16", "bf16")


# --------------------------------------------------------------------------
# value helpers (rounding inputs onto a storage grid; not method arithmetic)
# --------------------------------------------------------------------------
def round_to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    """Return ``a`` as float32 whose every value is exactly representable in ``dtype``.

    Round-to-nearest-even, as a tensor library's cast would do.  bf16 is done on
    the bit pattern because numpy has no bfloat16.
    """
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype == "f16":
        return a.astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        u = a.view(np.uint32).astype(np.uint64)
        bias = np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
        r = ((u + bias) >> np.uint64(16)) << np.uint64(16)
        return r.astype(np.uint32).view(np.float32).reshape(a.shape)
    raise ValueError(f"unknown dtype {dtype!r}")


def to_storage_bits(a: np.ndarray, dtype: str) -> np.ndarray:
    """Bit pattern of already-rounded float32 values in the storage dtype.

    f32 -> float32 array, f16 -> float16 array, bf16 -> uint16 array holding the
    upper halves.  Used to hand the same numbers to device memory.
    """
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype == "f16":
        return a.astype(np.float16)
    if dtype == "bf16":
        return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(a.shape)
    raise ValueError(f"unknown dtype {dtype!r}")


def from_storage_bits(a: np.ndarray, dtype: str) -> np.ndarray:
    """Inverse of :func:`to_storage_bits`: storage array -> float32 values."""
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f16":
        return np.asarray(a).view(np.float16).astype(np.float32)
    if dtype == "bf16":
        u = np.asarray(a).view(np.uint16).astype(np.uint32) << np.uint32(16)
        return u.view(np.float32).reshape(np.asarray(a).shape)
    raise ValueError(f"unknown dtype {dtype!r}")


def features(n: int, channels: int, dtype: str, seed: int) -> np.ndarray:
    """Feature rows ``[n, channels]`` ~ N(0, 1), rounded onto ``dtype``'s grid."""
    rng = np.random.default_rng([seed, 0xFEA7])
    return round_to_dtype(rng.standard_normal((n, channels), dtype=np.float32), dtype)


def weights(kernel_volume: int, cin: int, cout: int, dtype: str, seed: int) -> np.ndarray:
    """Weights ``[K^3, cin, cout]`` ~ N(0, 1/(K^3 * cin)), rounded onto ``dtype``'s grid."""
    rng = np.random.default_rng([seed, 0x3E16])
    w = rng.standard_normal((kernel_volume, cin, cout), dtype=np.float32)
    w *= np.float32(1.0 / np.sqrt(kernel_volume * cin))
    return round_to_dtype(w, dtype)


# --------------------------------------------------------------------------
# coordinate helpers
# --------------------------------------------------------------------------
def _unique_rows(b: int, v: np.ndarray) -> np.ndarray:
    c = np.concatenate([np.full((len(v), 1), b, np.int64), v.astype(np.int64)], axis=1)
    return np.unique(c, axis=0).astype(np.int32)


def shuffle_rows(coords: np.ndarray, seed: int) -> np.ndarray:
    """The same voxel set in a seeded random row order."""
    rng = np.random.default_rng([seed, 0x5F1E])
    return np.ascontiguousarray(coords[rng.permutation(len(coords))])


def uniform_voxels(n: int, grid: int, seed: int, batch: int = 0) -> np.ndarray:
    """``n`` distinct voxels drawn uniformly from a ``grid``^3 cube (workload 1)."""
    rng = np.random.default_rng(seed)
    idx = rng.choice(grid ** 3, size=n, replace=False)
    v = np.stack([idx // (grid * grid), (idx // grid) % grid, idx % grid], axis=1)
    return _unique_rows(batch, v)


def indoor_surfaces(seed: int, target: int = 100_000, batch: int = 0) -> np.ndarray:
    """Voxels on the surfaces of 20 axis-aligned boxes and 5 spheres in 512x512x128 (workload 2).

    Each of the 25 shapes receives the same number of uniformly drawn surface
    samples (``1.3 * target / 25``); samples are floored to voxels and
    deduplicated, which lands near ``target`` voxels.
    """
    rng = np.random.default_rng(seed)
    dims = np.array([512, 512, 128], dtype=np.float64)
    per = target * 13 // 10 // 25
    pts = []
    for _ in range(20):
        size = rng.uniform(20, 160, 3) * np.array([1.0, 1.0, 0.4])
        lo = rng.uniform(0, 1, 3) * (dims - size)
        face = rng.integers(0, 6, per)
        u = rng.uniform(0, 1, (per, 3))
        u[np.arange(per), face // 2] = face % 2
        pts.append(lo + u * size)
    for _ in range(5):
        r = rng.uniform(15, 50)
        c = np.array([rng.uniform(r, 512 - r), rng.uniform(r, 512 - r), rng.uniform(r, 128 - r)])
        d = rng.normal(size=(per, 3))
        d /= np.linalg.norm(d, axis=1, keepdims=True)
        pts.append(c + r * d)
    v = np.floor(np.concatenate(pts)).astype(np.int64)
    keep = ((v >= 0) & (v < dims.astype(np.int64))).all(axis=1)
    return _unique_rows(batch, v[keep])


LIDAR_GRID = (1408, 1600, 41)


LIDAR_ORIGIN = (-35.2, -40.0, -3.0)
LIDAR_VOXEL = (0.05, 0.05, 0.1)


def _lidar_hits(seed: int) -> np.ndarray:
    """Hit points (float64 [m, 3], metres, sensor at the origin) of one synthetic sweep; see :func:`lidar_sweep`."""
    rng = np.random.default_rng(seed)
    el = np.deg2rad(np.linspace(-25.0, 3.0, 64))
    az = np.arange(2048) * (2.0 * np.pi / 2048)
    e, a = np.meshgrid(el, az, indexing="ij")
    d = np.stack([np.cos(e) * np.cos(a), np.cos(e) * np.sin(a), np.sin(e)], axis=-1).reshape(-1, 3)
    t = np.full(len(d), np.inf)
    down = d[:, 2] < 0
    t[down] = -1.7 / d[down, 2]
    for _ in range(30):
        rad = rng.uniform(5, 60)
        th = rng.uniform(0, 2 * np.pi)
        size = rng.uniform(1.5, 5, 3)
        c = np.array([rad * np.cos(th), rad * np.sin(th), -1.7 + size[2] / 2])
        lo, hi = c - size / 2, c + size / 2
        with np.errstate(divide="ignore", invalid="ignore"):
            t1, t2 = lo / d, hi / d
        tn = np.minimum(t1, t2).max(axis=1)
        tf = np.maximum(t1, t2).min(axis=1)
        hit = (tn <= tf) & (tn > 0)
        t = np.where(hit & (tn < t), tn, t)
    ok = t <= 70.0
    t = t[ok] + rng.uniform(-0.02, 0.02, int(ok.sum()))
    return d[ok] * t[:, None]


def lidar_sweep(seed: int, batch: int = 0) -> np.ndarray:
    """One sweep of a synthetic 64-beam spinning LiDAR, voxelised (workload 3).

    64 elevations uniform in [-25, +3] degrees x 2048 azimuth steps from a sensor
    at the origin.  A ray stops at the ground plane z = -1.7 m or at the nearest
    of 30 random boxes (edges 1.5-5 m, standing on the ground, centres at range
    5-60 m and uniform bearing); hits beyond 70 m are dropped; range noise is
    uniform +-2 cm.  Voxel size (0.05, 0.05, 0.1) m, grid 1408 x 1600 x 41 with
    origin (-35.2, -40.0, -3.0) m so the sensor sits at the centre.
    """
    p = _lidar_hits(seed)
    origin = np.array(LIDAR_ORIGIN)
    vsize = np.array(LIDAR_VOXEL)
    v = np.floor((p - origin) / vsize).astype(np.int64)
    keep = ((v >= 0) & (v < np.array(LIDAR_GRID))).all(axis=1)
    return _unique_rows(batch, v[keep])


def lidar_points(seed: int, n_feat: int = 1) -> np.ndarray:
    """The raw returns of the same sweep as float32 ``[m, 3 + n_feat]`` rows ``(x, y, z, features...)`` in beam
    order, for the voxeliser: positions rounded to float32, features uniform in [0, 1) from a stream of their own."""
    p = _lidar_hits(seed).astype(np.float32)
    f = np.random.default_rng([seed, 0xFEA7]).random((len(p), n_feat), dtype=np.float32)
    return np.ascontiguousarray(np.concatenate([p, f], axis=1))


def lidar_batch(seeds=(0, 1, 2, 3)) -> np.ndarray:
    """Independent sweeps concatenated with batch index 0..len(seeds)-1 (workload 5)."""
    return np.ascontiguousarray(np.concatenate([lidar_sweep(s, batch=b) for b, s in enumerate(seeds)]))


def random_blob(n: int, extent: int, seed: int, batches: int = 1) -> np.ndarray:
    """Small dense-ish random voxel set for tests: ``n`` draws in an ``extent``^3 cube per batch."""
    rng = np.random.default_rng([seed, 0xB10B])
    out = []
    for b in range(batches):
        v = rng.integers(0, extent, size=(n, 3))
        out.append(_unique_rows(b, v))
    return np.ascontiguousarray(np.concatenate(out))


# Encoder stack of workload 5: (kind, kernel, stride, cin, cout)
ENCODER_STACK = (
    ("subm", 3, 1, 16, 16),
    ("spconv", 3, 2, 16, 32),
    ("subm", 3, 1, 32, 32),
    ("spconv", 3, 2, 32, 64),
    ("subm", 3, 1, 64, 64),
    ("spconv", 3, 2, 64, 128),
    ("subm", 3, 1, 128, 128),
)


def config(index: int, seed: int = 0) -> dict:
    """Workload ``index`` in 1..5 as a dict: coords plus the layer list to run on them.

    Each layer is ``dict(kind, kernel, stride, dilation, cin, cout, dtype)``.
    """
    if index == 1:
        coords = uniform_voxels(2000, 64, seed)
        layers = [dict(kind="subm", kernel=3, stride=1, dilation=1, cin=16, cout=16, dtype="f32")]
        name = "tiny-subm3-16x16-f32"
    elif index == 2:
        coords = indoor_surfaces(seed)
        layers = [dict(kind="subm", kernel=3, stride=1, dilation=1, cin=32, cout=32, dtype="f16")]
        name = "indoor-subm3-32x32-f16"
    elif index == 3:
        coords = lidar_sweep(seed)
        layers = [dict(kind="subm", kernel=3, stride=1, dilation=1, cin=64, cout=64, dtype="bf16")]
        name = "lidar-subm3-64x64-bf16"
    elif index == 4:
        coords = lidar_sweep(seed)
        layers = [
            dict(kind="spconv", kernel=3, stride=2, dilation=1, cin=64, cout=128, dtype="bf16"),
            dict(kind="spconv", kernel=2, stride=2, dilation=1, cin=64, cout=64, dtype="bf16"),
        ]
        name = "lidar-spconv-s2-bf16"
    elif index == 5:
        coords = lidar_batch(tuple(range(seed, seed + 4)))
        layers = [
            dict(kind=k, kernel=ks, stride=s, dilation=1, cin=ci, cout=co, dtype="bf16")
            for (k, ks, s, ci, co) in ENCODER_STACK
        ]
        name = "lidar-batch4-encoder-bf16"
    else:
        raise ValueError("config index must be 1..5")
    return dict(name=name, index=index, seed=seed, coords=coords, layers=layers)
