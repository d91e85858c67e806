"""The voxeliser on the GPU against the CPU oracle's point-by-point definition, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def _check(points_np, n_feat, batch, origin, vsize, grid):
    ref = oracle.voxelize(points_np, n_feat, batch, origin, vsize, grid)
    pts = torch.from_numpy(points_np).cuda()
    coords, feats, counts = binding.spconv_voxelize(pts, n_feat, batch, origin, vsize, grid, with_counts=True)
    torch.cuda.synchronize()
    assert np.array_equal(coords.cpu().numpy(), ref["coords"])            # integer work: bit-exact, same numbering
    assert np.array_equal(counts.cpu().numpy(), ref["counts"])
    if n_feat:
        got = feats.cpu().numpy().astype(np.float64)
        assert np.abs(got - ref["feats"]).max() <= 1e-5 * max(1.0, np.abs(ref["feats"]).max())   # fp32 sums of up to tens of values
    return coords, feats


def test_lidar_returns_to_voxels_and_on_into_a_kernel_map():
    """All 121 k returns of a synthetic sweep (two feature columns, beam order): voxel rows, counts and means equal the
    oracle's; twice the same rows; and the rows go straight into a kernel map that equals the oracle's for them."""
    pts = wl.lidar_points(0, n_feat=2)
    coords, _ = _check(pts, 2, 3, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID)
    again, _ = _check(pts, 2, 3, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID)
    assert torch.equal(coords, again)
    assert len(coords) == len(wl.lidar_sweep(0)) or abs(len(coords) - len(wl.lidar_sweep(0))) < 50   # float32 vs float64 cell edges
    km = binding.spconv_build_kmap(coords.contiguous(), 1, 1, 3, True)
    ref = oracle.build_kmap(coords.cpu().numpy(), 3, 1, 1, True)
    assert np.array_equal(km.nbr.cpu().numpy().T, ref["oft"]) and km.total_pairs == len(ref["pair_in"])


@pytest.mark.parametrize("n_feat,stride", [(0, 3), (1, 4), (5, 9)])
def test_small_clouds_edges_and_extra_columns(n_feat, stride):
    rng = np.random.default_rng(n_feat)
    pts = np.zeros((5000, stride), np.float32)
    pts[:, :3] = rng.uniform(-1.2, 1.2, (5000, 3))          # some points fall outside the unit grid below
    pts[:, 3:] = rng.standard_normal((5000, stride - 3))
    pts[:40, :3] = np.round(pts[:40, :3] * 8) / 8            # points exactly on cell boundaries
    _check(pts, n_feat, 0, (-1.0, -1.0, -1.0), (0.125, 0.125, 0.25), (16, 16, 8))


def test_voxelize_limits_and_errors():
    E = binding.SpconvError
    pts = torch.from_numpy(wl.lidar_points(1, n_feat=1)[:20000]).cuda()
    with pytest.raises(E) as e:                                            # room for 10 rows only
        binding.spconv_voxelize(pts, 1, 0, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID, capacity=10)
    assert e.value.status == 9 and e.value.n_voxels > 10
    coords, feats = binding.spconv_voxelize(pts, 1, 0, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID, capacity=e.value.n_voxels)
    assert len(coords) == e.value.n_voxels
    far = torch.full((100, 4), 1e6, dtype=torch.float32, device="cuda")   # every point outside the grid
    coords, feats = binding.spconv_voxelize(far, 1, 0, (0, 0, 0), (1, 1, 1), (4, 4, 4))
    assert len(coords) == 0
    coords, feats = binding.spconv_voxelize(pts[:0].contiguous(), 1, 0, (0, 0, 0), (1, 1, 1), (4, 4, 4))
    assert len(coords) == 0
    for kwargs in (dict(voxel_size=(0.0, 1, 1)), dict(grid_shape=(0, 4, 4)), dict(batch_index=70000), dict(n_feat=2)):
        args = dict(n_feat=1, batch_index=0, origin=(0, 0, 0), voxel_size=(1, 1, 1), grid_shape=(4, 4, 4))
        args.update(kwargs)
        with pytest.raises(E) as e:
            binding.spconv_voxelize(pts, **args)
        assert e.value.status == 1
