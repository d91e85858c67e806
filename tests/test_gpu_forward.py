"""GPU forward vs the CPU oracle (Algorithm 2 in fp64), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL, check_layer, gpu_kmap, kmap_to_numpy, rel_err, to_device

pytestmark = pytest.mark.gpu


def _layer(kind, K, s, cin, cout, dtype, d=1):
    return dict(kind=kind, kernel=K, stride=s, dilation=d, cin=cin, cout=cout, dtype=dtype)


def test_config1_fp32_simt():
    cfg = wl.config(1)
    check_layer(cfg["coords"], cfg["layers"][0])


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("cin,cout", [(16, 16), (8, 24), (64, 32), (160, 136)])
def test_simt_kernel_small(dtype, cin, cout):
    if dtype == "f32" and (cin % 4 or cout % 4):
        pytest.skip("row bytes must be a multiple of 16")
    if dtype != "f32" and (cin % 8 or cout % 8):
        pytest.skip("row bytes must be a multiple of 16")
    coords = wl.shuffle_rows(wl.random_blob(1200, 14, 3, batches=2), seed=5)
    check_layer(coords, _layer("subm", 3, 1, cin, cout, dtype), algo="simt")
    check_layer(coords, _layer("spconv", 3, 2, cin, cout, dtype), algo="simt")


@pytest.mark.parametrize("cin,cout,K", [(16, 16, 3), (32, 32, 3), (16, 16, 5), (12, 20, 3), (4, 4, 1), (16, 64, 2)])
def test_fp32_weights_resident_kernel(cin, cout, K):
    """fp32 layers whose weights fit shared memory take the kernel that stages all of them once (more than 48 KB for
    32 -> 32, K = 3 and for K = 5): submanifold and strided maps, channel counts that do not divide a warp, every
    row checked at the fp32 tolerance, and the result must not depend on the neighbours of a block (ragged tail)."""
    coords = wl.shuffle_rows(wl.random_blob(2100, 15, 9, batches=2), seed=8)
    if K % 2 == 1:
        km, y = check_layer(coords, _layer("subm", K, 1, cin, cout, "f32"), algo="simt")
        _, y_auto = check_layer(coords, _layer("subm", K, 1, cin, cout, "f32"), km=km)
        assert torch.equal(y, y_auto)            # fp32 always runs on the CUDA-core path
    check_layer(coords, _layer("spconv", K, 2, cin, cout, "f32"), algo="simt")


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("cin", [16, 32, 64, 128])
@pytest.mark.parametrize("cout", [16, 32, 64, 128])
def test_tcgen05_kernel_all_channel_pairs(dtype, cin, cout):
    """Several tiles plus a ragged tail; submanifold and strided maps; dense-ish blob so most offsets are used."""
    coords = wl.shuffle_rows(wl.random_blob(2500, 16, 7, batches=2), seed=6)
    km, _ = check_layer(coords, _layer("subm", 3, 1, cin, cout, dtype), algo="tcgen05")
    assert km.n_out % 128 != 0
    check_layer(coords, _layer("spconv", 3, 2, cin, cout, dtype), algo="tcgen05")


@pytest.mark.parametrize("n", [1, 127, 128, 129, 300])
def test_tcgen05_tile_edges(n):
    coords = wl.random_blob(400, 9, 8)[:n]
    check_layer(coords, _layer("subm", 3, 1, 64, 64, "bf16"), algo="tcgen05")
    check_layer(coords, _layer("spconv", 2, 2, 32, 64, "f16"), algo="tcgen05")


def test_tcgen05_many_tiles_per_cta_and_multiple_rounds():
    """Cout = 128 keeps 4 tiles in TMEM; > 148*4 tiles forces a second round on every CTA."""
    coords = wl.shuffle_rows(wl.indoor_surfaces(3, target=100_000), seed=9)
    assert len(coords) > 148 * 4 * 128
    check_layer(coords, _layer("subm", 3, 1, 16, 128, "bf16"), algo="tcgen05", sample_rows=4000)


@pytest.mark.parametrize("cin,cout", [(16, 16), (32, 32), (32, 128), (64, 64), (64, 32)])
def test_tcgen05_steps_of_several_offsets(cin, cout):
    """Shapes whose steps take several offsets of a tile: one offset in all (K = 1), eight (K = 2), an odd count
    that leaves the last step short, dilation, a solid cube (tiles with all 27 offsets), and K = 5, whose 125
    offsets do not fit the step word and take the one-offset path."""
    blob = wl.shuffle_rows(wl.random_blob(3000, 20, 7), seed=5)
    check_layer(blob, _layer("subm", 1, 1, cin, cout, "bf16"), algo="tcgen05")
    check_layer(blob, _layer("spconv", 2, 2, cin, cout, "f16"), algo="tcgen05")
    check_layer(blob, _layer("subm", 3, 1, cin, cout, "bf16", d=2), algo="tcgen05")
    g = np.arange(12, dtype=np.int32)
    cube = np.stack(np.meshgrid(np.zeros(1, np.int32), g, g, g, indexing="ij"), axis=-1).reshape(-1, 4)
    check_layer(np.ascontiguousarray(cube), _layer("subm", 3, 1, cin, cout, "bf16"), algo="tcgen05")
    check_layer(blob[:600], _layer("subm", 5, 1, cin, cout, "bf16"), algo="tcgen05")


def test_tcgen05_sparse_isolated_voxels_only_centre_tap():
    coords = wl.config(1)["coords"]
    check_layer(coords, _layer("subm", 3, 1, 64, 64, "bf16"), algo="tcgen05")


def test_tcgen05_matches_simt_bitwise_inputs_same_rounding():
    """Both kernels accumulate in fp32 and round once: they may differ only by summation order."""
    coords = wl.shuffle_rows(wl.random_blob(3000, 18, 10), seed=2)
    lay = _layer("subm", 3, 1, 64, 64, "bf16")
    km, y_tc = check_layer(coords, lay, algo="tcgen05")
    _, y_simt = check_layer(coords, lay, algo="simt", km=km)
    diff = (y_tc.float() - y_simt.float()).abs().max().item()
    assert diff <= 2.0 ** -7 * y_simt.float().abs().max().item()


def test_config2_indoor_fp16():
    cfg = wl.config(2)
    check_layer(cfg["coords"], cfg["layers"][0])


def test_config3_lidar_bf16_full():
    cfg = wl.config(3)
    km, _ = check_layer(cfg["coords"], cfg["layers"][0])
    assert km.n_in == len(cfg["coords"])


def test_config4_strided_bf16_full():
    cfg = wl.config(4)
    for layer in cfg["layers"]:
        check_layer(cfg["coords"], layer)


def test_config5_encoder_stack_with_kmap_reuse():
    """Seven chained layers; each layer is checked in isolation (its input is the GPU's rounded output of
    the previous one) on sampled output rows; a submanifold map is reused for a second forward."""
    cfg = wl.config(5)
    coords = cfg["coords"]
    dtype = "bf16"
    x = to_device(wl.features(len(coords), 16, dtype, 0), dtype)
    for li, layer in enumerate(cfg["layers"]):
        subm = layer["kind"] == "subm"
        K, s, cin, cout = layer["kernel"], layer["stride"], layer["cin"], layer["cout"]
        km = gpu_kmap(coords, K, s, 1, subm)
        w_np = wl.weights(K ** 3, cin, cout, dtype, li)
        w = to_device(w_np, dtype)
        y = binding.spconv_forward(x, w, km)
        if subm:   # reuse: same map, second forward must reproduce the first bit for bit
            y2 = binding.spconv_forward(x, w, km)
            assert torch.equal(y, y2)
        torch.cuda.synchronize()
        assert binding.spconv_last_device_status(km) == 0
        oft = np.ascontiguousarray(km.nbr.cpu().numpy().T)
        rows = np.sort(np.random.default_rng(li).choice(len(oft), min(3000, len(oft)), replace=False))
        ref = oracle.forward(x.float().cpu().numpy(), w_np, oft[rows])
        err = rel_err(y[torch.from_numpy(rows).cuda()], ref)
        assert err <= TOL[dtype], (li, err)
        if not subm:
            coords = km.out_coords.cpu().numpy()
        x = y


def test_forward_argument_errors():
    coords = wl.random_blob(100, 8, 1)
    km = gpu_kmap(coords, 3)
    x = torch.zeros(len(coords), 24, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(27, 24, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SpconvError) as e:           # 24 channels: not a tensor-core shape
        binding.spconv_forward(x, w, km, algo="tcgen05")
    assert e.value.status == 1
    binding.spconv_forward(x, w, km)                          # auto falls to the CUDA-core kernel
    x4 = torch.zeros(len(coords), 4, dtype=torch.bfloat16, device="cuda")   # 8-byte rows
    w4 = torch.zeros(27, 4, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SpconvError):
        binding.spconv_forward(x4, w4, km)
    with pytest.raises(ValueError):
        binding.spconv_forward(x[:-1], w, km)


def test_layer_from_host_buffers():
    coords = wl.shuffle_rows(wl.random_blob(2000, 16, 4), seed=3)
    dtype = "bf16"
    x = wl.features(len(coords), 32, dtype, 1)
    w = wl.weights(27, 32, 64, dtype, 1)
    tx = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    tw = torch.from_numpy(w).to(torch.bfloat16).pin_memory()
    tc = torch.from_numpy(coords).pin_memory()
    cap = len(coords) * 2
    out = torch.empty(cap, 64, dtype=torch.bfloat16).pin_memory()
    oc = torch.empty(cap, 4, dtype=torch.int32).pin_memory()
    n_out = binding.spconv_layer_host(tc, tx, tw, 2, 1, 3, False, out, oc)
    ref_km = oracle.build_kmap(coords, 3, 2, 1, False)
    assert n_out == ref_km["n_out"]
    # map the GPU's output numbering onto the oracle's through the coordinates
    order_gpu = np.lexsort(tuple(oc[:n_out].numpy()[:, a] for a in (3, 2, 1, 0)))
    assert np.array_equal(oc[:n_out].numpy()[order_gpu], ref_km["out_coords"])
    ref = oracle.forward(x, w, ref_km["oft"])
    got = out[:n_out].float().numpy()[order_gpu].astype(np.float64)
    assert np.abs(got - ref).max() / np.abs(ref).max() <= TOL[dtype]
    small = torch.empty(1, 64, dtype=torch.bfloat16)
    with pytest.raises(binding.SpconvError) as e:
        binding.spconv_layer_host(tc, tx, tw, 2, 1, 3, False, small)
    assert e.value.status == 9


@pytest.mark.parametrize("kind,dtype,cin,cout", [("subm", "bf16", 64, 64), ("subm", "f16", 32, 128), ("subm", "f32", 16, 16),
                                                 ("spconv", "bf16", 64, 32)])
def test_layer_on_device_buffers_matches_build_then_forward(kind, dtype, cin, cout):
    """spconv_layer (for a submanifold layer the forward is enqueued before the host has the build's report) gives
    the oracle's result, the same kernel map as a separate build, and bit-identical rows to build + forward."""
    coords = wl.shuffle_rows(wl.random_blob(6000, 24, 5), seed=11)
    subm = kind == "subm"
    stride = 1 if subm else 2
    td = binding.DTYPE_BY_NAME[dtype]
    x = wl.features(len(coords), cin, dtype, 2)
    w = wl.weights(27, cin, cout, dtype, 2)
    tc, tx, tw = torch.from_numpy(coords).cuda(), torch.from_numpy(x).to(td).cuda(), torch.from_numpy(w).to(td).cuda()
    ref_km = oracle.build_kmap(coords, 3, stride, 1, subm)
    ref = oracle.forward(x, w, ref_km["oft"])
    out = None if subm else torch.zeros(len(coords) * 2, cout, dtype=td, device="cuda")
    for _ in range(3):                                   # repeated: scratch and handles are recycled between calls
        km, got = binding.spconv_layer(tc, tx, tw, stride, 1, 3, subm, out=out)
        torch.cuda.synchronize()
        assert km.n_out == ref_km["n_out"] and km.total_pairs == len(ref_km["pair_in"])
        oc = km.out_coords.cpu().numpy()
        order = np.lexsort(tuple(oc[:, a] for a in (3, 2, 1, 0))) if not subm else np.arange(km.n_out)
        assert np.array_equal(oc[order], ref_km["out_coords"])
        rows = got[:km.n_out].float().cpu().numpy()[order].astype(np.float64)
        assert np.abs(rows - ref).max() / np.abs(ref).max() <= TOL[dtype]
        km2 = binding.spconv_build_kmap(tc, stride, 1, 3, subm)
        assert torch.equal(km2.nbr, km.nbr) and torch.equal(km2.out_coords, km.out_coords)
        again = binding.spconv_forward(tx, tw, km2)
        assert torch.equal(again, got[:km.n_out])
        assert binding.spconv_last_device_status(km) == 0
        km.close(); km2.close()
    if subm:
        with pytest.raises(binding.SpconvError) as e:     # no room for n rows: refused before anything is enqueued
            binding.spconv_layer(tc, tx, tw, 1, 1, 3, True, out=torch.empty(10, cout, dtype=td, device="cuda"))
        assert e.value.status == 1
    else:
        with pytest.raises(binding.SpconvError) as e:
            binding.spconv_layer(tc, tx, tw, 2, 1, 3, False, out=torch.empty(10, cout, dtype=td, device="cuda"))
        assert e.value.status == 9
    km0, out0 = binding.spconv_layer(tc[:0], tx[:0], tw, 1, 1, 3, True)   # empty input
    assert km0.n_out == 0 and out0.shape[0] == 0


@pytest.mark.parametrize("max_ctas,cin,cout", [(1, 64, 64), (3, 64, 64), (1, 32, 128), (2, 128, 16)])
def test_tcgen05_many_tiles_per_cta_on_a_small_input(max_ctas, cin, cout):
    """The grid cap (a test hook read once per process, hence the child process) makes a small input exercise
    many tiles per CTA, several rounds and reuse of the TMEM accumulators."""
    import os
    import subprocess
    import sys
    code = f"""
import sys, numpy as np, torch
sys.path.insert(0, {os.path.dirname(os.path.dirname(os.path.abspath(__file__)))!r}); sys.path.insert(0, {os.path.dirname(os.path.abspath(__file__))!r})
from paper_2402_07710_b200 import workloads as wl
from gpu_util import check_layer
coords = wl.shuffle_rows(wl.random_blob(4000, 18, 3), seed=4)
lay = dict(kind="subm", kernel=3, stride=1, dilation=1, cin={cin}, cout={cout}, dtype="bf16")
km, _ = check_layer(coords, lay, algo="tcgen05")
assert km.n_tiles > 16
lay["kind"], lay["stride"] = "spconv", 2
check_layer(coords, lay, algo="tcgen05")
print("ok")
"""
    env = dict(os.environ, SPCONV_TC_MAX_CTAS=str(max_ctas))
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


@pytest.mark.gpu
def test_tile_plan_sort_paths_agree():
    """The two ways the tile plan sorts the rows -- grid-wide in one cooperative launch, and the library's radix sort
    (the switch is read once per process, hence the child processes) -- are stable sorts of the same keys, so they
    must cut the rows into identical tiles; every plan must hold every output row exactly once, pack a LiDAR sweep
    into few (tile, offset) blocks, and give the oracle's result."""
    import os
    import subprocess
    import sys
    import tempfile
    code = f"""
import sys, numpy as np, torch
sys.path.insert(0, {os.path.dirname(os.path.dirname(os.path.abspath(__file__)))!r}); sys.path.insert(0, {os.path.dirname(os.path.abspath(__file__))!r})
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import check_layer
coords = wl.shuffle_rows(wl.random_blob(9000, 26, 3), seed=7)
lay = dict(kind="subm", kernel=3, stride=1, dilation=1, cin=32, cout=32, dtype="f16")
km, _ = check_layer(coords, lay, algo="tcgen05")
rows = km.tile_rows.cpu().numpy().ravel()
live = np.sort(rows[rows >= 0])
assert np.array_equal(live, np.arange(km.n_out)), "every output row exactly once"
assert (rows < 0).sum() == rows.size - km.n_out and (rows[km.n_out:] < 0).all(), "only the padding of the last tile is negative"
lay["kind"], lay["stride"] = "spconv", 2
km2, _ = check_layer(coords, lay, algo="tcgen05")
sweep = wl.lidar_sweep(3)
km3, _ = check_layer(sweep, dict(kind="subm", kernel=3, stride=1, dilation=1, cin=64, cout=64, dtype="bf16"), algo="tcgen05", sample_rows=2000)
assert km3.tile_blocks < 12 * km3.n_tiles, (km3.tile_blocks, km3.n_tiles)    # input order: about 25 blocks per tile
np.savez(sys.argv[1], a=km.tile_rows.cpu().numpy(), b=km2.tile_rows.cpu().numpy(), c=km3.tile_rows.cpu().numpy())
print("ok")
"""
    plans = []
    for env in ({}, {"SPCONV_KMAP_LIBRARY_SORT": "1"}):
        with tempfile.NamedTemporaryFile(suffix=".npz", delete=False) as f:
            path = f.name
        res = subprocess.run([sys.executable, "-c", code, path], env=dict(os.environ, **env), capture_output=True, text=True, timeout=600)
        assert res.returncode == 0 and "ok" in res.stdout, str(env) + res.stdout[-2000:] + res.stderr[-2000:]
        with np.load(path) as z:
            plans.append({k: z[k] for k in z.files})
        os.unlink(path)
    for other in plans[1:]:
        for k in plans[0]:
            assert np.array_equal(plans[0][k], other[k]), k


@pytest.mark.gpu
def test_back_to_back_layers_and_graph_replay():
    """Two layers enqueued without any synchronisation between them, the second reading the first one's output:
    the forward is launched with programmatic dependent launch, so its set-up may overlap the kernel before it,
    and it must not touch its input before that kernel is complete.  The same pair captured in a CUDA graph and
    replayed must give the same bits."""
    coords = wl.shuffle_rows(wl.random_blob(20000, 40, 21), seed=3)
    n = len(coords)
    km = gpu_kmap(coords, 3, 1, 1, True)
    x = to_device(wl.features(n, 64, "bf16", 5), "bf16")
    w1 = to_device(wl.weights(27, 64, 64, "bf16", 6), "bf16")
    w2 = to_device(wl.weights(27, 64, 64, "bf16", 7), "bf16")
    y1 = torch.empty(n, 64, dtype=torch.bfloat16, device="cuda")
    y2 = torch.empty(n, 64, dtype=torch.bfloat16, device="cuda")
    binding.spconv_forward(x, w1, km, out=y1)       # warm-up: one-time set-up happens outside the capture
    torch.cuda.synchronize()
    for _ in range(3):                              # several pairs in a row, no synchronisation anywhere
        binding.spconv_forward(x, w1, km, out=y1)
        binding.spconv_forward(y1, w2, km, out=y2)
    torch.cuda.synchronize()
    assert binding.spconv_last_device_status(km) == 0
    oft = np.ascontiguousarray(km.nbr.cpu().numpy().T)
    ref1 = oracle.forward(wl.features(n, 64, "bf16", 5), wl.weights(27, 64, 64, "bf16", 6), oft)
    assert rel_err(y1, ref1) <= TOL["bf16"]
    y1_np = y1.float().cpu().numpy().astype(np.float64)          # the second layer sees the rounded output of the first
    ref2 = oracle.forward(y1_np, wl.weights(27, 64, 64, "bf16", 7), oft)
    assert rel_err(y2, ref2) <= TOL["bf16"]
    eager1, eager2 = y1.clone(), y2.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    y1.zero_(); y2.zero_()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        binding.spconv_forward(x, w1, km, out=y1)
        binding.spconv_forward(y1, w2, km, out=y2)
    torch.cuda.synchronize()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(y1, eager1) and torch.equal(y2, eager2)
