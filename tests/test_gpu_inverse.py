"""Inverse (transposed) sparse convolution on the GPU against the CPU oracle (Sec. III-E), through the C ABI.

The kernel map must equal the oracle's bit for bit (the fine rows keep their numbering and the coarse rows
theirs, so nothing is relabelled; pair lists are compared after sorting each offset's list), and the forward over
it must give the oracle's rows within the feature tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL, kmap_to_numpy, rel_err, to_device
from kmap_util import assert_kmaps_equal, canonical

pytestmark = pytest.mark.gpu


def _canon(d):
    return canonical(d["out_coords"], d["oft"], d["offset_start"], d["pair_in"], d["pair_out"], relabel_outputs=False)


def _check_inverse(fine, coarse, K, s, d, cin=None, cout=None, dtype="bf16", algo="auto", seed=0):
    tf, tc = torch.from_numpy(fine).cuda(), torch.from_numpy(coarse).cuda()
    km = binding.spconv_build_inverse_kmap(tf, tc, s, d, K)
    ref = oracle.build_inverse_kmap(fine, coarse, K, s, d)
    assert km.inverse == 1 and km.n_in == len(coarse) and km.n_out == len(fine) and km.kvol == K ** 3
    assert km.total_pairs == len(ref["pair_in"])
    if km.n_out == 0:
        return km
    got = kmap_to_numpy(km)
    assert np.array_equal(got["out_coords"], fine)
    assert np.array_equal(got["oft"], ref["oft"])
    assert_kmaps_equal(_canon(got), _canon(ref))
    tr = km.tile_rows.cpu().numpy().reshape(-1)
    assert np.array_equal(np.sort(tr[tr >= 0]), np.arange(km.n_out)) and (tr[km.n_out:] == -1).all()
    if cin is not None:
        x = wl.features(len(coarse), cin, dtype, seed)
        w = wl.weights(K ** 3, cin, cout, dtype, seed)
        y = binding.spconv_forward(to_device(x, dtype), to_device(w, dtype), km, algo=algo)
        torch.cuda.synchronize()
        assert binding.spconv_last_device_status(km) == 0
        want = oracle.forward(x, w, ref["oft"])
        err = rel_err(y, want)
        assert err <= TOL[dtype], f"relative max-abs error {err:.3e} ({dtype}, algo={algo})"
    return km


def _strided_outputs(fine, K, s, d):
    km = binding.spconv_build_kmap(torch.from_numpy(fine).cuda(), s, d, K, False)
    return km, km.out_coords.cpu().numpy()


@pytest.mark.parametrize("K,s,d", [(2, 2, 1), (3, 2, 1), (3, 1, 1), (3, 2, 2), (4, 2, 1), (3, 3, 1), (1, 1, 1), (5, 2, 1)])
def test_inverse_kmap_and_forward_on_blobs(K, s, d):
    fine = wl.shuffle_rows(wl.random_blob(3000, 22, seed=K * 10 + s, batches=2), seed=3)
    _, coarse = _strided_outputs(fine, K, s, d)          # the GPU's own output cells, in the GPU's order
    _check_inverse(fine, coarse, K, s, d, 32, 64, "f16", seed=1)
    _check_inverse(fine, coarse, K, s, d, 16, 16, "f32", seed=2)


@pytest.mark.parametrize("which,cin,cout", [(0, 128, 64), (1, 64, 64)], ids=["cfg4-k3s2", "cfg4-k2s2"])
def test_inverse_of_config4_maps_all_rows(which, cin, cout):
    """Up-sampling back onto the config-3 sweep from the cells of config 4's two strided layers, bf16, every row."""
    cfg = wl.config(4)
    fine, layer = cfg["coords"], cfg["layers"][which]
    K, s = layer["kernel"], layer["stride"]
    fwd, coarse = _strided_outputs(fine, K, s, 1)
    km = _check_inverse(fine, coarse, K, s, 1, cin, cout, "bf16", algo="tcgen05", seed=4)
    # the same relation as the strided map's with the roles swapped: (i, o, k) there <=> (o, i, k) here
    a, b = kmap_to_numpy(fwd), kmap_to_numpy(km)
    assert np.array_equal(a["offset_start"], b["offset_start"])
    for k in range(K ** 3):
        lo, hi = int(a["offset_start"][k]), int(a["offset_start"][k + 1])
        fa = set(zip(a["pair_in"][lo:hi].tolist(), a["pair_out"][lo:hi].tolist()))
        fb = set(zip(b["pair_out"][lo:hi].tolist(), b["pair_in"][lo:hi].tolist()))
        assert fa == fb


def test_inverse_adjoint_of_strided_forward_on_gpu():
    """<conv(x), y> = <x, inverse(y)> with transposed weight slices, both sides computed by the library in fp32."""
    fine = wl.shuffle_rows(wl.random_blob(2500, 20, seed=8), seed=2)
    fwd, coarse = _strided_outputs(fine, 3, 2, 1)
    inv = binding.spconv_build_inverse_kmap(torch.from_numpy(fine).cuda(), fwd.out_coords, 2, 1, 3)   # device pointer of the map itself
    rng = np.random.default_rng(0)
    x = torch.from_numpy(rng.standard_normal((len(fine), 16)).astype(np.float32)).cuda()
    y = torch.from_numpy(rng.standard_normal((len(coarse), 8)).astype(np.float32)).cuda()
    w = torch.from_numpy(rng.standard_normal((27, 16, 8)).astype(np.float32)).cuda()
    conv_x = binding.spconv_forward(x, w, fwd)
    inv_y = binding.spconv_forward(y, w.transpose(1, 2).contiguous(), inv)
    lhs, rhs = (conv_x.double() * y.double()).sum().item(), (x.double() * inv_y.double()).sum().item()
    assert abs(lhs - rhs) <= 1e-4 * max(1.0, abs(lhs))


def test_inverse_edge_cases_and_errors():
    E = binding.SpconvError
    fine = np.array([[0, 4, 4, 4], [0, 9, 9, 9], [1, 4, 4, 4]], np.int32)
    coarse = np.array([[0, 2, 2, 2]], np.int32)
    km = _check_inverse(fine, coarse, 2, 2, 1, 16, 16, "f32")           # two fine rows without a parent: zero rows
    y = binding.spconv_forward(torch.ones(1, 16, device="cuda"), torch.ones(8, 16, 16, device="cuda"), km)
    assert (y[1] == 0).all() and (y[2] == 0).all() and (y[0] == 16).all()
    empty = np.zeros((0, 4), np.int32)
    km0 = _check_inverse(empty, coarse, 2, 2, 1)
    assert km0.n_out == 0 and km0.total_pairs == 0
    km1 = _check_inverse(fine, empty, 2, 2, 1, 16, 16, "f32")           # no coarse rows at all
    assert km1.total_pairs == 0
    tf = torch.from_numpy(fine).cuda()
    dup = torch.tensor([[0, 2, 2, 2], [0, 2, 2, 2]], dtype=torch.int32, device="cuda")
    with pytest.raises(E) as e:
        binding.spconv_build_inverse_kmap(tf, dup, 2, 1, 2)
    assert e.value.status == 3
    bad = torch.tensor([[0, -1, 2, 2]], dtype=torch.int32, device="cuda")
    with pytest.raises(E) as e:
        binding.spconv_build_inverse_kmap(bad, torch.from_numpy(coarse).cuda(), 2, 1, 2)
    assert e.value.status == 2
    with pytest.raises(E) as e:
        binding.spconv_build_inverse_kmap(tf, torch.from_numpy(coarse).cuda(), 0, 1, 2)
    assert e.value.status == 1
    _check_inverse(fine, coarse, 2, 2, 1, 16, 16, "f32")                # the context still works
