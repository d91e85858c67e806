"""The calls the benchmark times, at the benchmark's sizes, against the CPU oracle on ALL output rows.

``spconv_layer`` enqueues the forward before the host has the build's report (submanifold layers) and writes the
pair lists on a second stream; ``spconv_layer_host`` overlaps the uploads with the build.  Both orderings only
show at sizes where every SM has several tiles, so they are checked here on the LiDAR-sized workloads
(config 3 and config 4), three calls in a row, every row compared (Algorithm 2 in fp64 on the oracle's side).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL

pytestmark = pytest.mark.gpu


def _lex(c):
    return np.lexsort((c[:, 3], c[:, 2], c[:, 1], c[:, 0]))


def _reference(coords, layer, seed):
    subm = layer["kind"] == "subm"
    K, s = layer["kernel"], layer["stride"]
    x = wl.features(len(coords), layer["cin"], layer["dtype"], seed)
    w = wl.weights(K ** 3, layer["cin"], layer["cout"], layer["dtype"], seed)
    ref_km = oracle.build_kmap(coords, K, s, 1, subm)
    return x, w, ref_km, oracle.forward(x, w, ref_km["oft"])


def _check_rows(out_rows, out_coords, ref_km, ref, dtype, subm):
    """GPU rows (any output numbering) against the oracle's rows (lexicographic numbering)."""
    order = np.arange(len(out_coords)) if subm else _lex(out_coords)
    assert np.array_equal(out_coords[order], ref_km["out_coords"])
    got = out_rows.astype(np.float64)[order]
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= TOL[dtype], f"relative max-abs error {err:.3e} on {len(ref)} rows"
    return err


@pytest.mark.parametrize("index,which", [(3, 0), (4, 0), (4, 1)], ids=["cfg3-subm3-64-64", "cfg4-k3s2-64-128", "cfg4-k2s2-64-64"])
def test_spconv_layer_full_size_all_rows(index, which):
    cfg = wl.config(index)
    coords, layer = cfg["coords"], cfg["layers"][which]
    subm = layer["kind"] == "subm"
    dtype = layer["dtype"]
    td = binding.DTYPE_BY_NAME[dtype]
    x, w, ref_km, ref = _reference(coords, layer, seed=index)
    if subm:   # submanifold outputs keep the input numbering on both sides
        assert np.array_equal(coords, ref_km["out_coords"])
    tc, tx, tw = torch.from_numpy(coords).cuda(), torch.from_numpy(x).to(td).cuda(), torch.from_numpy(w).to(td).cuda()
    cap = len(coords) if subm else 2 * len(coords)
    out = torch.empty(cap, layer["cout"], dtype=td, device="cuda")
    first = None
    for call in range(3):
        out.fill_(float("nan"))
        km, got = binding.spconv_layer(tc, tx, tw, layer["stride"], 1, layer["kernel"], subm, out=out)
        torch.cuda.synchronize()
        assert binding.spconv_last_device_status(km) == 0
        assert km.n_out == ref_km["n_out"] and km.total_pairs == len(ref_km["pair_in"])
        rows = got[:km.n_out].float().cpu().numpy()
        oc = km.out_coords.cpu().numpy()
        _check_rows(rows, oc, ref_km, ref, dtype, subm)
        if first is None:
            first = got[:km.n_out].clone()
        else:
            assert torch.equal(first, got[:km.n_out]), "the same call gives the same bits"
        km.close()


def test_spconv_layer_host_config3_all_rows():
    cfg = wl.config(3)
    coords, layer = cfg["coords"], cfg["layers"][0]
    dtype = layer["dtype"]
    x, w, ref_km, ref = _reference(coords, layer, seed=7)
    hc = torch.from_numpy(coords).pin_memory()
    hx = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    hw = torch.from_numpy(w).to(torch.bfloat16).pin_memory()
    ho = torch.empty(len(coords), layer["cout"], dtype=torch.bfloat16).pin_memory()
    hoc = torch.empty(len(coords), 4, dtype=torch.int32).pin_memory()
    for call in range(3):
        ho.fill_(float("nan")); hoc.fill_(-1)
        n_out = binding.spconv_layer_host(hc, hx, hw, 1, 1, 3, True, ho, hoc)
        assert n_out == len(coords)
        assert np.array_equal(hoc.numpy(), coords)
        _check_rows(ho.float().numpy(), hoc.numpy(), ref_km, ref, dtype, True)
