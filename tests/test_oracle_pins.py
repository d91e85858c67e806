"""Pins for the CPU oracle: everything here is independent of the oracle's own code.

The oracle is checked against (a) the two worked figures the paper prints, (b) the closed
form of Eq. 1-5, (c) a dense 3-D convolution from a tensor library on tiny grids, (d) brute
force enumeration, and (e) invariants of the definition.  A dropped term, a flipped
orientation, a transposed weight slice or an off-by-one in the padding fails at least one.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import workloads as wl
from kmap_util import assert_kmaps_equal, brute_force_kmap, canonical, triples_of

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _sections(path):
    out, cur = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.isupper() and line.isalpha():
            cur = out.setdefault(line, [])
        else:
            cur.append(line.split())
    return out


def _canon(km, relabel=True):
    return canonical(km["out_coords"], km["oft"], km["offset_start"], km["pair_in"], km["pair_out"], relabel)


# ----------------------------------------------------------------------------- paper figures
def test_paper_2d_submanifold_example():
    """Figure "submanifold convolution on a 2D matrix": 24 printed entries match, the 25th is a known typo."""
    sec = _sections(os.path.join(GOLDEN, "subm_2d_example.txt"))
    I = np.array(sec["INPUT"], dtype=np.int64)
    K2 = np.array(sec["KERNEL"], dtype=np.float64)
    printed = np.array(sec["PRINTED"], dtype=np.float64)
    tr, tc, tv = (int(v) for v in sec["TYPO"][0])
    rows, cols = np.nonzero(I)
    coords = np.stack([np.zeros_like(rows), rows, cols, np.zeros_like(rows)], 1).astype(np.int32)
    km = oracle.build_kmap(coords, kernel=3, submanifold=True)
    w = np.zeros((27, 1, 1))
    for kx, ky in itertools.product(range(3), repeat=2):
        w[kx * 9 + ky * 3 + 1, 0, 0] = K2[kx, ky]        # the 2-D kernel sits in the kz = 1 slice
    y = oracle.forward(np.ones((len(coords), 1)), w, km["oft"])[:, 0]
    got = np.zeros((7, 7))
    got[rows, cols] = y
    interior = got[1:6, 1:6]
    expect = printed.copy()
    expect[tr, tc] = tv
    assert np.array_equal(interior, expect)
    assert printed[tr, tc] == 0 and (interior != printed).sum() == 1


def test_paper_oft_figure_orientation():
    """Figure "Result OFT": offset 0 is the (-1,-1) neighbour, the last offset the (+1,+1) one."""
    sec = _sections(os.path.join(GOLDEN, "oft_diagonal_trio.txt"))
    names = [p[0] for p in sec["POINTS"]]
    coords = np.array([[0, int(p[1]), int(p[2]), 0] for p in sec["POINTS"]], np.int32)
    km = oracle.build_kmap(coords, kernel=3, submanifold=True)
    for row in sec["OFT"]:
        j = names.index(row[0])
        for k2, sym in enumerate(row[1:]):
            kx, ky = divmod(k2, 3)
            got = km["oft"][j, kx * 9 + ky * 3 + 1]
            assert got == (-1 if sym == "-1" else names.index(sym)), (row[0], k2)
    # Nothing outside the z = 0 plane.
    mask = np.ones(27, bool)
    mask[[kx * 9 + ky * 3 + 1 for kx in range(3) for ky in range(3)]] = False
    assert (km["oft"][:, mask] == -1).all()


# ----------------------------------------------------------------------------- Eq. 1-5
@pytest.mark.parametrize("s", [2, 1])
def test_eq1_to_5_closed_form_kernel_equals_stride(s):
    """K == s with zero padding (K = 2 or 1 under pad = floor((K-1)/2)): each input lies in exactly
    one cell; o = floor(p/s), k = offX*K^2 + offY*K + offZ."""
    coords = wl.random_blob(400, 23, seed=s, batches=2)
    km = oracle.build_kmap(coords, kernel=s, stride=s, submanifold=False)
    p = coords[:, 1:].astype(np.int64)
    start = (p // s) * s                       # Eq. 2
    off = p - start                            # Eq. 3
    o = start // s                             # Eq. 4
    k = off[:, 0] * s * s + off[:, 1] * s + off[:, 2]   # Eq. 5
    cells = np.unique(np.concatenate([coords[:, :1].astype(np.int64), o], 1), axis=0)
    assert km["n_out"] == len(cells)
    assert np.array_equal(km["out_coords"], cells.astype(np.int32))
    assert km["offset_start"][-1] == len(coords)         # P = n
    index_of = {tuple(c): i for i, c in enumerate(cells.tolist())}
    want = {(i, index_of[(int(coords[i, 0]), *o[i].tolist())], int(k[i])) for i in range(len(coords))}
    assert triples_of(_canon(km)) == want


# ----------------------------------------------------------------------------- dense conv3d
def _dense_reference(coords, x, w, K, s, d, pad, grid):
    """torch conv3d in float64 on the densified input; dense axes (D,H,W) = (x,y,z)."""
    B = int(coords[:, 0].max()) + 1
    cin, cout = w.shape[1], w.shape[2]
    dense = torch.zeros(B, cin, *grid, dtype=torch.float64)
    c = torch.from_numpy(coords.astype(np.int64))
    dense[c[:, 0], :, c[:, 1], c[:, 2], c[:, 3]] = torch.from_numpy(x)
    wd = torch.from_numpy(w).reshape(K, K, K, cin, cout).permute(4, 3, 0, 1, 2).contiguous()
    return torch.nn.functional.conv3d(dense, wd, stride=s, padding=pad, dilation=d).numpy()


@pytest.mark.parametrize("K,d", [(3, 1), (3, 2), (5, 1), (1, 1)])
def test_submanifold_equals_masked_dense_conv(K, d):
    rng = np.random.default_rng(7)
    coords = wl.shuffle_rows(wl.random_blob(260, 9, seed=K * 10 + d, batches=2), seed=1)
    cin, cout = 3, 5
    x = rng.standard_normal((len(coords), cin))
    w = rng.standard_normal((K ** 3, cin, cout))
    km = oracle.build_kmap(coords, kernel=K, dilation=d, submanifold=True)
    y = oracle.forward(x, w, km["oft"])
    ref = _dense_reference(coords, x, w, K, 1, d, d * ((K - 1) // 2), (9, 9, 9))
    got = ref[coords[:, 0], :, coords[:, 1], coords[:, 2], coords[:, 3]]
    assert np.array_equal(km["out_coords"], coords)
    np.testing.assert_allclose(y, got, rtol=0, atol=1e-12)


@pytest.mark.parametrize("K,s,d", [(3, 2, 1), (2, 2, 1), (3, 1, 1), (3, 2, 2), (3, 3, 1), (4, 2, 1)])
def test_strided_equals_dense_conv_everywhere(K, s, d):
    """Scattering the sparse result into a dense grid reproduces conv3d at *every* cell.

    The dense grid is zero-extended on the high side so that every output cell the
    unbounded definition can touch exists in the dense result as well.
    """
    rng = np.random.default_rng(11)
    ext = 8
    coords = wl.shuffle_rows(wl.random_blob(120, ext, seed=K * 100 + s * 10 + d, batches=2), seed=2)
    cin, cout = 4, 3
    x = rng.standard_normal((len(coords), cin))
    w = rng.standard_normal((K ** 3, cin, cout))
    pad = d * ((K - 1) // 2)
    grid = (ext + 2 * d * K + s,) * 3
    km = oracle.build_kmap(coords, kernel=K, stride=s, dilation=d, submanifold=False)
    y = oracle.forward(x, w, km["oft"])
    ref = _dense_reference(coords, x, w, K, s, d, pad, grid)         # [B, cout, X, Y, Z]
    oc = km["out_coords"]
    assert (oc[:, 1:] < np.array(ref.shape[2:])).all()
    sparse = np.zeros_like(ref)
    sparse[oc[:, 0], :, oc[:, 1], oc[:, 2], oc[:, 3]] = y
    np.testing.assert_allclose(sparse, ref, rtol=0, atol=1e-12)
    # Generated cells == cells an all-ones kernel over the occupancy grid makes non-zero.
    occ = _dense_reference(coords, np.ones((len(coords), 1)), np.ones((K ** 3, 1, 1)), K, s, d, pad, grid)
    cells = np.argwhere(occ[:, 0] > 0).astype(np.int32)
    assert np.array_equal(cells, oc)


# ----------------------------------------------------------------------------- brute force
@pytest.mark.parametrize("K,s,d,subm", [(3, 1, 1, True), (3, 1, 2, True), (3, 2, 1, False), (2, 2, 1, False),
                                        (3, 1, 1, False), (5, 1, 1, True)])
def test_kmap_equals_brute_force(K, s, d, subm):
    coords = wl.shuffle_rows(wl.random_blob(90, 7, seed=5 + K + s, batches=2), seed=3)
    km = _canon(oracle.build_kmap(coords, kernel=K, stride=s, dilation=d, submanifold=subm))
    outs, triples = brute_force_kmap(coords, K, s, d, subm)
    assert np.array_equal(km["out_coords"], outs)
    assert triples_of(km) == triples
    # The table and the pair lists describe the same relation.
    from_table = {(int(km["nbr"][o, k]), o, k) for o, k in zip(*np.nonzero(km["nbr"] >= 0))}
    assert from_table == triples


# ----------------------------------------------------------------------------- invariants
def test_submanifold_invariants():
    coords = wl.uniform_voxels(1500, 20, seed=4)
    km = oracle.build_kmap(coords, kernel=3, submanifold=True)
    n, oft = len(coords), km["oft"]
    assert np.array_equal(oft[:, 13], np.arange(n))                       # centre tap = identity
    for k in range(27):                                                   # (i, j, k) <=> (j, i, 26 - k)
        j = np.nonzero(oft[:, k] >= 0)[0]
        assert np.array_equal(oft[oft[j, k], 26 - k], j)
        assert len(np.unique(oft[j, k])) == len(j)                        # injective per offset
    assert km["offset_start"][-1] == (oft >= 0).sum() <= 27 * n


def test_translation_invariance():
    coords = wl.random_blob(300, 12, seed=9)
    shift = np.array([0, 5, 2, 7], np.int32)
    a = oracle.build_kmap(coords, kernel=3, submanifold=True)
    b = oracle.build_kmap(coords + shift, kernel=3, submanifold=True)
    assert np.array_equal(a["oft"], b["oft"])
    # strided: translating inputs by s*t translates outputs by t and keeps the pairs
    s = 2
    a = _canon(oracle.build_kmap(coords, kernel=3, stride=s, submanifold=False))
    b = _canon(oracle.build_kmap(coords + s * shift, kernel=3, stride=s, submanifold=False))
    assert np.array_equal(a["out_coords"] + shift, b["out_coords"])
    assert np.array_equal(a["nbr"], b["nbr"])


def test_isolated_voxel_and_batch_separation():
    rng = np.random.default_rng(3)
    w = rng.standard_normal((27, 4, 6))
    x = rng.standard_normal((2, 4))
    # same spatial neighbourhood but different batch index: they must not pair
    coords = np.array([[0, 5, 5, 5], [1, 5, 5, 6]], np.int32)
    km = oracle.build_kmap(coords, kernel=3, submanifold=True)
    assert (km["oft"] >= 0).sum() == 2
    y = oracle.forward(x, w, km["oft"])
    np.testing.assert_allclose(y, x @ w[13], rtol=0, atol=1e-14)          # only the centre tap
    # strided K3 s2 pad1: output cell o covers input positions 2o-1, 2o, 2o+1 on each axis.
    # A lone voxel at an even position 4 lies only in cell 2 (through the centre offset) ...
    km = oracle.build_kmap(np.array([[0, 4, 4, 4]], np.int32), kernel=3, stride=2, submanifold=False)
    assert km["n_out"] == 1 and km["out_coords"].tolist() == [[0, 2, 2, 2]]
    assert np.nonzero(km["oft"][0] >= 0)[0].tolist() == [13]
    # ... and one at an odd position 3 lies in cells 1 (offset 2) and 2 (offset 0) per axis: 8 cells.
    km = oracle.build_kmap(np.array([[0, 3, 3, 3]], np.int32), kernel=3, stride=2, submanifold=False)
    assert km["n_out"] == 8
    assert km["out_coords"].tolist() == [[0, a, b, c] for a in (1, 2) for b in (1, 2) for c in (1, 2)]
    assert np.nonzero(km["oft"][0] >= 0)[0].tolist() == [26] and np.nonzero(km["oft"][7] >= 0)[0].tolist() == [0]
    y = oracle.forward(x[:1], w, km["oft"])
    for o in range(8):
        k = int(np.nonzero(km["oft"][o] >= 0)[0][0])
        np.testing.assert_allclose(y[o], x[0] @ w[k], rtol=0, atol=1e-14)


def test_zero_weight_offset_and_linearity():
    rng = np.random.default_rng(5)
    coords = wl.random_blob(200, 8, seed=2)
    km = oracle.build_kmap(coords, kernel=3, submanifold=True)
    x = rng.standard_normal((len(coords), 3))
    x2 = rng.standard_normal((len(coords), 3))
    w = rng.standard_normal((27, 3, 2))
    y = oracle.forward(x, w, km["oft"])
    for k in (0, 13, 20):
        wz = w.copy()
        wz[k] = 0
        rows = km["oft"][:, k]
        term = np.where((rows >= 0)[:, None], x[np.maximum(rows, 0)] @ w[k], 0.0)
        np.testing.assert_allclose(oracle.forward(x, wz, km["oft"]), y - term, rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.forward(2 * x + x2, w, km["oft"]),
                               2 * y + oracle.forward(x2, w, km["oft"]), rtol=0, atol=1e-12)


def test_weight_slice_is_cin_by_cout_not_transposed():
    """One voxel, one offset: y = x @ W_k with W_k [cin][cout] (a transposed read would fail: cin != cout)."""
    x = np.array([[1.0, 10.0, 100.0]])
    w = np.zeros((27, 3, 2))
    w[13] = np.array([[1, 2], [3, 4], [5, 6]], float)
    km = oracle.build_kmap(np.array([[0, 1, 1, 1]], np.int32), kernel=3, submanifold=True)
    assert oracle.forward(x, w, km["oft"]).tolist() == [[531.0, 642.0]]


def test_input_errors():
    with pytest.raises(oracle.OracleError) as e:
        oracle.build_kmap(np.array([[0, 1, 1, 1], [0, 1, 1, 1]], np.int32), kernel=3)
    assert e.value.code == 3
    with pytest.raises(oracle.OracleError) as e:
        oracle.build_kmap(np.array([[0, -1, 1, 1]], np.int32), kernel=3)
    assert e.value.code == 2
    for bad in (dict(kernel=2, submanifold=True), dict(kernel=3, stride=2, submanifold=True), dict(kernel=0)):
        with pytest.raises(oracle.OracleError) as e:
            oracle.build_kmap(np.array([[0, 1, 1, 1]], np.int32), **bad)
        assert e.value.code == 1
    km = oracle.build_kmap(np.zeros((0, 4), np.int32), kernel=3)
    assert km["n_out"] == 0 and km["offset_start"].tolist() == [0] * 28


def test_workload_generators_are_seeded_and_sized():
    a, b = wl.lidar_sweep(0), wl.lidar_sweep(0)
    assert np.array_equal(a, b) and not np.array_equal(a, wl.lidar_sweep(1)[: len(a)])
    assert 60_000 < len(a) < 160_000 and (a[:, 1:].max(0) < np.array(wl.LIDAR_GRID)).all() and a.min() >= 0
    assert len(np.unique(a, axis=0)) == len(a)
    c1 = wl.config(1)["coords"]
    assert c1.shape == (2000, 4) and c1[:, 1:].max() < 64
    x = wl.features(10, 16, "bf16", 0)
    assert np.array_equal(wl.from_storage_bits(wl.to_storage_bits(x, "bf16"), "bf16"), x)
    assert np.array_equal(torch.from_numpy(x).to(torch.bfloat16).float().numpy(), x)
    raw = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    assert np.array_equal(wl.round_to_dtype(raw, "bf16"), torch.from_numpy(raw).to(torch.bfloat16).float().numpy())


# ----------------------------------------------------------------------------- inverse convolution (Sec. III-E)
INVERSE_CASES = [(2, 2, 1), (3, 2, 1), (3, 1, 1), (3, 2, 2), (4, 2, 1), (3, 3, 1)]   # (K, s, d)


def _fine_and_coarse(K, s, d, seed, n=240, extent=11):
    fine = wl.shuffle_rows(wl.random_blob(n, extent, seed=seed, batches=2), seed=seed + 1)
    coarse = oracle.build_kmap(fine, K, s, d, False)["out_coords"]     # the cells the strided convolution generates
    coarse = wl.shuffle_rows(coarse, seed=seed + 2)                      # in an order of their own
    return fine, coarse


@pytest.mark.parametrize("K,s,d", INVERSE_CASES)
def test_inverse_equals_dense_conv_transpose_at_every_fine_cell(K, s, d):
    """The inverse convolution is the dense transposed convolution of the densified coarse features, read at the
    fine positions: library conv_transpose3d in float64, weight[ci][co][kx][ky][kz] = W[k][ci][co]."""
    rng = np.random.default_rng(100 + K * 7 + s * 3 + d)
    fine, coarse = _fine_and_coarse(K, s, d, seed=K * 100 + s * 10 + d)
    cin, cout = 3, 4
    x = rng.standard_normal((len(coarse), cin))
    w = rng.standard_normal((K ** 3, cin, cout))
    km = oracle.build_inverse_kmap(fine, coarse, K, s, d)
    assert km["n_in"] == len(coarse) and km["n_out"] == len(fine)
    assert np.array_equal(km["out_coords"], fine)
    y = oracle.forward(x, w, km["oft"])
    pad = d * ((K - 1) // 2)
    B = int(max(fine[:, 0].max(), coarse[:, 0].max())) + 1
    grid = tuple(int(coarse[:, a].max()) + 1 for a in (1, 2, 3))
    dense = torch.zeros(B, cin, *grid, dtype=torch.float64)
    c = torch.from_numpy(coarse.astype(np.int64))
    dense[c[:, 0], :, c[:, 1], c[:, 2], c[:, 3]] = torch.from_numpy(x)
    wd = torch.from_numpy(w).reshape(K, K, K, cin, cout).permute(3, 4, 0, 1, 2).contiguous()
    up = torch.nn.functional.conv_transpose3d(dense, wd, stride=s, padding=pad, dilation=d, output_padding=s - 1 if s > 1 else 0).numpy()
    for j, (b, px, py, pz) in enumerate(fine.tolist()):
        inside = px < up.shape[2] and py < up.shape[3] and pz < up.shape[4]
        want = up[b, :, px, py, pz] if inside else np.zeros(cout)
        assert np.allclose(y[j], want, rtol=0, atol=1e-12), (j, fine[j])


@pytest.mark.parametrize("K,s,d", INVERSE_CASES)
def test_inverse_is_the_adjoint_of_the_strided_convolution(K, s, d):
    """<conv(x), y> = <x, inverse(y)> when the inverse layer uses the transposed weight slices: the defining
    property of a transposed convolution, checked without looking at either kernel map."""
    rng = np.random.default_rng(K * 31 + s * 5 + d)
    fine, _ = _fine_and_coarse(K, s, d, seed=K * 50 + s * 9 + d)
    fwd = oracle.build_kmap(fine, K, s, d, False)
    coarse = fwd["out_coords"]
    cf, cc = 3, 2
    w = rng.standard_normal((K ** 3, cf, cc))
    x = rng.standard_normal((len(fine), cf))
    y = rng.standard_normal((len(coarse), cc))
    conv_x = oracle.forward(x, w, fwd["oft"])                                  # [n_coarse, cc]
    inv = oracle.build_inverse_kmap(fine, coarse, K, s, d)
    inv_y = oracle.forward(y, np.ascontiguousarray(w.transpose(0, 2, 1)), inv["oft"])   # [n_fine, cf]
    assert abs((conv_x * y).sum() - (x * inv_y).sum()) <= 1e-10 * max(1.0, abs((conv_x * y).sum()))


@pytest.mark.parametrize("K,s,d", INVERSE_CASES)
def test_inverse_kmap_brute_force_and_role_swap(K, s, d):
    """Brute force over all (fine, coarse, offset) triples with explicit coordinate comparison; and the same
    relation as the strided convolution's with the roles of the two sets swapped."""
    fine, coarse = _fine_and_coarse(K, s, d, seed=K * 13 + s + d, n=90, extent=8)
    pad = d * ((K - 1) // 2)
    inv = oracle.build_inverse_kmap(fine, coarse, K, s, d)
    want = set()
    for j, (fb, fx, fy, fz) in enumerate(fine.tolist()):
        for q, (cb, cx, cy, cz) in enumerate(coarse.tolist()):
            for k, (kx, ky, kz) in enumerate(itertools.product(range(K), repeat=3)):
                if fb == cb and fx == cx * s + d * kx - pad and fy == cy * s + d * ky - pad and fz == cz * s + d * kz - pad:
                    want.add((q, j, k))
    got = triples_of(_canon(inv, relabel=False))
    assert got == want
    from_table = {(int(inv["oft"][j, k]), j, k) for j in range(len(fine)) for k in range(K ** 3) if inv["oft"][j, k] >= 0}
    assert from_table == want
    # role swap: (i_fine, o_coarse, k) of the strided map <=> (o_coarse, i_fine, k) here
    fwd = oracle.build_kmap(fine, K, s, d, False)
    index_of = {tuple(c): i for i, c in enumerate(coarse.tolist())}
    relabel = [index_of[tuple(c)] for c in fwd["out_coords"].tolist()]
    swapped = {(relabel[o], i, k) for (i, o, k) in triples_of(_canon(fwd, relabel=False))}
    assert swapped == want


@pytest.mark.parametrize("s", [2, 1])
def test_inverse_kernel_equals_stride_is_one_pair_per_fine_position(s):
    """K == s with zero padding (K = 2 or 1 under pad = floor((K-1)/2)): Eq. 1-5 give every fine position exactly
    one coarse parent floor(p/s) and the offset p mod s, so each output row is a single weight-feature product,
    as Sec. III-E says."""
    fine, coarse = _fine_and_coarse(s, s, 1, seed=77)
    inv = oracle.build_inverse_kmap(fine, coarse, s, s, 1)
    assert (np.sum(inv["oft"] >= 0, axis=1) == 1).all() and inv["offset_start"][-1] == len(fine)
    index_of = {tuple(c): i for i, c in enumerate(coarse.tolist())}
    p = fine[:, 1:].astype(np.int64)
    off = p - (p // s) * s
    k = off[:, 0] * s * s + off[:, 1] * s + off[:, 2]
    for j in range(len(fine)):
        parent = index_of[(int(fine[j, 0]), *(p[j] // s).tolist())]
        assert inv["oft"][j, k[j]] == parent
    rng = np.random.default_rng(5)
    x = rng.standard_normal((len(coarse), 2)); w = rng.standard_normal((s ** 3, 2, 3))
    y = oracle.forward(x, w, inv["oft"])
    for j in range(len(fine)):
        assert np.allclose(y[j], x[inv["oft"][j, k[j]]] @ w[k[j]], rtol=0, atol=1e-13)


def test_inverse_missing_parent_gives_zero_row_and_errors():
    fine = np.array([[0, 4, 4, 4], [0, 9, 9, 9]], np.int32)
    coarse = np.array([[0, 2, 2, 2]], np.int32)                 # the parent of the first position only
    inv = oracle.build_inverse_kmap(fine, coarse, 2, 2, 1)
    assert inv["oft"][0].tolist().count(-1) == 7 and inv["oft"][0, 0] == 0 and (inv["oft"][1] == -1).all()
    y = oracle.forward(np.ones((1, 2)), np.ones((8, 2, 2)), inv["oft"])
    assert (y[1] == 0).all() and (y[0] == 2).all()
    with pytest.raises(oracle.OracleError):
        oracle.build_inverse_kmap(np.array([[0, 1, 1, 1], [0, 1, 1, 1]], np.int32), coarse, 2, 2, 1)
    with pytest.raises(oracle.OracleError):
        oracle.build_inverse_kmap(fine, np.array([[0, -1, 0, 0]], np.int32), 2, 2, 1)


# ----------------------------------------------------------------------------- voxelisation of raw points
def test_voxelize_hand_example():
    """Five points, voxel size 0.5 from origin (-1, -1, 0) on a 4 x 4 x 2 grid, worked by hand: two points share cell
    (2, 2, 0) (their mean is the voxel's feature), one lies exactly on a cell boundary (it belongs to the upper
    cell), one is outside the grid (dropped), cells are numbered by first appearance."""
    pts = np.array([[0.10, 0.20, 0.30, 1.0, 10.0],     # cell (2, 2, 0)
                    [-0.75, 0.90, 0.99, 2.0, 20.0],    # cell (0, 3, 1)
                    [0.40, 0.49, 0.10, 3.0, 30.0],     # cell (2, 2, 0) again
                    [0.00, -1.00, 0.50, 4.0, 40.0],    # exactly on boundaries: cell (2, 0, 1)
                    [1.00, 0.00, 0.00, 5.0, 50.0]],    # x cell 4: outside
                   np.float32)
    r = oracle.voxelize(pts, 2, 7, (-1.0, -1.0, 0.0), (0.5, 0.5, 0.5), (4, 4, 2))
    assert r["coords"].tolist() == [[7, 2, 2, 0], [7, 0, 3, 1], [7, 2, 0, 1]]
    assert r["counts"].tolist() == [2, 1, 1]
    assert np.allclose(r["feats"], [[2.0, 20.0], [2.0, 20.0], [4.0, 40.0]])
    assert r["voxel_of_point"].tolist() == [0, 1, 0, 2, -1]


def test_voxelize_agrees_with_the_workload_generator_and_library_routines():
    """On the LiDAR returns the set of voxels equals what the workload generator builds with array operations
    (unique rows of the floored positions, here in float32), counts sum to the points inside the grid, every
    voxel's mean lies between its points' extremes, and a permutation of the points permutes the numbering only."""
    pts = wl.lidar_points(5, n_feat=2)[:6000]
    o, v, g = wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID
    r = oracle.voxelize(pts, 2, 0, o, v, g)
    cells = np.floor((pts[:, :3] - np.asarray(o, np.float32)) / np.asarray(v, np.float32)).astype(np.int64)
    inside = ((cells >= 0) & (cells < np.asarray(g))).all(axis=1)
    uniq, first, inv, cnt = np.unique(cells[inside], axis=0, return_index=True, return_inverse=True, return_counts=True)
    order = np.argsort(first, kind="stable")                      # first appearance
    assert np.array_equal(r["coords"][:, 1:], uniq[order])
    assert np.array_equal(r["counts"], cnt[order]) and r["counts"].sum() == inside.sum()
    sums = np.zeros((len(uniq), 2)); np.add.at(sums, inv.ravel(), pts[inside, 3:5].astype(np.float64))
    assert np.allclose(r["feats"], (sums / cnt[:, None])[order], rtol=0, atol=1e-12)
    perm = np.random.default_rng(1).permutation(len(pts))
    r2 = oracle.voxelize(pts[perm], 2, 0, o, v, g)
    a = {tuple(c): (f.round(12).tolist(), int(k)) for c, f, k in zip(r["coords"].tolist(), r["feats"], r["counts"])}
    b = {tuple(c): (f.round(12).tolist(), int(k)) for c, f, k in zip(r2["coords"].tolist(), r2["feats"], r2["counts"])}
    assert a.keys() == b.keys() and all(a[k][1] == b[k][1] and np.allclose(a[k][0], b[k][0], atol=1e-9) for k in a)
