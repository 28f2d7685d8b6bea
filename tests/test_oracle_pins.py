"""Pins for the CPU oracle: every check here compares the oracle with
something that is not the oracle -- the paper's worked example, brute force
on tiny inputs, closed forms, and library routines on the special cases where
the method reduces to them."""
import itertools
import os
import struct

import numpy as np
import pytest

import oracle
import ubp_synth
from conftest import GOLDEN, parse_golden


# ---------------------------------------------------------------- helpers
def blob_sections(blob):
    """Independent reader of the canonical layout (header 64 B, sections 64-B aligned)."""
    assert blob[:4] == b"UBP1"
    ver, M, C, R, Nb, m, flags = struct.unpack_from("<I5iI", blob, 4)
    assert ver == 1 and flags == 1
    up = lambda x: (x + 63) // 64 * 64
    o1 = 64
    o2 = o1 + up(4 * (M + 1))
    o3 = o2 + up(4 * m)
    end = o3 + up(4 * m * Nb * R)
    assert len(blob) == end
    indptr = np.frombuffer(blob, "<i4", M + 1, o1)
    indices = np.frombuffer(blob, "<i4", m, o2)
    values = np.frombuffer(blob, "<f4", m * Nb * R, o3).reshape(m, Nb, R)
    # padding bytes are zero
    pad = bytes(blob[32:64]) + bytes(blob[o1 + 4 * (M + 1):o2]) + bytes(blob[o2 + 4 * m:o3]) + \
        bytes(blob[o3 + 4 * m * Nb * R:end])
    assert pad.count(0) == len(pad)
    return dict(M=M, C=C, R=R, Nb=Nb, m=m, indptr=indptr, indices=indices, values=values)


def all_placements(M, Nb):
    """Every set of non-overlapping block start rows in one column of M rows."""
    out = [[]]
    def rec(first, cur):
        for i in range(first, M - Nb + 1):
            nxt = cur + [i]
            out.append(nxt)
            rec(i + Nb, nxt)
    rec(0, [])
    return out


def scatter_reference(M, C, Nb, starts, W, X, bias=None, relu=False):
    """Scalar per-block scatter with Python integers/floats: the sum the
    block-sparse product means, written block by block."""
    Nc = X.shape[1]
    Y = [[0] * Nc for _ in range(M)]
    for j in range(C):
        for i in starts[j]:
            for t in range(Nb):
                w = W[i + t][j]
                for n in range(Nc):
                    Y[i + t][n] += w * X[j][n]
    if bias is not None:
        for o in range(M):
            for n in range(Nc):
                Y[o][n] += bias[o]
    if relu:
        Y = [[max(v, 0) for v in row] for row in Y]
    return np.array(Y, dtype=np.float64)


# ---------------------------------------------------------------- worked example
def load_worked_example():
    g = parse_golden(os.path.join(GOLDEN, "wros_worked_example.txt"))
    N, M, C = int(g["N"][0]), int(g["M"][0]), int(g["C"][0])
    let = dict((kv.split("=")[0], int(kv.split("=")[1])) for kv in g["letters"][0].split())
    W = np.zeros((M, C), np.float32)
    mask = np.zeros((M, C), np.uint8)
    for b in g["block"]:
        pos, ws = b.split("=")
        i, j = (int(v) for v in pos.split(","))
        for t, name in enumerate(ws.split(",")):
            W[i + t, j] = let[name]
            mask[i + t, j] = 1
    X = np.array([[int(v) for v in g[f"x{c}"][0].split()] for c in range(C)], np.float32)
    return g, N, M, C, let, W, mask, X


def eval_expr(expr, let, X):
    tot = np.zeros(X.shape[1])
    for term in expr.split("+"):
        w, x = term.strip().split("*")
        tot += let[w] * X[int(x[1:])]
    return tot


def test_worked_example_format():
    g, N, M, C, let, W, mask, X = load_worked_example()
    blob = oracle.pack(W, mask, N)
    s = blob_sections(blob)
    assert list(s["indptr"]) == [int(v) for v in g["indptr"][0].split()]
    assert list(s["indices"]) == [int(v) for v in g["indices"][0].split()]
    want = [[let[n] for n in grp.split()] for grp in g["values"][0].split("|")]
    assert s["values"][:, :, 0].tolist() == want
    # the weight D (output row 1) sits in slot 1 of the block that starts at row 1
    b_tile1 = s["indptr"][1]
    assert s["values"][b_tile1, 1, 0] == let["D"]


def test_worked_example_outputs():
    g, N, M, C, let, W, mask, X = load_worked_example()
    want = np.stack([eval_expr(g[f"O{o}"][0], let, X) for o in range(M)])
    Y, A = oracle.masked_matmul(W, mask, X)
    assert np.array_equal(Y, want)
    blob = oracle.pack(W, mask, N)
    for tw in (1, 3, 4, 7):
        assert np.array_equal(oracle.wros_spmm(blob, X, tile_w=tw), want)
    # unused channel 1 must not leak in
    X2 = X.copy(); X2[1] = 1000
    assert np.array_equal(oracle.masked_matmul(W, mask, X2)[0], want)


# ---------------------------------------------------------------- block budget
@pytest.mark.parametrize("M,C,p,Nb,want", [
    (64, 64, 50, 4, 512), (512, 512, 70, 4, 19660), (256, 256, 80, 8, 1638),
    (2048, 2048, 50, 2, 1048576), (2048, 2048, 90, 16, 26214), (64, 32, 80, 4, 102),
    (1024, 1024, 80, 4, 52428),
])
def test_block_budget_closed_form(M, C, p, Nb, want):
    # m = floor(b (1-p) / N), Section 3.1; values worked out by hand
    assert oracle.block_budget(M, C, p, Nb) == want
    import math
    from fractions import Fraction
    assert want == math.floor(Fraction(M * C) * (1 - Fraction(p, 100)) / Nb)
    assert ubp_synth.block_budget(M, C, p, Nb) == want


# ---------------------------------------------------------------- decode: Algorithm 2
def division_reference(expanded_starts, N):
    """Algorithm 2 as printed: sorted index list in, final block starts out."""
    out, next_idx = [], 0
    for k in sorted(expanded_starts):
        if next_idx > k:
            out.append(next_idx); next_idx += N
        else:
            out.append(k); next_idx = k + N
    return out


def test_decode_brute_force_single_column():
    for M, Nb in [(6, 1), (6, 2), (7, 3), (9, 4), (5, 5)]:
        for starts in all_placements(M, Nb):
            mask = np.zeros((M, 1), np.uint8)
            for i in starts:
                mask[i:i + Nb, 0] = 1
            bi, bj = oracle.decode_mask(mask, Nb)
            # adjacent blocks merge into one run; any cut of that run from its top is the same set
            assert list(bi) == starts and not bj.any()


def test_decode_matches_block_division_on_expanded_runs():
    # a run of 2N ones can come from an expanded selection {k, k+1}: Algorithm 2 re-cuts it from its top
    N, M = 3, 12
    mask = np.zeros((M, 2), np.uint8)
    mask[2:8, 0] = 1            # run of 6 starting at row 2 in column 0
    mask[0:3, 1] = 1; mask[9:12, 1] = 1
    bi, bj = oracle.decode_mask(mask, N)
    k = sorted(int(i) + M * int(j) for i, j in zip(bi, bj))
    assert k == division_reference([2, 3, M + 0, M + 9], N) == [2, 5, 12, 21]


@pytest.mark.parametrize("bad", ["short_run", "hole", "edge", "value"])
def test_decode_rejects_illegal_masks(bad):
    M, Nb = 8, 3
    mask = np.zeros((M, 2), np.uint8)
    if bad == "short_run":
        mask[1:5, 0] = 1                       # run of 4, not a multiple of 3
        code = oracle.E_RAGGED
    elif bad == "hole":
        mask[1:3, 1] = 1                       # run of 2
        code = oracle.E_RAGGED
    elif bad == "edge":
        mask[6:8, 0] = 1                       # would run past the last output channel (Eq. 1)
        code = oracle.E_RAGGED
    else:
        mask[0:3, 0] = 1; mask[1, 0] = 2
        code = oracle.E_ARG
    with pytest.raises(oracle.OracleError) as e:
        oracle.decode_mask(mask, Nb)
    assert e.value.code == code


def test_nb_larger_than_m_is_an_error():
    with pytest.raises(oracle.OracleError):
        oracle.decode_mask(np.zeros((3, 3), np.uint8), 4)


# ---------------------------------------------------------------- product: brute force
def test_product_brute_force_all_placements():
    """All legal placements for small shapes, integer data: exact equality of
    the definition, the paper's walk, and a scalar block-by-block scatter."""
    rng = np.random.default_rng(7)
    n_checked = 0
    for M, C, Nb in [(4, 2, 1), (5, 2, 2), (6, 2, 3), (6, 1, 2), (4, 3, 2), (7, 2, 2)]:
        cols = all_placements(M, Nb)
        for combo in itertools.product(cols, repeat=C):
            W = rng.integers(-9, 10, size=(M, C)).astype(np.float32)
            X = rng.integers(-9, 10, size=(C, 5)).astype(np.float32)
            bias = rng.integers(-5, 6, size=M).astype(np.float32)
            mask = ubp_synth.mask_from_starts(M, C, Nb, [np.array(s, np.int64) for s in combo])
            want = scatter_reference(M, C, Nb, combo, W.tolist(), X, bias.tolist(), relu=True)
            Y, A = oracle.masked_matmul(W, mask, X, bias, relu=True)
            assert np.array_equal(Y, want)
            Yw = oracle.wros_spmm(oracle.pack(W, mask, Nb), X, bias, relu=True, tile_w=4)
            assert np.array_equal(Yw, want)
            n_checked += 1
    assert n_checked > 900


# ---------------------------------------------------------------- product: library special cases
def test_dense_case_is_plain_matmul():
    import torch
    rng = np.random.default_rng(11)
    M, C, Nc, Nb = 24, 17, 33, 4          # p = 0 and Nb | M: every weight kept
    W = rng.standard_normal((M, C)).astype(np.float32)
    X = rng.standard_normal((C, Nc)).astype(np.float32)
    b = rng.standard_normal(M).astype(np.float32)
    mask = np.ones((M, C), np.uint8)
    Y, A = oracle.masked_matmul(W, mask, X, b, relu=False)
    want = (torch.from_numpy(W).double() @ torch.from_numpy(X).double() + torch.from_numpy(b).double()[:, None]).numpy()
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-13)
    wantA = (torch.from_numpy(W).double().abs() @ torch.from_numpy(X).double().abs()).numpy() + np.abs(b.astype(np.float64))[:, None]
    np.testing.assert_allclose(A, wantA, rtol=1e-13)
    assert len(oracle.decode_mask(mask, Nb)[0]) == M * C // Nb
    np.testing.assert_allclose(oracle.wros_spmm(oracle.pack(W, mask, Nb), X, b), want, rtol=0, atol=1e-13)


def test_nb1_is_csr_spmm():
    import scipy.sparse as sp
    rng = np.random.default_rng(12)
    M, C, Nc = 40, 23, 19
    mask, _ = ubp_synth.random_mask(M, C, 1, 75, seed=3)
    W = rng.standard_normal((M, C)).astype(np.float32)
    X = rng.standard_normal((C, Nc)).astype(np.float32)
    csr = sp.csr_matrix((W * mask).astype(np.float64))
    want = csr @ X.astype(np.float64)
    Y, _ = oracle.masked_matmul(W, mask, X)
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-13)
    # with Nb = 1 the packed form *is* CSR: indptr over rows, indices = columns, values in order
    s = blob_sections(oracle.pack(W, mask, 1))
    assert np.array_equal(s["indptr"], csr.indptr) and np.array_equal(s["indices"], csr.indices)
    assert np.array_equal(s["values"].ravel(), csr.data.astype(np.float32))


def test_aligned_blocks_are_block_sparse_rows():
    # starts restricted to multiples of N (the aligned pattern): the result is a block-CSR product
    import scipy.sparse as sp
    rng = np.random.default_rng(13)
    M, C, Nb, Nc = 32, 12, 4, 9
    mask, starts = ubp_synth.random_mask(M, C, Nb, 60, seed=5, aligned=True)
    assert all((s % Nb == 0).all() for s in starts)
    W = rng.standard_normal((M, C)).astype(np.float32)
    X = rng.standard_normal((C, Nc)).astype(np.float32)
    bsr = sp.bsr_matrix((W * mask).astype(np.float64), blocksize=(Nb, 1))
    Y, _ = oracle.masked_matmul(W, mask, X)
    np.testing.assert_allclose(Y, bsr @ X.astype(np.float64), rtol=0, atol=1e-13)
    s = blob_sections(oracle.pack(W, mask, Nb))
    # only aligned start rows own blocks
    counts = np.diff(s["indptr"])
    assert counts[np.arange(M) % Nb != 0].sum() == 0


def test_conv3x3_is_library_conv():
    import torch
    import torch.nn.functional as F
    rng = np.random.default_rng(14)
    M, C, Nb, B, H, Wd = 16, 6, 4, 3, 5, 7
    mask, _ = ubp_synth.random_mask(M, C, Nb, 50, seed=9)
    W = rng.standard_normal((M, C, 9)).astype(np.float32)
    In = rng.standard_normal((C, B, H, Wd)).astype(np.float32)
    b = rng.standard_normal(M).astype(np.float32)
    Y, A = oracle.masked_conv3x3(W, mask, In, b, relu=True)
    Wm = torch.from_numpy(W * mask[:, :, None]).double().reshape(M, C, 3, 3)
    x = torch.from_numpy(In).double().permute(1, 0, 2, 3)           # NCHW
    want = F.relu(F.conv2d(x, Wm, torch.from_numpy(b).double(), padding=1)).permute(1, 0, 2, 3).numpy()
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-12)
    wantA = F.conv2d(x.abs(), Wm.abs(), torch.from_numpy(b).double().abs(), padding=1).permute(1, 0, 2, 3).numpy()
    np.testing.assert_allclose(A, wantA, rtol=1e-12)
    # asymmetric taps: a delta input returns the flipped kernel around it (cross-correlation)
    In0 = np.zeros((C, 1, 5, 5), np.float32); In0[2, 0, 2, 2] = 1
    Y0, _ = oracle.masked_conv3x3(W, mask, In0)
    for o in range(M):
        want0 = (W[o, 2] * mask[o, 2]).reshape(3, 3)[::-1, ::-1]
        np.testing.assert_array_equal(Y0[o, 0, 1:4, 1:4], want0.astype(np.float64))


def test_samples_equal_full():
    L = ubp_synth.make_layer("t", 48, 20, 4, 60, 21, Nc=37)
    Y, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias, relu=True)
    rng = np.random.default_rng(1)
    so = rng.integers(0, 48, 50); sn = rng.integers(0, 37, 50)
    ys, as_ = oracle.masked_matmul_samples(L.W, L.mask, L.X, so, sn, L.bias, relu=True)
    assert np.array_equal(ys, Y[so, sn]) and np.array_equal(as_, A[so, sn])
    L3 = ubp_synth.make_layer("c", 16, 8, 4, 50, 22, B=2, H=6, Wd=5, R=9)
    Y3, A3 = oracle.masked_conv3x3(L3.W, L3.mask, L3.X, L3.bias, relu=True)
    sb = rng.integers(0, 2, 40); so = rng.integers(0, 16, 40); sy = rng.integers(0, 6, 40); sx = rng.integers(0, 5, 40)
    ys, as_ = oracle.masked_conv3x3_samples(L3.W, L3.mask, L3.X, sb, so, sy, sx, L3.bias, relu=True)
    assert np.array_equal(ys, Y3[so, sb, sy, sx]) and np.array_equal(as_, A3[so, sb, sy, sx])


# ---------------------------------------------------------------- invariants
def test_unit_vectors_and_identity():
    L = ubp_synth.make_layer("t", 20, 9, 4, 40, 31, Nc=9, bias=False, relu=False)
    Y, _ = oracle.masked_matmul(L.W, L.mask, np.eye(9, dtype=np.float32))
    assert np.array_equal(Y, (L.W[:, :, 0] * L.mask).astype(np.float64))     # X = e_c picks column c of Wm
    M = 7
    X = np.arange(M * 3, dtype=np.float32).reshape(M, 3)
    Yi, _ = oracle.masked_matmul(np.eye(M, dtype=np.float32), np.eye(M, dtype=np.uint8), X)
    assert np.array_equal(Yi, X.astype(np.float64))
    assert np.array_equal(oracle.wros_spmm(oracle.pack(np.eye(M, dtype=np.float32), np.eye(M, dtype=np.uint8), 1), X), X)


def test_linearity_and_relu_bias():
    rng = np.random.default_rng(5)
    L = ubp_synth.make_layer("t", 24, 10, 3, 50, 32, Nc=11, x_dist="normal")
    X1 = L.X; X2 = rng.integers(-4, 5, size=X1.shape).astype(np.float32)
    Wq = np.round(L.W * 64).astype(np.float32)        # integer weights -> exact sums
    X1q = np.round(X1 * 8).astype(np.float32)
    Ya, _ = oracle.masked_matmul(Wq, L.mask, X1q)
    Yb, _ = oracle.masked_matmul(Wq, L.mask, X2)
    Yc, _ = oracle.masked_matmul(Wq, L.mask, X1q + 2 * X2)
    assert np.array_equal(Yc, Ya + 2 * Yb)
    bias = np.arange(24, dtype=np.float32) - 12
    Yd, Ad = oracle.masked_matmul(Wq, L.mask, X1q, bias, relu=False)
    assert np.array_equal(Yd, Ya + bias[:, None])
    Ye, _ = oracle.masked_matmul(Wq, L.mask, X1q, bias, relu=True)
    assert np.array_equal(Ye, np.maximum(Yd, 0))
    assert (Ad >= np.abs(Yd)).all()
    # masked-out weights never matter
    W2 = Wq + (1 - L.mask[:, :, None].astype(np.float32)) * 1000
    assert np.array_equal(oracle.masked_matmul(W2, L.mask, X1q)[0], Ya)


@pytest.mark.parametrize("M,C,Nb,p,R", [(64, 64, 4, 50, 1), (37, 11, 3, 40, 1), (40, 16, 8, 80, 9),
                                        (33, 5, 16, 50, 1), (16, 16, 2, 90, 9)])
def test_pack_invariants_and_round_trip(M, C, Nb, p, R):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 77, Nc=4 if R == 1 else None, R=R, B=1, H=2, Wd=2)
    blob = oracle.pack(L.W, L.mask, Nb)
    s = blob_sections(blob)
    m = ubp_synth.block_budget(M, C, p, Nb)
    assert s["m"] == m == L.m and int(L.mask.sum()) == m * Nb          # Section 3.1 budget
    ip, idx, val = s["indptr"], s["indices"], s["values"]
    assert ip[0] == 0 and ip[-1] == m and (np.diff(ip) >= 0).all()
    assert (np.diff(ip)[M - Nb + 1:] == 0).all()                         # Eq. 1: no start past M - Nb
    cover = np.zeros((M, C), np.int32)
    for i in range(M):
        js = idx[ip[i]:ip[i + 1]]
        assert (np.diff(js) > 0).all()                                   # ascending input channel
        for b in range(ip[i], ip[i + 1]):
            j = idx[b]
            cover[i:i + Nb, j] += 1
            for t in range(Nb):                                          # rotation: row rho -> slot rho mod N
                assert np.array_equal(val[b, (i + t) % Nb].view(np.uint32), L.W[i + t, j].view(np.uint32))
    assert np.array_equal(cover, L.mask.astype(np.int32))               # Eq. 2: no overlap, full cover
    W2, mask2 = oracle.unpack(blob)
    assert np.array_equal(mask2, L.mask)
    assert np.array_equal(W2.view(np.uint32), (L.W * L.mask[:, :, None]).view(np.uint32) * L.mask[:, :, None])
    assert oracle.blob_dims(blob) == (M, C, R, Nb, m)


def test_pack_keeps_bits_of_special_values():
    M, C, Nb = 6, 2, 3
    mask = np.zeros((M, C), np.uint8); mask[0:3, 0] = 1; mask[3:6, 1] = 1
    W = np.ones((M, C, 1), np.float32)
    W[0, 0, 0] = -0.0; W[1, 0, 0] = 0.0; W[2, 0, 0] = np.float32(1e-42); W[4, 1, 0] = np.float32(-3e-45)
    W2, m2 = oracle.unpack(oracle.pack(W, mask, Nb))
    keep = mask.astype(bool)
    assert np.array_equal(W2[keep].view(np.uint32), W[keep].view(np.uint32))
    assert (W2[~keep].view(np.uint32) == 0).all()


def test_wros_walk_equals_definition_on_floats():
    for (M, C, Nb, p) in [(64, 64, 4, 50), (50, 30, 3, 60), (33, 8, 16, 50), (40, 40, 2, 80), (17, 9, 1, 70)]:
        L = ubp_synth.make_layer("t", M, C, Nb, p, 100 + M, Nc=29, x_dist="normal")
        Y, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias, relu=True)
        Yw = oracle.wros_spmm(oracle.pack(L.W, L.mask, Nb), L.X, L.bias, relu=True, tile_w=4)
        assert np.max(np.abs(Y - Yw) / A) < 1e-15


def test_generator_statistics():
    # most starts are unaligned, and the mask decodes back to the drawn starts
    mask, starts = ubp_synth.random_mask(128, 64, 4, 70, seed=1)
    bi, bj = oracle.decode_mask(mask, 4)
    got = [sorted(bi[bj == j].tolist()) for j in range(64)]
    # adjacent drawn blocks merge; cutting from the run top returns the same starts
    assert got == [sorted(s.tolist()) for s in starts]
    allst = np.concatenate(starts)
    assert 0.6 < (allst % 4 != 0).mean() < 0.9
