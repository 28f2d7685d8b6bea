"""CPU tests of the library's host code: the C ABI surface, the packer against
the oracle's independent packer (bit-exact), error paths, and the plan builder."""
import ctypes
import os
import re
import struct

import numpy as np
import pytest

import oracle
import ubp_synth
import paper_2407_19644_b200 as ubp
from helpers import plan_to_dense, krun_plan_to_dense

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "ubp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(ubp_[a-z0-9_]+)\s*\(", hdr))
    assert {"ubp_pack", "ubp_unpack", "ubp_spmm", "ubp_conv1x1", "ubp_conv3x3_implicit",
            "ubp_plan_build", "ubp_plan_size"} <= names
    L = ctypes.CDLL(ubp.lib_path())
    for n in sorted(names):
        assert hasattr(L, n), n


def test_strerror_and_variants():
    L = ubp.load()
    assert L.ubp_strerror(0) == b"ok"
    assert b"whole number of blocks" in L.ubp_strerror(-2)
    v = ubp.variants()
    assert len(v) >= 8 and all(isinstance(s, str) and s for s in v.values())


CASES = [(64, 64, 4, 50, 1), (37, 11, 3, 40, 1), (40, 16, 8, 80, 9), (33, 5, 16, 50, 1), (16, 16, 2, 90, 9),
         (5, 3, 1, 30, 1), (128, 96, 4, 70, 1), (20, 7, 5, 0, 1), (48, 48, 16, 50, 1)]


@pytest.mark.parametrize("M,C,Nb,p,R", CASES)
def test_pack_bit_exact_vs_oracle_and_round_trip(M, C, Nb, p, R):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 900 + M, Nc=4 if R == 1 else None, R=R, B=1, H=2, Wd=2)
    blob = ubp.ubp_pack(L.W, L.mask, Nb)
    assert blob == oracle.pack(L.W, L.mask, Nb)                       # bit-exact format
    W2, m2 = ubp.ubp_unpack(blob)
    Wo, mo = oracle.unpack(blob)
    assert np.array_equal(m2, L.mask) and np.array_equal(mo, m2)
    assert np.array_equal(W2.view(np.uint32), Wo.view(np.uint32))
    keep = L.mask.astype(bool)
    assert np.array_equal(W2[keep].view(np.uint32), L.W[keep].view(np.uint32)) and (W2[~keep].view(np.uint32) == 0).all()
    d = ubp.blob_view(blob)
    assert (d["M"], d["C"], d["R"], d["Nb"], d["m"]) == (M, C, R, Nb, L.m)
    assert d["m"] == oracle.block_budget(M, C, p, Nb)


def test_pack_special_values_and_aligned_pattern():
    M, C, Nb = 12, 3, 4
    mask, _ = ubp_synth.random_mask(M, C, Nb, 34, seed=2, aligned=True)
    W = np.random.default_rng(0).standard_normal((M, C, 1)).astype(np.float32)
    W[mask.astype(bool)][:1] = -0.0
    W[0, 0, 0] = np.float32(-0.0); W[1, 0, 0] = np.float32(1e-42)
    assert ubp.ubp_pack(W, mask, Nb) == oracle.pack(W, mask, Nb)


@pytest.mark.parametrize("kind", ["ragged", "edge", "value", "nb_gt_m", "nb_zero"])
def test_pack_rejects_bad_input(kind):
    M, C, Nb = 8, 2, 3
    mask = np.zeros((M, C), np.uint8)
    W = np.ones((M, C), np.float32)
    want = -2
    if kind == "ragged":
        mask[1:5, 0] = 1
    elif kind == "edge":
        mask[6:8, 1] = 1
    elif kind == "value":
        mask[0:3, 0] = 1; mask[2, 0] = 3; want = -1
    elif kind == "nb_gt_m":
        Nb = 9; want = -1
    else:
        Nb = 0; want = -1
    with pytest.raises(ubp.UbpError) as e:
        ubp.ubp_pack(W, mask, Nb)
    assert e.value.code == want
    if kind in ("ragged", "edge", "value"):
        with pytest.raises(oracle.OracleError):
            oracle.pack(W, mask, Nb)


def test_pack_null_and_small_buffer():
    L = ubp.load()
    n = ctypes.c_size_t(0)
    assert L.ubp_pack(None, None, 4, 4, 1, 2, None, 0, ctypes.byref(n)) == -1
    W = np.ones((4, 4), np.float32); mask = np.zeros((4, 4), np.uint8); mask[0:2, 1] = 1
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    assert L.ubp_pack(p(W), p(mask), 4, 4, 1, 2, None, 0, ctypes.byref(n)) == 0 and n.value > 64
    small = np.zeros(32, np.uint8)
    assert L.ubp_pack(p(W), p(mask), 4, 4, 1, 2, p(small), 32, ctypes.byref(n)) == -3


def test_blob_view_rejects_corruption():
    L = ubp_synth.make_layer("t", 16, 8, 4, 50, 3, Nc=4)
    blob = bytearray(ubp.ubp_pack(L.W, L.mask, 4))
    for mutate in ("magic", "trunc", "indptr", "index"):
        b = bytearray(blob)
        if mutate == "magic":
            b[0] = ord("X")
        elif mutate == "trunc":
            b = b[:len(b) - 64]
        elif mutate == "indptr":
            struct.pack_into("<i", b, 64 + 4, 9999)
        else:
            off = 64 + (4 * 17 + 63) // 64 * 64
            struct.pack_into("<i", b, off, 1000)
        with pytest.raises(ubp.UbpError) as e:
            ubp.blob_view(bytes(b))
        assert e.value.code == -4


def test_blob_with_overlapping_blocks_is_refused_everywhere():
    """Two blocks of one input channel that share rows violate Eq. 2. Such a blob must be refused by the validation
    every consumer runs (view, unpack, plan size, plan image), so that no plan is ever built from it: the sparse and
    the dense part of a plan would otherwise disagree about the doubly covered rows."""
    M, C, Nb = 12, 3, 4
    mask = np.zeros((M, C), np.uint8)
    mask[0:4, 1] = 1; mask[6:10, 1] = 1; mask[2:6, 2] = 1
    W = np.arange(M * C, dtype=np.float32).reshape(M, C) + 1
    blob = bytearray(ubp.ubp_pack(W, mask, Nb))
    d = ubp.blob_view(bytes(blob))
    assert d["m"] == 3 and list(d["indptr"][:8]) == [0, 1, 1, 2, 2, 2, 2, 3]
    # move the block that starts at row 6 of channel 1 up to row 2: rows 2 and 3 of channel 1 are now covered twice.
    # New start rows: 0 (channel 1), 2 (channels 1 and 2) -> indptr 0,1,1,3,...; indices 1,1,2; channels ascending
    indptr = [0, 1, 1] + [3] * (M - 2)
    struct.pack_into(f"<{M + 1}i", blob, 64, *indptr)
    off_idx = 64 + (4 * (M + 1) + 63) // 64 * 64
    struct.pack_into("<3i", blob, off_idx, 1, 1, 2)
    for call in (lambda b: ubp.blob_view(b), lambda b: ubp.ubp_unpack(b), lambda b: ubp.plan_size(b),
                 lambda b: ubp.plan_image(b), lambda b: ubp.plan_size(b, 32)):
        with pytest.raises(ubp.UbpError) as e:
            call(bytes(blob))
        assert e.value.code == -4
    # adjacent blocks (a run of two blocks) are fine
    mask2 = np.zeros((M, C), np.uint8); mask2[0:8, 0] = 1
    assert ubp.blob_view(ubp.ubp_pack(W, mask2, Nb))["m"] == 2


@pytest.mark.parametrize("M,C,Nb,p,R,variant", [
    (64, 64, 4, 50, 1, 0), (100, 70, 4, 60, 1, 1), (100, 70, 4, 60, 1, 3), (100, 70, 4, 60, 1, 4), (100, 70, 4, 60, 1, 5), (100, 70, 4, 60, 1, 7),
    (37, 45, 3, 40, 1, 0), (50, 33, 2, 50, 1, 0), (72, 40, 8, 50, 1, 0), (72, 40, 8, 50, 1, 9),
    (80, 40, 16, 50, 1, 0), (60, 20, 12, 40, 1, 0), (45, 17, 1, 70, 1, 0), (40, 20, 8, 50, 9, 0),
    (24, 18, 4, 50, 9, 0), (30, 10, 6, 40, 9, 0),
])
def test_plan_image_replays_to_masked_weight(M, C, Nb, p, R, variant):
    """Every kept weight appears exactly once among the rows the panels own, with
    its value; nothing else appears. Entries crossing a panel boundary are listed twice."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 70 + M, Nc=4 if R == 1 else None, R=R, B=1, H=2, Wd=2)
    blob = ubp.ubp_pack(L.W, L.mask, Nb)
    img, geom = ubp.plan_image(blob, variant)
    assert len(img) == ubp.plan_size(blob, variant) and len(img) % 256 == 0
    Wd, hits, n_entries = plan_to_dense(img, geom, M, C, R)
    assert np.array_equal(hits, L.mask.astype(np.int32))
    assert np.array_equal(Wd.view(np.uint32), (L.W * L.mask[:, :, None]).view(np.uint32) * L.mask[:, :, None])
    nbk, P = geom["nbk"], geom["panel_rows"]
    assert Nb % nbk == 0
    bi, bj = oracle.decode_mask(L.mask, Nb)
    sub = np.concatenate([bi + u * nbk for u in range(Nb // nbk)])
    crossing = int(((sub % P) + nbk > P).sum())
    assert n_entries == len(sub) + crossing


def test_plan_of_the_paper_dataflow_variants_is_the_canonical_arrays():
    """Variants 60 / 61 walk the packed format itself: their plan image is a 256-byte header followed by indptr,
    indices and the rotated values, each on a 16-byte boundary, bit for bit as in the blob."""
    L = ubp_synth.make_layer("t", 50, 30, 4, 60, 77, Nc=4)
    blob = ubp.ubp_pack(L.W, L.mask, 4)
    d = ubp.blob_view(blob)
    for variant in (60, 61):
        img, _ = ubp.plan_image(blob, variant)
        assert len(img) % 256 == 0 and not img[:256].any()
        o1 = (256 + 4 * 51 + 15) // 16 * 16
        o2 = (o1 + 4 * d["m"] + 15) // 16 * 16
        assert np.array_equal(np.frombuffer(img, "<i4", 51, 256), d["indptr"])
        assert np.array_equal(np.frombuffer(img, "<i4", d["m"], o1), d["indices"])
        assert np.array_equal(np.frombuffer(img, "<u4", d["m"] * 4, o2), d["values"].view(np.uint32).ravel())
    L3 = ubp_synth.make_layer("t", 24, 12, 3, 50, 78, Nc=4)
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(ubp.ubp_pack(L3.W, L3.mask, 3), 60)         # block sizes 1, 2, 4, 8, 16 only
    L9 = ubp_synth.make_layer("t", 16, 8, 4, 50, 79, R=9, B=1, H=2, Wd=2)
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(ubp.ubp_pack(L9.W, L9.mask, 4), 61)         # 1x1 only


def test_plan_rejects_wrong_kind():
    L = ubp_synth.make_layer("t", 16, 8, 4, 50, 3, Nc=4)
    blob = ubp.ubp_pack(L.W, L.mask, 4)
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(blob, 20)         # a 3x3 configuration for an R = 1 blob
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(blob, 9)          # 8 rows per entry do not divide a block of 4
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(blob, 999)
    assert ubp.plan_size(blob, 7) > 0   # 2 rows per entry: each block becomes two entries


@pytest.mark.parametrize("M,C,Nb,p,R,variant,sparse_variant", [(130, 140, 4, 60, 1, 32, 14), (128, 20, 8, 50, 9, 40, 20)])
def test_tensor_core_plan_dense_part(M, C, Nb, p, R, variant, sparse_variant):
    """The dense part of a tensor-core plan: Wh + Wl reproduces the masked weight to 2^-21 relative, both pieces are
    exact TF32 numbers (low 13 mantissa bits clear), pruned positions are zero; k = tap * C + channel."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 33 + M, Nc=4 if R == 1 else None, R=R, B=1, H=2, Wd=2)
    blob = ubp.ubp_pack(L.W, L.mask, Nb)
    img, geom = ubp.plan_image(blob, variant)
    tc_off = ubp.plan_size(blob, sparse_variant)             # same geometry without the dense part
    kp = (C * R + 3) // 4 * 4
    kp16 = (C * R + 15) // 16 * 16
    tc16_off = tc_off + (2 * M * kp * 4 + 255) // 256 * 256
    nrt, nch = (M + 255) // 256 * 2, kp16 // 16                # whole pairs of 128-row tiles
    assert len(img) == tc16_off + nrt * nch * 8192
    # the embedded sparse plan is byte-identical to the stand-alone one
    img_s, _ = ubp.plan_image(blob, sparse_variant)
    assert np.array_equal(img[:tc_off], img_s)
    Wh = np.frombuffer(img, "<f4", M * kp, tc_off).reshape(M, kp)
    Wl = np.frombuffer(img, "<f4", M * kp, tc_off + 4 * M * kp).reshape(M, kp)
    assert not (Wh.view(np.uint32) & 0x1fff).any() and not (Wl.view(np.uint32) & 0x1fff).any()
    Wm = np.ascontiguousarray((L.W * L.mask[:, :, None]).transpose(0, 2, 1)).reshape(M, R * C)   # k = tap * C + channel
    assert not Wh[:, C * R:].any() and not Wl[:, C * R:].any()
    got = Wh[:, :C * R].astype(np.float64) + Wl[:, :C * R]
    assert np.all(np.abs(got - Wm) <= np.abs(Wm) * 2.0 ** -20)
    assert not got[Wm == 0].any()
    assert np.array_equal(Wh[:, :C * R], (Wm.view(np.uint32) & 0xffffe000).view(np.float32))
    # the same matrix as two bf16 pieces (8-bit significands): W1 = nearest bf16, so |W - W1| <= 2^-8 |W|, and
    # W1 + W2 within 2^-16 |W|
    # tiled: 8 KB blocks [row tile][chunk] = [piece][128 rows][16 channels], rows of 32 bytes whose 16-byte halves
    # are swapped on rows with bit 2 set
    blocks = np.frombuffer(img, "<u2", nrt * nch * 4096, tc16_off).reshape(nrt, nch, 2, 128, 2, 8)
    rows = np.arange(128)
    swap = ((rows >> 2) & 1).astype(bool)
    blocks = blocks.copy()
    blocks[:, :, :, swap] = blocks[:, :, :, swap][..., ::-1, :]
    W12 = blocks.reshape(nrt, nch, 2, 128, 16).transpose(2, 0, 3, 1, 4)          # [piece][row tile][row in tile][k]
    W12 = W12.reshape(2, nrt, 128, kp16)
    # row tile t holds rows 128 t .. 128 t + 127 of the matrix in order (a layer of at most 128 rows: tile 0 holds it,
    # tile 1 is zero: both CTAs of a pair multiply tile 0 and split the columns)
    W12 = W12.reshape(2, nrt * 128, kp16)
    assert not W12[:, M:].any()                                # padding rows
    W1 = (W12[0, :M].astype(np.uint32) << 16).view(np.float32)
    W2 = (W12[1, :M].astype(np.uint32) << 16).view(np.float32)
    assert not W1[:, C * R:].any() and not W2[:, C * R:].any()
    assert np.all(np.abs(W1[:, :C * R].astype(np.float64) - Wm) <= np.abs(Wm) * 2.0 ** -8)
    got16 = W1[:, :C * R].astype(np.float64) + W2[:, :C * R]
    assert np.all(np.abs(got16 - Wm) <= np.abs(Wm) * 2.0 ** -16)
    assert not got16[Wm == 0].any()


def test_bf16_three_term_product_error_bound():
    """The arithmetic of the bf16-product tensor-core variants, emulated in numpy: with x1 = bf16(x), x2 = bf16(x - x1)
    (round to nearest even, 8 significant bits) and likewise w, the three-term product w1 x1 + w2 x1 + w1 x2 is within
    3 * 2^-16 of w x, relative to |w x|, for every pair - the bound the GPU tests assert and the 1e-4 gate contains."""
    def bf16(v):
        b = v.astype(np.float32).view(np.uint32).astype(np.uint64)
        b = ((b + 0x7fff + ((b >> 16) & 1)) >> 16) << 16
        return b.astype(np.uint32).view(np.float32)

    rng = np.random.default_rng(12)
    n = 1_000_000
    cases = [(rng.standard_normal(n), rng.standard_normal(n) * 0.05), (rng.uniform(1, 2, n), rng.uniform(1, 2, n)),
             (1 + 2.0 ** -8 - 2.0 ** -16 * rng.uniform(0.9, 1.1, n),) * 2,       # just below a rounding boundary
             (rng.standard_normal(n) * 1e-20, rng.standard_normal(n) * 1e15)]    # far from 1: bf16 has fp32's range
    for x, w in cases:
        x, w = x.astype(np.float32), w.astype(np.float32)
        x1, w1 = bf16(x), bf16(w)
        x2, w2 = bf16(x - x1), bf16(w - w1)
        assert np.all(np.abs((x - x1).astype(np.float64)) <= np.abs(x) * 2.0 ** -8)
        assert np.all(np.abs(x.astype(np.float64) - x1 - x2) <= np.abs(x) * 2.0 ** -16)
        approx = x1.astype(np.float64) * w1 + x1.astype(np.float64) * w2 + x2.astype(np.float64) * w1
        exact = x.astype(np.float64) * w
        assert np.all(np.abs(approx - exact) <= np.abs(exact) * 3 * 2.0 ** -16)
    # The bound cannot be tightened to 3 * 2^-18: bf16 keeps 8 significant bits, so rounding to nearest leaves up to
    # 2^-8 |x| (not 2^-9), the second piece up to 2^-16 |x|, and the dropped terms w1 x3, w3 x1 and w2 x2 reach
    # 2^-16 |w x| each. One witness pair (both operands a little above 1):
    x = np.array([float.fromhex("0x1.0aea86p+0")], np.float32)
    w = np.array([float.fromhex("0x1.031c8ap+0")], np.float32)
    x1, w1 = bf16(x), bf16(w)
    x2, w2 = bf16(x - x1), bf16(w - w1)
    approx = x1.astype(np.float64) * w1 + x1.astype(np.float64) * w2 + x2.astype(np.float64) * w1
    rel = float(np.abs(approx - x.astype(np.float64) * w)[0] / (float(x[0]) * float(w[0])))
    assert 3 * 2.0 ** -18 < rel <= 3 * 2.0 ** -16


def test_kmajor_blocks_pack_as_the_transposed_layer_and_convert_to_a_plan_blob():
    """Blocks of B consecutive input channels inside one output row (the other orientation): the blob is the oracle's
    blob of the transposed layer, bit for bit; a run that is not a whole number of blocks is refused; the conversion
    for the plan builder keeps exactly the same weights as blocks of one output channel."""
    import paper_2407_19644_b200 as ubp
    M, Cin, B = 24, 40, 4
    Lt = ubp_synth.make_layer("kmajor", Cin, M, B, 70, 4242, Nc=8, make_x=False)      # transposed roles: [C][M]
    W = np.ascontiguousarray(Lt.W[:, :, 0].T)                                         # [M][C]
    mask = np.ascontiguousarray(Lt.mask.T)
    kblob = ubp.ubp_pack_kmajor(W, mask, B)
    assert kblob == oracle.pack(np.ascontiguousarray(W.T), np.ascontiguousarray(mask.T), B)
    v = ubp.blob_view(kblob)
    assert (v["M"], v["C"], v["Nb"], v["m"]) == (Cin, M, B, Lt.m)
    pblob = ubp.ubp_kmajor_to_plan_blob(kblob)
    assert pblob == oracle.pack(W, mask, 1)
    W2, m2 = ubp.unpack_ubp(pblob)
    assert np.array_equal(m2, mask) and np.array_equal(W2[:, :, 0].view(np.uint32), np.where(mask == 1, W, np.float32(0)).view(np.uint32))
    bad = mask.copy()
    i, j = np.argwhere(bad == 1)[0]
    bad[i, j] = 0                                      # shortens one run by one element
    with pytest.raises(ubp.UbpError) as e:
        ubp.ubp_pack_kmajor(W, bad, B)
    assert e.value.code == -2


@pytest.mark.parametrize("M,Cin,B,p", [(40, 200, 4, 60), (70, 130, 2, 50), (24, 96, 8, 70), (33, 160, 16, 50), (50, 64, 4, 90)])
def test_krun_plan_image_replays_to_the_masked_weight(M, Cin, B, p):
    """The plan of the K-run sparse kernel (one entry = one run of B consecutive input channels of one output row):
    replayed on the host it gives exactly the masked weight; it holds ONE channel index per run, plus one more for
    every run that crosses a 64-channel tile boundary (cut there, each piece padded with zero weights)."""
    Lt = ubp_synth.make_layer("t", Cin, M, B, p, 60 + M, Nc=4, make_x=False)        # transposed roles: [C][M]
    W = np.ascontiguousarray(Lt.W[:, :, 0].T)
    mask = np.ascontiguousarray(Lt.mask.T)
    kblob = ubp.ubp_pack_kmajor(W, mask, B)
    variant = {2: 70, 4: 71, 8: 72, 16: 73}[B]
    img, geom = ubp.plan_image(kblob, variant, kmajor=True)
    assert geom["nbk"] == B and len(img) == ubp.plan_size(kblob, variant, kmajor=True)
    Wd, n_entries = krun_plan_to_dense(img, geom, M, Cin)
    assert np.array_equal(Wd.astype(np.float32), W * mask)
    k0, rows = oracle.decode_mask(mask.T, B)                 # blocks of the transposed layer: (first channel, output row)
    crossing = int(((k0 % geom["k_tile"]) + B > geom["k_tile"]).sum())
    assert n_entries == len(k0) + crossing
    # sparse layers choose this plan by themselves, dense-enough large ones the tensor-core plan of the re-expressed layer
    assert ubp.plan_size(kblob, 0, kmajor=True) == len(img) if (M < 128 or p >= 93) else True
    with pytest.raises(ubp.UbpError):
        ubp.plan_size(kblob, variant)                        # a K-run configuration needs the K-major entry points


def test_block_selection_argument_checks_need_no_device():
    """Size query and limits of the block-selection entry points (no kernel runs): bad sizes are refused, layers
    beyond the supported row count are reported as unsupported, the scratch grows with the layer."""
    import ctypes as C
    import paper_2407_19644_b200 as ubp
    L = ubp.load()
    n = C.c_size_t(0)
    assert L.ubp_bed_workspace_size(64, 32, 4, C.byref(n)) == 0 and n.value > 64 * 32 * 10
    small = n.value
    assert L.ubp_bed_workspace_size(512, 512, 2, C.byref(n)) == 0 and n.value > small
    assert L.ubp_bed_workspace_size(64, 32, 0, C.byref(n)) == -1          # block size < 1
    assert L.ubp_bed_workspace_size(3, 32, 4, C.byref(n)) == -1           # block longer than the column
    assert L.ubp_bed_workspace_size(64, 32, 4, None) == -1
    assert L.ubp_bed_workspace_size(16385, 8, 4, C.byref(n)) == -6        # more rows than the kernel's lists hold
    assert L.ubp_bed_workspace_size(16384, 1 << 17, 4, C.byref(n)) == -6  # M * C >= 2^31
    # null pointers are refused before anything is launched
    assert L.ubp_bed_select(None, 64, 32, 1, 4, 10, None, 0, None, None, None) == -1
    assert L.ubp_block_scores(None, 64, 32, 1, 4, None, 0, None, None) == -1


@pytest.mark.parametrize("M,C,p,tensor", [(256, 256, 90, True), (256, 256, 95, True), (256, 256, 98, False),
                                          (1024, 1024, 99, True), (1024, 1024, 99.7, False), (64, 256, 70, False),
                                          (256, 32, 70, False)])
def test_automatic_variant_by_density_and_size(M, C, p, tensor):
    """Variant 0: the dense tensor-core form from 128 rows x 64 channels on whenever at least 3 % of the weights are
    kept (0.5 % for layers of a million weights or more), else the sparse kernel. Seen on the host through the plan's
    size: a tensor-core plan carries the dense weight beside the sparse plan."""
    rng = np.random.default_rng(int(M + C + 10 * p))
    Nb = 4
    m = int(M * C * (100 - p) / 100) // Nb
    mask = np.zeros((M, C), np.uint8)
    # m blocks at aligned, distinct places (the rule only looks at their number)
    for q in rng.choice((M // Nb) * C, m, replace=False):
        mask[(q % (M // Nb)) * Nb:(q % (M // Nb)) * Nb + Nb, q // (M // Nb)] = 1
    W = rng.standard_normal((M, C, 1)).astype(np.float32)
    blob = ubp.ubp_pack(W, mask, Nb)
    sparse_id = 14 if M > 64 else 51
    auto, dense, sparse = ubp.plan_size(blob, 0), ubp.plan_size(blob, 36), ubp.plan_size(blob, sparse_id)
    assert dense > sparse
    assert auto == (dense if tensor else sparse)
