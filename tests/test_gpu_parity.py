"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the
same seeded inputs. Gate: max |Y - Yref| / (|Wm||X| + |bias|) <= 1e-4 (fp32
multiply-add, fp32 accumulation against a double reference); the tighter
summation bound (L + 2) * 2^-24, L = kept terms per output, is asserted too."""
import numpy as np
import pytest

import oracle
import ubp_synth
from helpers import scaled_error

pytestmark = pytest.mark.gpu

TOL = 1e-4


@pytest.fixture(scope="module")
def env():
    import torch
    import paper_2407_19644_b200 as ubp
    assert torch.cuda.is_available()
    ubp.load()
    return torch, ubp


def terms_per_output(L):
    return int(L.mask.sum(axis=1).max()) * L.R


def run_spmm(env, L, variant=0, pad=0, misalign=0, relu=None, use_bias=True):
    torch, ubp = env
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert blob == oracle.pack(L.W, L.mask, L.Nb)
    plan = ubp.Plan(blob, variant)
    Nc = L.X.shape[1]
    ld = Nc + pad
    xbuf = torch.zeros(L.C * ld + 8, dtype=torch.float32, device="cuda")
    X = xbuf[misalign:misalign + L.C * ld].view(L.C, ld)[:, :Nc]
    X.copy_(torch.from_numpy(L.X))
    ybuf = torch.full((L.M * ld + 8,), float("nan"), dtype=torch.float32, device="cuda")
    Y = ybuf[misalign:misalign + L.M * ld].view(L.M, ld)[:, :Nc]
    bias = torch.from_numpy(L.bias).cuda() if (use_bias and L.bias is not None) else None
    r = L.relu if relu is None else relu
    ubp.ubp_spmm(plan, X, bias, r, out=Y)
    plan.check()
    Yh = Y.cpu().numpy()
    if pad:
        assert torch.isnan(ybuf[misalign:misalign + L.M * ld].view(L.M, ld)[:, Nc:]).all()   # padding untouched
    Yref, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias if bias is not None else None, relu=r)
    return Yh, Yref, A, plan


def is_bf16(variant):
    """Tensor-core variants whose CTA-pair kernel multiplies with three bf16 products instead of three TF32 ones."""
    return 34 <= variant <= 37 or 44 <= variant <= 47 or 64 <= variant <= 67


def arith_bound(L, variant):
    """Summation bound of the arithmetic that ran: (L + 2) 2^-24 for the fp32 kernels; the tensor-core variants split
    each operand into two pieces and drop the low x low product and the bits below the low pieces, and their
    accumulator truncates: TF32 pieces (each dropped term <= 2^-20 |w||x|) 2^-18 + (L + 2) 2^-23; bf16 pieces (three
    dropped terms <= 2^-16 |w||x| each) 3 * 2^-16 + (L + 2) 2^-23."""
    n = terms_per_output(L) + 2
    if is_bf16(variant):
        return 3 * 2.0 ** -16 + n * 2.0 ** -23
    if variant >= 30:
        return 2.0 ** -18 + n * 2.0 ** -23
    return n * 2.0 ** -24


def check(Yh, Yref, A, L, tensor_core=False, variant=None):
    """Gate 1e-4, plus the bound of the arithmetic that ran (arith_bound; tensor_core=True without a variant means
    the TF32 form)."""
    assert np.isfinite(Yh).all()
    err = scaled_error(Yh, Yref, A)
    assert err <= TOL, err
    bound = arith_bound(L, variant if variant is not None else (32 if tensor_core else 0))
    assert err <= bound, (err, bound)
    return err


SMALL = [
    # M, C, Nb, p, Nc, variant
    (64, 64, 4, 50, 256, 0), (100, 70, 4, 60, 300, 1), (100, 70, 4, 60, 520, 3),
    (300, 150, 4, 70, 260, 4), (300, 150, 4, 70, 260, 5), (300, 150, 4, 70, 516, 51), (300, 150, 4, 70, 516, 14), (64, 300, 8, 70, 516, 55), (64, 300, 2, 70, 516, 53),
    (64, 32, 4, 60, 1028, 0), (48, 24, 8, 50, 516, 0), (40, 100, 2, 50, 516, 0), (33, 20, 1, 50, 260, 0), (37, 45, 3, 40, 132, 0), (50, 33, 2, 50, 388, 0), (72, 40, 8, 50, 264, 0),
    (200, 40, 8, 50, 264, 9), (80, 40, 16, 50, 260, 0), (60, 20, 12, 40, 128, 0), (45, 17, 1, 70, 256, 0),
    (16, 8, 4, 50, 4, 0), (130, 257, 4, 80, 1028, 0), (64, 64, 4, 0, 256, 0),
]


@pytest.mark.parametrize("M,C,Nb,p,Nc,variant", SMALL)
def test_spmm_small(env, M, C, Nb, p, Nc, variant):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 10 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0))
    Yh, Yref, A, plan = run_spmm(env, L, variant)
    check(Yh, Yref, A, L, variant=plan.variant)


@pytest.mark.parametrize("M,C,Nb,p,Nc,variant", [c for c in SMALL if c[2] > 1 and c[3] > 0] +
                         [c for c in [(128, 64, 4, 50, 256, 32), (300, 150, 4, 70, 520, 32), (520, 200, 8, 50, 1028, 33),
                                      (256, 256, 4, 70, 4128, 36), (100, 200, 4, 50, 8200, 36), (260, 40, 16, 50, 516, 37)]])
def test_spmm_aligned_blocks(env, M, C, Nb, p, Nc, variant):
    """The aligned pattern (every block starts at a multiple of its size: Section 3.1's remark that aligned pruning is
    the special case of the unaligned one) through the same kernels: sparse configurations and tensor-core variants."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 20 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0), aligned=True)
    assert all((s % Nb == 0).all() for s in L.starts)
    Yh, Yref, A, plan = run_spmm(env, L, variant)
    check(Yh, Yref, A, L, variant=plan.variant)


@pytest.mark.parametrize("variant", [60, 61])
@pytest.mark.parametrize("M,C,Nb,p,Nc,aligned,pad,misalign", [
    (64, 64, 4, 50, 256, False, 0, 0), (100, 70, 4, 60, 300, False, 0, 0), (300, 150, 2, 70, 516, False, 0, 0),
    (33, 20, 1, 50, 260, False, 0, 0), (72, 40, 8, 50, 264, False, 0, 0), (80, 40, 16, 50, 260, False, 0, 0),
    (130, 257, 4, 80, 1028, False, 0, 0), (16, 8, 4, 50, 4, False, 0, 0), (8, 40, 8, 50, 128, False, 0, 0),
    (100, 70, 4, 60, 300, True, 0, 0), (72, 40, 8, 50, 264, True, 0, 0), (96, 64, 2, 70, 520, True, 0, 0),
    (70, 50, 4, 60, 130, False, 2, 0), (70, 50, 4, 60, 131, False, 1, 0), (70, 50, 4, 60, 255, False, 0, 0),
    (70, 50, 4, 60, 256, False, 0, 1), (70, 50, 2, 60, 1, False, 3, 0), (512, 96, 4, 80, 2048, False, 0, 0),
])
def test_paper_dataflow_variants(env, variant, M, C, Nb, p, Nc, aligned, pad, misalign):
    """The comparison kernels that keep the paper's own loop (row step 1 over the canonical arrays; Section 3.3 and
    Section 4.2): weight-rotating output-stationary (60) and naive with shifted outputs (61), on unaligned and aligned
    masks, element-wise pruning (Nb = 1), ragged and misaligned operands. fp32 FMA: the fp32 summation bound holds."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 30 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0), aligned=aligned)
    Yh, Yref, A, plan = run_spmm(env, L, variant, pad=pad, misalign=misalign)
    assert plan.variant == variant and plan.tile_choice(Nc)[0] == 3
    check(Yh, Yref, A, L, variant=0)


def test_paper_dataflow_variants_agree_bitwise_where_the_order_is_the_same(env):
    """Both forms add a row's products in the same order (tiles ascending, channels ascending inside a tile), so the
    rotation changes where an accumulator lives, not what it holds: identical bits."""
    torch, ubp = env
    L = ubp_synth.make_layer("t", 200, 120, 4, 70, 4711, Nc=1024, x_dist="normal")
    blob = ubp.ubp_pack(L.W, L.mask, 4)
    X = torch.from_numpy(L.X).cuda(); b = torch.from_numpy(L.bias).cuda()
    Y60 = ubp.ubp_spmm(ubp.Plan(blob, 60), X, b, True)
    Y61 = ubp.ubp_spmm(ubp.Plan(blob, 61), X, b, True)
    assert torch.equal(Y60, Y61)


TC_CASES = [
    # M, C, Nb, p, Nc, variant  (30..33 = tensor-core variants for 1 / 2 / 4 / 8-row entries)
    (128, 64, 4, 50, 256, 32), (128, 16, 4, 50, 256, 32), (100, 70, 4, 60, 300, 32), (300, 150, 4, 70, 520, 32),
    (257, 33, 1, 60, 260, 30), (64, 64, 2, 50, 256, 31), (520, 200, 8, 50, 1028, 33), (260, 40, 16, 50, 516, 33),
    (130, 257, 4, 80, 1028, 32), (384, 100, 12, 40, 772, 32), (256, 128, 4, 0, 512, 32), (200, 20, 4, 100, 256, 32),
    # more than 128 rows: the two-CTA kernel; whole 32-column groups (one 3-D copy of X per chunk) with and without
    # a ragged last column tile, more chunks than pipeline stages, a ragged last row pair
    (512, 96, 4, 60, 2048, 32), (300, 150, 4, 70, 544, 32), (256, 256, 4, 70, 4128, 32), (640, 40, 8, 50, 96, 33),
    # at most 128 rows through the bf16-product CTA-pair kernel: each CTA of the pair takes half of the rows
    (128, 128, 4, 60, 4100, 36), (100, 200, 4, 50, 8200, 36), (72, 144, 8, 50, 8196, 37), (128, 64, 2, 50, 16384, 35),
    # ... and a quarter of those in each tensor-memory lane quarter: 2, 6, 10 and 14 rows per quarter, with row
    # counts that leave the last quarters partly or wholly empty
    (8, 128, 4, 50, 8192, 36), (40, 160, 4, 60, 4160, 36), (66, 128, 2, 50, 8200, 35), (120, 256, 8, 70, 4096, 37),
    (9, 64, 1, 50, 4100, 34),
]


@pytest.mark.parametrize("M,C,Nb,p,Nc,variant", TC_CASES)
def test_spmm_tensor_core_variant(env, M, C, Nb, p, Nc, variant):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 10 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0))
    Yh, Yref, A, plan = run_spmm(env, L, variant)
    assert plan.variant == variant
    check(Yh, Yref, A, L, variant=variant)
    if (M, C) == (128, 128):
        assert plan.tile_choice(Nc)[0] == 2          # the CTA pair splits the 128 rows 64 / 64
    if M > 128:                          # the same layer through the bf16-product form of the CTA-pair kernel
        Yh, Yref, A, plan = run_spmm(env, L, variant + 4)
        assert plan.variant == variant + 4 and plan.tile_choice(Nc)[0] in (1, 2)
        err = check(Yh, Yref, A, L, variant=variant + 4)
        assert err <= 2e-5               # far inside its worst-case bound on random data


@pytest.mark.parametrize("M,C,Nb,p,Nc,variant", [(256, 256, 4, 70, 4128, 86), (300, 150, 4, 70, 544, 86), (520, 200, 8, 50, 1028, 87),
                                                  (128, 128, 4, 60, 4100, 86), (72, 144, 8, 50, 8196, 87), (257, 33, 1, 60, 260, 84),
                                                  (512, 512, 2, 80, 6272, 85)])
def test_spmm_three_piece_variant(env, M, C, Nb, p, Nc, variant):
    """The bf16 CTA-pair kernel with every operand in three bf16 pieces and six products per fp32 product (variants
    84..87): the dropped terms are below 2^-23 |w||x|, so what is left is the tensor core's fp32 accumulation (it
    truncates): inside 2^-22 + (L + 2) 2^-23, about 1-2 * 10^-6 of |Wm||X| on random data -- closer to the oracle than
    the two-piece form, not as close as the fp32 FMA kernel (3 * 10^-7), whose roundings are to nearest."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 10 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0))
    Yh, Yref, A, plan = run_spmm(env, L, variant)
    assert plan.variant == variant and plan.tile_choice(Nc)[0] == 2
    assert np.isfinite(Yh).all()
    err = scaled_error(Yh, Yref, A)
    n = terms_per_output(L) + 2
    assert err <= 2.0 ** -22 + n * 2.0 ** -23 and err <= 3e-6
    Y2, _, _, _ = run_spmm(env, L, variant - 50)                 # the two-piece form of the same layer
    assert scaled_error(Y2, Yref, A) > err


@pytest.mark.parametrize("M,C,Nb,p,Nc,rows", [(512, 256, 4, 80, 12544, 512), (1024, 96, 8, 50, 6001, 512),
                                              (1000, 160, 2, 70, 4099, 512), (768, 128, 4, 70, 6272, 256),
                                              (512, 64, 4, 60, 14208, 512), (512, 64, 4, 60, 19201, 512),
                                              (512, 48, 4, 60, 45001, 512), (1024, 32, 2, 50, 30003, 512)])
def test_spmm_stacked_row_tiles(env, M, C, Nb, p, Nc, rows):
    """Layers whose rows fill whole 512-row tiles may run two 256-row MMA tiles on one staged activation tile (one copy
    and one split pass for both), with one tile per CTA pair or several (then a tile's epilogue is not hidden: both
    accumulators belong to it); an odd number of 256-row tiles keeps the plain tiles. Same arithmetic either way."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 3 * M + C, Nc=Nc, x_dist="normal", relu=(Nc % 2 == 0))
    Yh, Yref, A, plan = run_spmm(env, L, 34 + {2: 1, 4: 2, 8: 3}[Nb])
    assert (plan.tile_choice(Nc)[:2] == (2, 512)) == (rows == 512)
    check(Yh, Yref, A, L, variant=36)


@pytest.mark.parametrize("M,C,Nb,p,Nc,pad", [(256, 520, 4, 70, 2100, 0), (300, 1000, 2, 80, 1531, 4), (128, 777, 1, 60, 2050, 0),
                                             (512, 512, 4, 70, 1030, 8), (1024, 528, 8, 80, 900, 0), (260, 2048, 4, 90, 777, 0),
                                             (768, 1037, 4, 75, 4100, 0)])
def test_spmm_long_reductions(env, M, C, Nb, p, Nc, pad):
    """Reductions of 32 sixteen-channel chunks and more: a pipeline stage of the bf16 pair kernel holds two chunks, their
    weight blocks arrive in one copy and their 32 channel rows in one box. Odd chunk counts (the last stage holds a single
    chunk and the box reaches past the last channel), channel counts that are no multiple of 16, every tile kind
    (plain, both CTAs on one row tile, several tiles per pair), padded leading dimensions."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 5 * M + C, Nc=Nc, x_dist="normal", relu=(C % 2 == 0))
    Yh, Yref, A, plan = run_spmm(env, L, 34 + {1: 0, 2: 1, 4: 2, 8: 3}[Nb], pad=pad)
    assert plan.tile_choice(Nc)[0] == 2 and (C + 15) // 16 >= 32
    check(Yh, Yref, A, L, variant=36)


@pytest.mark.parametrize("M,C,Nb,p,Nc", [(512, 64, 4, 60, 13000), (256, 256, 4, 70, 12900), (1024, 48, 2, 50, 6500)])
def test_spmm_tile_widths_in_steps_of_16(env, M, C, Nb, p, Nc):
    """Where every CTA pair gets one tile, the narrowest width that still fits one round is taken, in steps of 16 columns
    (the MMA's step): each CTA then holds a number of columns that is no multiple of 16, its last 64-column atom is
    partly used, and the epilogue's 16-column units no longer pair up."""
    torch, ubp = env
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    L = ubp_synth.make_layer("t", M, C, Nb, p, 7 * M + C, Nc=Nc, x_dist="normal", relu=True)
    Yh, Yref, A, plan = run_spmm(env, L, 34 + {2: 1, 4: 2}[Nb])
    kernel, rows, cols = plan.tile_choice(Nc)
    assert kernel == 2
    if sms == 148:
        assert cols % 32 == 16, (rows, cols)
    check(Yh, Yref, A, L, variant=36)


def test_tensor_core_variant_ragged_unaligned_and_auto(env):
    torch, ubp = env
    # ragged last strip on the fast path, then operands the fast path cannot take (falls back to the embedded
    # sparse plan: fp32 arithmetic, so the tighter bound holds)
    L = ubp_synth.make_layer("t", 200, 150, 4, 60, 777, Nc=130, x_dist="normal")
    check(*run_spmm(env, L, 32, pad=2)[:3], L, tensor_core=True)
    check(*run_spmm(env, L, 36, pad=2)[:3], L, variant=36)          # the same through the bf16-product kernel
    check(*run_spmm(env, L, 32, pad=0, misalign=1)[:3], L)
    check(*run_spmm(env, L, 36, pad=0, misalign=1)[:3], L)
    L2 = ubp_synth.make_layer("t", 200, 150, 4, 60, 778, Nc=131, x_dist="normal")
    check(*run_spmm(env, L2, 32)[:3], L2)
    # the automatic choice: dense-enough layers run on tensor cores, very sparse or small ones do not
    dense = ubp_synth.make_layer("t", 256, 256, 4, 70, 779, Nc=512)
    sparse = ubp_synth.make_layer("t", 256, 256, 4, 98, 780, Nc=512)
    small = ubp_synth.make_layer("t", 64, 32, 4, 50, 781, Nc=512)
    pv = lambda l: ubp.Plan(ubp.ubp_pack(l.W, l.mask, l.Nb)).variant
    assert pv(dense) == 36 and pv(sparse) == 14 and pv(small) == 50      # 36 = 32 with bf16 products (more than 128 rows)
    # bitwise reproducible run to run
    plan = ubp.Plan(ubp.ubp_pack(dense.W, dense.mask, 4))
    X = torch.from_numpy(dense.X).cuda()
    assert torch.equal(ubp.ubp_spmm(plan, X).clone(), ubp.ubp_spmm(plan, X))


@pytest.mark.parametrize("Nc,pad,misalign", [(130, 2, 0), (131, 1, 0), (1, 3, 0), (3, 1, 0), (257, 3, 0),
                                              (130, 0, 0), (255, 0, 0), (256, 0, 1), (64, 0, 3)])
def test_spmm_ragged_and_unaligned(env, Nc, pad, misalign):
    """pad > 0 with (Nc + pad) % 4 == 0 keeps the fast path with a ragged last strip; pad == 0 with odd Nc or a
    misaligned base pointer takes the slower kernel."""
    L = ubp_synth.make_layer("t", 70, 50, 4, 60, 4242 + Nc, Nc=Nc, x_dist="normal")
    Yh, Yref, A, _ = run_spmm(env, L, 0, pad=pad, misalign=misalign)
    check(Yh, Yref, A, L)


def test_spmm_empty_and_degenerate(env):
    torch, ubp = env
    L = ubp_synth.make_layer("t", 32, 16, 4, 100, 5, Nc=64)           # no block kept at all
    assert L.m == 0
    Yh, Yref, A, plan = run_spmm(env, L, relu=False)
    assert np.array_equal(Yh, np.broadcast_to(L.bias[:, None], Yh.shape))
    # zero columns: no launch, no error
    out = ubp.ubp_spmm(plan, torch.zeros((16, 0), device="cuda"))
    assert out.shape == (32, 0)
    # no bias, no relu
    L2 = ubp_synth.make_layer("t", 48, 24, 4, 50, 6, Nc=128, bias=False, relu=False)
    check(*run_spmm(env, L2)[:3], L2)
    # Nb == M: one possible start row
    L3 = ubp_synth.make_layer("t", 8, 40, 8, 50, 7, Nc=128)
    check(*run_spmm(env, L3)[:3], L3)


def test_spmm_bad_arguments(env):
    torch, ubp = env
    L = ubp_synth.make_layer("t", 32, 16, 4, 50, 5, Nc=64)
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, 4))
    lib = ubp.load()
    import ctypes as C
    X = torch.zeros((16, 64), device="cuda"); Y = torch.zeros((32, 64), device="cuda")
    vp = lambda t: C.c_void_p(t.data_ptr())
    assert lib.ubp_spmm(plan.handle, None, 64, 64, None, 0, vp(Y), 64, None) == -1
    assert lib.ubp_spmm(plan.handle, vp(X), 32, 64, None, 0, vp(Y), 64, None) == -1      # ldx < Nc
    assert lib.ubp_spmm(plan.handle, vp(X), 64, -1, None, 0, vp(Y), 64, None) == -1
    assert lib.ubp_spmm(None, vp(X), 64, 64, None, 0, vp(Y), 64, None) == -1
    assert lib.ubp_conv3x3_implicit(plan.handle, vp(X), 1, 8, 8, 64, 64, None, 0, vp(Y), 64, 64, None) == -1  # R != 9
    torch.cuda.synchronize()


def test_spmm_is_bitwise_reproducible(env):
    torch, ubp = env
    L = ubp_synth.make_layer("t", 256, 256, 4, 70, 99, Nc=1024)
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, 4), 14)          # sparse kernel
    X = torch.from_numpy(L.X).cuda(); b = torch.from_numpy(L.bias).cuda()
    Y1 = ubp.ubp_spmm(plan, X, b, True).clone()
    Y2 = ubp.ubp_spmm(plan, X, b, True)
    assert torch.equal(Y1, Y2)
    # the slower kernel sums in the same order: identical bits
    xb = torch.zeros(256 * 1024 + 1, device="cuda")
    Xm = xb[1:].view(256, 1024); Xm.copy_(X)
    Y3 = ubp.ubp_spmm(plan, Xm, b, True)
    assert torch.equal(Y1, Y3)


def test_fc64_config(env):
    L = ubp_synth.config_layers("fc64")[0]
    Yh, Yref, A, _ = run_spmm(env, L)
    check(Yh, Yref, A, L)


def test_mbv1_pw512_config_full(env):
    """The benchmark workload at full size, every output compared."""
    L = ubp_synth.config_layers("mbv1_pw512")[0]
    assert (L.M, L.C, L.Nc, L.m) == (512, 512, 6272, 19660)
    torch, ubp = env
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert blob == oracle.pack(L.W, L.mask, L.Nb)
    plan = ubp.Plan(blob)
    X = torch.from_numpy(L.X).cuda()                       # [C][B][H][W], channel-major
    Y = ubp.ubp_conv1x1(plan, X, torch.from_numpy(L.bias).cuda(), True, layout="CNHW")
    plan.check()
    Yref, A = oracle.masked_matmul(L.W, L.mask, L.X.reshape(L.C, -1), L.bias, relu=True)
    check(Y.cpu().numpy().reshape(L.M, -1), Yref, A, L, variant=plan.variant)
    # and the sparse kernel on the same layer
    plan_s = ubp.Plan(blob, 14)
    Ys = ubp.ubp_conv1x1(plan_s, X, torch.from_numpy(L.bias).cuda(), True, layout="CNHW")
    plan_s.check()
    check(Ys.cpu().numpy().reshape(L.M, -1), Yref, A, L)


def test_conv1x1_nchw_matches_cnhw(env):
    torch, ubp = env
    L = ubp_synth.make_layer("t", 96, 64, 4, 70, 31, B=3, H=14, Wd=14)
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, 4))
    b = torch.from_numpy(L.bias).cuda()
    Xc = torch.from_numpy(L.X).cuda()
    Yc = ubp.ubp_conv1x1(plan, Xc, b, True, layout="CNHW")
    Xn = Xc.permute(1, 0, 2, 3).contiguous()
    Yn = ubp.ubp_conv1x1(plan, Xn, b, True, layout="NCHW")
    assert torch.equal(Yn.permute(1, 0, 2, 3), Yc)
    Yref, A = oracle.masked_matmul(L.W, L.mask, L.X.reshape(L.C, -1), L.bias, relu=True)
    check(Yc.cpu().numpy().reshape(L.M, -1), Yref, A, L)
    # 7x7 planes: 196-byte rows, not 16-byte aligned per image -> slower kernel, same answer
    L7 = ubp_synth.make_layer("t", 64, 32, 4, 70, 32, B=2, H=7, Wd=7)
    p7 = ubp.Plan(ubp.ubp_pack(L7.W, L7.mask, 4))
    X7 = torch.from_numpy(L7.X).cuda().permute(1, 0, 2, 3).contiguous()
    Y7 = ubp.ubp_conv1x1(p7, X7, None, False, layout="NCHW").permute(1, 0, 2, 3).contiguous()
    Yref, A = oracle.masked_matmul(L7.W, L7.mask, L7.X.reshape(L7.C, -1), None, relu=False)
    check(Y7.cpu().numpy().reshape(L7.M, -1), Yref, A, L7)


@pytest.mark.parametrize("nb,sp,variant", [(2, 50, 0), (4, 70, 0), (8, 80, 0), (16, 90, 0), (4, 70, 14), (2, 50, 15),
                                           (16, 90, 16), (4, 95, 0), (4, 95, 14)])
def test_sweep_config_sampled(env, nb, sp, variant):
    """Full-size sweep point (M = K = 2048, Nc = 8192): sampled outputs against the oracle one by one, for the
    automatically chosen kernel and for the sparse kernel."""
    torch, ubp = env
    L = ubp_synth.config_layers("sweep", Nb=nb, sparsity_pct=sp)[0]
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert blob == oracle.pack(L.W, L.mask, L.Nb)
    plan = ubp.Plan(blob, variant)
    Y = ubp.ubp_spmm(plan, torch.from_numpy(L.X).cuda()).cpu().numpy()
    plan.check()
    rng = np.random.default_rng(nb * 100 + sp)
    so = np.concatenate([rng.integers(0, L.M, 4000), [0, L.M - 1, 0, L.M - 1]])
    sn = np.concatenate([rng.integers(0, L.Nc, 4000), [0, 0, L.Nc - 1, L.Nc - 1]])
    ys, as_ = oracle.masked_matmul_samples(L.W, L.mask, L.X, so, sn)
    err = scaled_error(Y[so, sn], ys, as_)
    n = terms_per_output(L) + 2
    assert err <= TOL and err <= arith_bound(L, plan.variant)
    # whole rows too (a panel's first / last row and one in the middle)
    for o in (0, 15, 16, 1000, L.M - 1):
        sn2 = np.arange(L.Nc)
        ys, as_ = oracle.masked_matmul_samples(L.W, L.mask, L.X, np.full(L.Nc, o), sn2)
        assert scaled_error(Y[o], ys, as_) <= TOL


def test_bf16_product_variant_few_terms_per_output(env):
    """Where the split products' error cannot average out: 98 % sparsity (most outputs are one or two products) and
    operands of magnitude >= 1 (no small values to hide behind). The bf16-product kernel must still be inside its worst-case
    bound 3 * 2^-16 (+ accumulation), hence inside the 1e-4 gate; the TF32-product kernel inside 2^-18."""
    torch, ubp = env
    L = ubp_synth.make_layer("t", 256, 256, 4, 98, 4321, Nc=1024, w_dist="uniform", x_dist="normal", relu=False)
    L.W[:] = np.abs(L.W) + 1.0
    L.X[:] = np.abs(L.X) + 1.0
    assert terms_per_output(L) <= 16
    for variant in (36, 32):
        Yh, Yref, A, plan = run_spmm(env, L, variant)
        assert plan.variant == variant and plan.tile_choice(1024)[0] == 2
        err = check(Yh, Yref, A, L, variant=variant)
        assert err <= (3 * 2.0 ** -16 + 2.0 ** -20 if variant == 36 else 2.0 ** -18)


def test_two_cta_kernel_padded_rows_and_repeated_launches(env):
    """The two-CTA tensor-core kernel with a leading dimension larger than the column count, and forty launches
    in a row on a layer with many column tiles and few chunks (several waves of CTA pairs; the copies of different
    chunks land out of order under load): every launch must finish with a clean status word and the same result."""
    torch, ubp = env
    L = ubp_synth.make_layer("t", 256, 64, 4, 60, 4242, Nc=512, x_dist="normal")
    check(*run_spmm(env, L, 32, pad=4)[:3], L, tensor_core=True)
    check(*run_spmm(env, L, 36, pad=4)[:3], L, variant=36)
    L = ubp_synth.make_layer("t", 384, 1040, 4, 70, 4243, Nc=260, x_dist="normal")   # 65 chunks: two per stage, odd count
    check(*run_spmm(env, L, 36, pad=0)[:3], L, variant=36)
    L = ubp_synth.config_layers("mbv1_chain", batch=64)[4]          # 256 -> 256 channels at 28 x 28: 50176 columns
    for variant in (32, 36):
        _repeated_launches(env, L, variant)


def _repeated_launches(env, L, variant):
    torch, ubp = env
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), variant)
    assert plan.tile_choice(L.Nc)[0] == 2                            # the CTA-pair kernel is what runs here
    X = torch.from_numpy(L.X).cuda().reshape(L.C, -1)
    bias = torch.from_numpy(L.bias).cuda()
    flush = torch.empty(192 << 20, dtype=torch.uint8, device="cuda")
    Y0 = ubp.ubp_spmm(plan, X, bias, True).clone()
    plan.check()
    Y = torch.empty_like(Y0)
    for i in range(40):
        if i % 2:
            flush.zero_()
        ubp.ubp_spmm(plan, X, bias, True, out=Y)
    plan.check()
    assert torch.equal(Y, Y0)
    Yh = Y.cpu().numpy()
    X2 = L.X.reshape(L.C, -1)
    rng = np.random.default_rng(5)
    so = rng.integers(0, L.M, 5000); sn = rng.integers(0, X2.shape[1], 5000)
    ys, as_ = oracle.masked_matmul_samples(L.W, L.mask, X2, so, sn, L.bias, relu=True)
    assert scaled_error(Yh[so, sn], ys, as_) <= TOL


@pytest.mark.parametrize("li", [0, 1, 3, 4, 5, 6, 11, 12])
def test_mbv1_chain_layers_sampled(env, li):
    torch, ubp = env
    L = ubp_synth.config_layers("mbv1_chain", batch=8 if li < 2 else 64)[li]
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb))
    Y = ubp.ubp_conv1x1(plan, torch.from_numpy(L.X).cuda(), torch.from_numpy(L.bias).cuda(), True)
    plan.check()
    Y = Y.cpu().numpy().reshape(L.M, -1)
    X2 = L.X.reshape(L.C, -1)
    rng = np.random.default_rng(li)
    so = rng.integers(0, L.M, 5000); sn = rng.integers(0, X2.shape[1], 5000)
    sn[:4] = [0, X2.shape[1] - 1, X2.shape[1] - 2, 1]
    ys, as_ = oracle.masked_matmul_samples(L.W, L.mask, X2, so, sn, L.bias, relu=True)
    assert scaled_error(Y[so, sn], ys, as_) <= TOL


# ------------------------------------------------------------------ 3x3
@pytest.mark.parametrize("M,C,Nb,p,B,H,Wd", [(16, 8, 4, 50, 2, 6, 5), (40, 20, 8, 60, 3, 14, 14), (24, 18, 2, 50, 1, 7, 9),
                                              (30, 10, 6, 40, 2, 4, 4), (17, 9, 1, 60, 2, 3, 5), (32, 40, 16, 50, 1, 8, 8)])
def test_conv3x3_small(env, M, C, Nb, p, B, H, Wd):
    torch, ubp = env
    L = ubp_synth.make_layer("c", M, C, Nb, p, 7 * M + C, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
    blob = ubp.ubp_pack(L.W, L.mask, Nb)
    assert blob == oracle.pack(L.W, L.mask, Nb)
    plan = ubp.Plan(blob)
    b = torch.from_numpy(L.bias).cuda()
    Y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), b, True, layout="CNHW")
    Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
    check(Y.cpu().numpy(), Yref, A, L)
    Yn = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda().permute(1, 0, 2, 3).contiguous(), b, True, layout="NCHW")
    assert torch.equal(Yn.permute(1, 0, 2, 3), Y)


@pytest.mark.parametrize("M,C,Nb,p,B,H,Wd,variant", [(128, 16, 8, 50, 2, 14, 14, 0), (256, 32, 4, 60, 3, 7, 9, 0),
                                                      (130, 20, 2, 50, 2, 5, 6, 42), (200, 24, 1, 70, 1, 8, 8, 43),
                                                      (128, 40, 16, 50, 5, 6, 6, 40), (64, 16, 8, 50, 2, 6, 6, 40),
                                                      # more than 128 rows and a multiple of 16 channels: CTA pairs.
                                                      # Ragged last row pair, column counts that are no multiple
                                                      # of 32, wide images (larger halo), several tiles per pair
                                                      (300, 48, 4, 60, 2, 14, 14, 41), (256, 16, 8, 50, 1, 28, 28, 40),
                                                      (260, 32, 2, 50, 3, 13, 11, 42), (512, 64, 4, 70, 7, 14, 14, 41),
                                                      (256, 32, 4, 60, 1, 9, 60, 41)])
def test_conv3x3_tensor_core_variant(env, M, C, Nb, p, B, H, Wd, variant):
    """3x3 as an implicit GEMM on tensor cores (variants 40..43; chosen automatically for dense-enough layers)."""
    torch, ubp = env
    L = ubp_synth.make_layer("c", M, C, Nb, p, 11 * M + C, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), variant)
    assert plan.variant >= 40
    b = torch.from_numpy(L.bias).cuda()
    if M > 128 and C % 16 == 0:
        assert plan.tile_choice(B * H * Wd, Wd)[0] == 2
    Y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), b, True, layout="CNHW")
    plan.check()
    Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
    check(Y.cpu().numpy(), Yref, A, L, variant=plan.variant)
    if plan.variant < 44 and M > 128:    # the same layer through the TF32 / the bf16 form explicitly (per-tap kernels)
        for v in (plan.variant, plan.variant + 4):
            pv = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), v)
            Yv = ubp.ubp_conv3x3_implicit(pv, torch.from_numpy(L.X).cuda(), b, True, layout="CNHW")
            pv.check()
            check(Yv.cpu().numpy(), Yref, A, L, variant=v)
    # NCHW output is not one [M][B*H*W] matrix: served by the plain kernel on the embedded sparse plan
    Yn = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda().permute(1, 0, 2, 3).contiguous(), b, True, layout="NCHW")
    check(Yn.permute(1, 0, 2, 3).contiguous().cpu().numpy(), Yref, A, L)


@pytest.mark.parametrize("M,C,Nb,p,B,H,Wd", [(256, 32, 4, 60, 3, 7, 9), (300, 48, 4, 60, 2, 14, 14), (256, 16, 8, 50, 1, 28, 28),
                                              (260, 32, 2, 50, 3, 13, 11), (512, 64, 4, 70, 7, 14, 14), (256, 32, 4, 60, 1, 9, 60),
                                              (256, 32, 4, 60, 2, 5, 80), (384, 160, 8, 80, 40, 14, 14), (256, 16, 1, 50, 150, 3, 3),
                                              (256, 32, 4, 100, 2, 6, 6)])
def test_conv3x3_taps_as_operand_shifts(env, M, C, Nb, p, B, H, Wd):
    """The 3x3 kernel that computes on the zero-padded pixel grid and takes the nine taps as shifts of one staged
    operand (variants 64..67, the automatic choice): small and wide images (up to 80 pixels: the halo grows with the
    width), image sizes that put tile boundaries anywhere in a row, batches that give a pair several tiles, a layer
    with no block kept. Against the oracle's direct convolution, at the bound of the bf16-product arithmetic."""
    torch, ubp = env
    L = ubp_synth.make_layer("c", M, C, Nb, p, 17 * M + C + Wd, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), 65 if p == 100 else 0)       # nothing kept: not the automatic choice
    assert 64 <= plan.variant <= 67
    kern, rows, cols = plan.tile_choice_conv(B, H, Wd)
    assert kern == 4 and rows == 256 and cols % 16 == 0 and cols // 2 + 2 * (Wd + 3) <= 256
    b = torch.from_numpy(L.bias).cuda()
    ybuf = torch.full((M, B, H, Wd), float("nan"), dtype=torch.float32, device="cuda")
    Y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), b, True, out=ybuf)
    plan.check()
    Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
    check(Y.cpu().numpy(), Yref, A, L, variant=plan.variant)
    # the per-tap kernel on the same layer gives the same result to the same bound; and twice the same bits
    Y2 = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), b, True)
    assert torch.equal(Y, Y2)
    pold = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), plan.variant - 20)
    assert pold.tile_choice_conv(B, H, Wd)[0] in (1, 2)
    check(ubp.ubp_conv3x3_implicit(pold, torch.from_numpy(L.X).cuda(), b, True).cpu().numpy(), Yref, A, L, variant=pold.variant)


def test_r50_3x3_config_sampled(env):
    torch, ubp = env
    L = ubp_synth.config_layers("r50_3x3")[0]
    assert (L.M, L.C, L.m, L.B) == (256, 256, 1638, 64)
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert blob == oracle.pack(L.W, L.mask, L.Nb)
    plan = ubp.Plan(blob)
    Y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), torch.from_numpy(L.bias).cuda(), True).cpu().numpy()
    rng = np.random.default_rng(3)
    n = 6000
    sb = rng.integers(0, L.B, n); so = rng.integers(0, L.M, n); sy = rng.integers(0, 14, n); sx = rng.integers(0, 14, n)
    sy[:8] = [0, 0, 13, 13, 0, 13, 7, 7]; sx[:8] = [0, 13, 0, 13, 7, 7, 0, 13]          # corners and edges
    ys, as_ = oracle.masked_conv3x3_samples(L.W, L.mask, L.X, sb, so, sy, sx, L.bias, relu=True)
    err = scaled_error(Y[so, sb, sy, sx], ys, as_)
    n_terms = terms_per_output(L) + 2
    assert err <= TOL and err <= arith_bound(L, plan.variant)
    # the plain 3x3 kernel on the same layer
    plan_s = ubp.Plan(blob, 20)
    Ys = ubp.ubp_conv3x3_implicit(plan_s, torch.from_numpy(L.X).cuda(), torch.from_numpy(L.bias).cuda(), True).cpu().numpy()
    assert scaled_error(Ys[so, sb, sy, sx], ys, as_) <= n_terms * 2.0 ** -24


def test_bounded_wait_is_reported_not_hung(env):
    """A wait that can never complete returns after its limit and is reported through the plan's status word; the
    context stays usable and the next product is correct."""
    import time
    torch, ubp = env
    L = ubp_synth.make_layer("t", 64, 32, 4, 50, 91, Nc=256)
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, 4))
    plan.check()
    t0 = time.perf_counter()
    plan.selftest_bounded_wait(limit_us=20000)
    with pytest.raises(ubp.UbpError) as e:
        plan.check()
    assert e.value.code == -7 and time.perf_counter() - t0 < 5.0
    plan.clear_status()
    plan.check()
    Yh, Yref, A, _ = run_spmm(env, L)
    check(Yh, Yref, A, L)


def test_launches_can_be_captured_in_a_cuda_graph(env):
    """Two layers chained through a CUDA graph (as the 13-layer benchmark does) give the eager results."""
    torch, ubp = env
    L1 = ubp_synth.make_layer("a", 256, 256, 4, 70, 92, Nc=1024)            # tensor-core kernel
    L2 = ubp_synth.make_layer("b", 64, 256, 4, 90, 93, Nc=1024)             # sparse kernel
    p1 = ubp.Plan(ubp.ubp_pack(L1.W, L1.mask, 4)); p2 = ubp.Plan(ubp.ubp_pack(L2.W, L2.mask, 4))
    X = torch.from_numpy(L1.X).cuda()
    b1 = torch.from_numpy(L1.bias).cuda(); b2 = torch.from_numpy(L2.bias).cuda()
    Y1 = torch.empty((256, 1024), device="cuda"); Y2 = torch.empty((64, 1024), device="cuda")
    ubp.ubp_spmm(p1, X, b1, True, out=Y1); ubp.ubp_spmm(p2, Y1, b2, True, out=Y2)   # eager (also first-launch set-up)
    want = Y2.clone()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream()):
        ubp.ubp_spmm(p1, X, b1, True, out=Y1)
        ubp.ubp_spmm(p2, Y1, b2, True, out=Y2)
    Y2.zero_()
    g.replay(); g.replay()
    torch.cuda.synchronize()
    p1.check(); p2.check()
    assert torch.equal(Y2, want)
    Yref1, _ = oracle.masked_matmul(L1.W, L1.mask, L1.X, L1.bias, relu=True)
    Yref2, A2 = oracle.masked_matmul(L2.W, L2.mask, Yref1.astype(np.float32), L2.bias, relu=True)
    assert scaled_error(Y2.cpu().numpy(), Yref2, A2) <= TOL


def test_bottleneck_trio_chained_through_fused_epilogues(env):
    """A ResNet-50-shaped bottleneck (1x1 1024->256 + ReLU, 3x3 256->256 + ReLU, 1x1 256->1024), each layer reading
    the previous layer's output tensor, eagerly and replayed from one CUDA graph. Every layer is checked against the
    oracle evaluated on the activations that layer actually read."""
    torch, ubp = env
    layers = ubp_synth.config_layers("r50_bottleneck", batch=4)
    x = torch.from_numpy(layers[0].X).cuda()
    plans, outs, ins, runs = [], [], [], []
    for L in layers:
        plan = ubp.Plan(ubp.pack_ubp(L.W, L.mask, L.Nb))
        bias = torch.from_numpy(L.bias).cuda()
        y = torch.empty((L.M, L.B, L.H, L.Wd), dtype=torch.float32, device="cuda")
        fn = ubp.ubp_conv3x3_implicit if L.R == 9 else ubp.ubp_conv1x1
        runs.append(lambda fn=fn, plan=plan, x=x, bias=bias, relu=L.relu, y=y: fn(plan, x, bias, relu, out=y))
        plans.append(plan); ins.append(x); outs.append(y)
        x = y
    for r in runs:
        r()
    torch.cuda.synchronize()
    eager = [y.cpu().numpy().copy() for y in outs]
    for L, plan, xin, y in zip(layers, plans, ins, eager):
        plan.check()
        xh = xin.cpu().numpy()
        if L.R == 9:
            Yref, A = oracle.masked_conv3x3(L.W, L.mask, xh, L.bias, relu=L.relu)
        else:
            Yref, A = oracle.masked_matmul(L.W, L.mask, xh.reshape(L.C, -1), L.bias, relu=L.relu)
            Yref, A = Yref.reshape(y.shape), A.reshape(y.shape)
        assert scaled_error(y, Yref, A) <= 1e-4
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    for y in outs:
        y.zero_()
    with torch.cuda.graph(g, stream=s):
        for r in runs:
            r()
    g.replay()
    torch.cuda.synchronize()
    for y, e in zip(outs, eager):
        assert np.array_equal(y.cpu().numpy(), e)


@pytest.mark.parametrize("layout", ["CNHW", "NCHW"])
@pytest.mark.parametrize("H,Wd", [(14, 14), (7, 9)])
def test_stride_two_convolutions(env, layout, H, Wd):
    """Downsampling layers: 1x1 stride 2 reads every other pixel of every other row; 3x3 stride 2 / pad 1 is the
    stride-1 result at those pixels. Both against the oracle's stride-1 definitions, subsampled."""
    torch, ubp = env
    B = 3
    L1 = ubp_synth.make_layer("s2_pw", 96, 64, 4, 70, 801, B=B, H=H, Wd=Wd)
    L3 = ubp_synth.make_layer("s2_3x3", 64, 32, 8, 75, 802, B=B, H=H, Wd=Wd, R=9)
    for L in (L1, L3):
        plan = ubp.Plan(ubp.pack_ubp(L.W, L.mask, L.Nb))
        x = torch.from_numpy(L.X).cuda()                       # [C][B][H][W]
        if layout == "NCHW":
            x = x.permute(1, 0, 2, 3).contiguous()
        bias = torch.from_numpy(L.bias).cuda()
        fn = ubp.ubp_conv3x3_implicit if L.R == 9 else ubp.ubp_conv1x1
        y = fn(plan, x, bias, True, layout=layout, stride=2)
        torch.cuda.synchronize()
        plan.check()
        y = y.cpu().numpy()
        if layout == "NCHW":
            y = y.transpose(1, 0, 2, 3)
        if L.R == 9:
            Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
            Yref, A = Yref[:, :, ::2, ::2], A[:, :, ::2, ::2]
        else:
            xs = np.ascontiguousarray(L.X[:, :, ::2, ::2])
            Yref, A = oracle.masked_matmul(L.W, L.mask, xs.reshape(L.C, -1), L.bias, relu=True)
            Yref, A = Yref.reshape(L.M, B, *xs.shape[2:]), A.reshape(L.M, B, *xs.shape[2:])
        assert y.shape == Yref.shape
        assert scaled_error(y, Yref, A) <= 1e-4


@pytest.mark.parametrize("M,C,Nb,p,B,H,Wd", [(256, 64, 4, 70, 5, 28, 28), (1024, 512, 4, 80, 6, 28, 28), (512, 96, 2, 60, 9, 56, 56),
                                             (128, 80, 4, 50, 4, 28, 28), (300, 40, 8, 60, 3, 8, 16), (256, 520, 4, 75, 7, 12, 20),
                                             (260, 64, 4, 70, 2, 14, 14), (256, 64, 4, 70, 3, 28, 26)])
def test_stride_two_1x1_without_gather(env, M, C, Nb, p, B, H, Wd):
    """1x1 with stride 2 under a bf16 tensor-core plan, channel-major input with even H and W a multiple of 4: the
    CTA-pair kernel reads the full-resolution input itself (boxes of the even rows, every other pixel in the split pass),
    tiles of whole output rows; plain, stacked and duplicated-row tiles, one or two chunks per stage, a ragged last tile.
    The last two shapes (W no multiple of 4) take the gathered copy instead. Against the oracle on the subsampled input;
    the scratch buffer must stay untouched on the direct path."""
    torch, ubp = env
    L = ubp_synth.make_layer("s2", M, C, Nb, p, 9 * M + C + Wd, B=B, H=H, Wd=Wd, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), 34 + {2: 1, 4: 2, 8: 3}[Nb])
    x = torch.from_numpy(L.X).cuda()                           # [C][B][H][W]
    Ho, Wo = H // 2, Wd // 2
    scratch = torch.full((C * B * Ho * Wo,), float("nan"), dtype=torch.float32, device="cuda")
    y = ubp.ubp_conv1x1(plan, x, torch.from_numpy(L.bias).cuda(), True, stride=2, scratch=scratch)
    torch.cuda.synchronize()
    plan.check()
    direct = Wd % 4 == 0
    assert bool(torch.isnan(scratch).all()) == direct
    xs = np.ascontiguousarray(L.X[:, :, ::2, ::2])
    Yref, A = oracle.masked_matmul(L.W, L.mask, xs.reshape(C, -1), L.bias, relu=True)
    yh = y.cpu().numpy().reshape(M, -1)
    assert yh.shape == Yref.shape and np.isfinite(yh).all()
    assert scaled_error(yh, Yref, A) <= 1e-4


@pytest.mark.parametrize("M,C,Nb,p,B,H,Wd,stride", [(128, 32, 4, 60, 3, 14, 14, 2), (256, 48, 8, 70, 2, 28, 28, 2),
                                                      (200, 20, 4, 50, 2, 7, 9, 2), (130, 16, 2, 50, 1, 13, 12, 3),
                                                      (256, 64, 4, 80, 4, 8, 8, 2), (300, 32, 4, 60, 5, 7, 7, 2),
                                                      (256, 32, 8, 50, 3, 15, 13, 2), (512, 128, 4, 80, 16, 28, 28, 2)])
def test_strided_conv3x3_on_tensor_cores(env, M, C, Nb, p, B, H, Wd, stride):
    """Downsampling 3x3 with a tensor-core plan. Stride 2, more than 128 rows, channels a multiple of 16: the four
    phase planes of the input are gathered into scratch and the padded-grid CTA-pair kernel runs on them (every tap a
    shift of 0 or -1 of one plane; odd image sizes leave the last row / column of the odd planes zero). Otherwise the
    one-CTA implicit-GEMM kernel, whose loaders gather the taps around input pixel (yo*stride, xo*stride). Against the
    oracle's stride-1 definition at those pixels."""
    torch, ubp = env
    L = ubp_synth.make_layer("s3", M, C, Nb, p, 13 * M + C, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb))
    assert 64 <= plan.variant <= 67
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    kern = plan.tile_choice_conv(B, H, Wd, stride)[0]
    assert kern == (4 if (stride == 2 and M > 128 and C % 16 == 0) else 1)
    bias = torch.from_numpy(L.bias).cuda()
    ybuf = torch.full((M, B, Ho, Wo), float("nan"), dtype=torch.float32, device="cuda")
    y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), bias, True, stride=stride, out=ybuf)
    plan.check()
    Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
    Yref, A = Yref[:, :, ::stride, ::stride], A[:, :, ::stride, ::stride]
    yh = y.cpu().numpy()
    assert yh.shape == Yref.shape == (M, B, Ho, Wo) and np.isfinite(yh).all()
    err = scaled_error(yh, Yref, A)
    assert err <= 1e-4 and err <= arith_bound(L, plan.variant if kern == 4 else 40)   # bf16 pieces / three TF32 products
    # without scratch the C entry point keeps its earlier route (one-CTA kernel): same result to the same gate
    lib = ubp.load()
    import ctypes as Ct
    y2 = torch.empty_like(ybuf)
    x = torch.from_numpy(L.X).cuda()
    rc = lib.ubp_conv3x3_strided(plan.handle, Ct.c_void_p(x.data_ptr()), B, H, Wd, stride, x.stride(1), x.stride(0),
                                 Ct.c_void_p(bias.data_ptr()), 1, Ct.c_void_p(y2.data_ptr()), y2.stride(1), y2.stride(0), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert scaled_error(y2.cpu().numpy(), Yref, A) <= 1e-4
    # the plain kernel on the same layer agrees to fp32 accuracy
    ys = ubp.ubp_conv3x3_implicit(ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), 20 if Nb % 8 == 0 else (21 if Nb % 4 == 0 else 22)),
                                  torch.from_numpy(L.X).cuda(), bias, True, stride=stride)
    assert scaled_error(ys.cpu().numpy(), Yref, A) <= (terms_per_output(L) + 2) * 2.0 ** -24


@pytest.mark.parametrize("M,Cin,B,p,Nc", [(256, 256, 4, 70, 1000), (192, 320, 8, 95, 520), (64, 96, 2, 50, 260)])
def test_kmajor_orientation_through_the_plan(env, M, Cin, B, p, Nc):
    """Blocks that run along the input channels of one output row: packed as the transposed layer, converted for
    the plan builder, run through ubp_spmm (tensor-core kernel at 70 %, sparse element-wise kernel at 95 %)."""
    torch, ubp = env
    Lt = ubp_synth.make_layer("kmajor", Cin, M, B, p, 900 + B, Nc=8, make_x=False)    # roles exchanged: [C][M]
    W = np.ascontiguousarray(Lt.W[:, :, 0].T)
    mask = np.ascontiguousarray(Lt.mask.T)
    rng = np.random.default_rng(5)
    X = rng.standard_normal((Cin, Nc)).astype(np.float32)
    bias = rng.standard_normal(M).astype(np.float32)
    plan = ubp.Plan(ubp.ubp_kmajor_to_plan_blob(ubp.ubp_pack_kmajor(W, mask, B)))
    assert plan.m == Lt.m * B and plan.Nb == 1
    Y = ubp.ubp_spmm(plan, torch.from_numpy(X).cuda(), torch.from_numpy(bias).cuda(), True)
    torch.cuda.synchronize()
    plan.check()
    Yref, A = oracle.masked_matmul(W, mask, X, bias, relu=True)
    assert scaled_error(Y.cpu().numpy(), Yref, A) <= 1e-4


def _kmajor_layer(M, Cin, B, p, Nc, seed):
    Lt = ubp_synth.make_layer("kmajor", Cin, M, B, p, seed, Nc=8, make_x=False)       # roles exchanged: [C][M]
    W = np.ascontiguousarray(Lt.W[:, :, 0].T)
    mask = np.ascontiguousarray(Lt.mask.T)
    rng = np.random.default_rng(seed)
    return W, mask, rng.standard_normal((Cin, Nc)).astype(np.float32), rng.standard_normal(M).astype(np.float32), Lt.m


@pytest.mark.parametrize("M,Cin,B,p,Nc,pad,misalign", [
    (256, 256, 4, 70, 1000, 0, 0), (192, 320, 8, 95, 520, 0, 0), (64, 96, 2, 50, 260, 0, 0), (100, 130, 16, 50, 516, 0, 0),
    (300, 70, 4, 80, 1028, 0, 0), (512, 512, 4, 90, 2048, 0, 0), (40, 200, 2, 60, 130, 2, 0), (40, 200, 8, 60, 131, 1, 0),
    (77, 64, 4, 50, 255, 0, 0), (77, 64, 4, 50, 256, 0, 1), (9, 48, 16, 34, 4, 0, 0),
])
def test_krun_sparse_kernel(env, M, Cin, B, p, Nc, pad, misalign):
    """The sparse kernel for the other orientation (variants 70..73): one plan entry, one channel index and B staged
    activation rows per run of B consecutive input channels of one output row. Against the definition (the oracle's
    dense masked product), through the staged kernel and, for operands it cannot take, the plain one; fp32 FMA, so the
    fp32 summation bound holds."""
    torch, ubp = env
    W, mask, X, bias, m = _kmajor_layer(M, Cin, B, p, Nc, 950 + B + M)
    kblob = ubp.ubp_pack_kmajor(W, mask, B)
    assert kblob == oracle.pack(np.ascontiguousarray(W.T), np.ascontiguousarray(mask.T), B)
    variant = {2: 70, 4: 71, 8: 72, 16: 73}[B]
    plan = ubp.Plan(kblob, variant, kmajor=True)
    assert (plan.variant, plan.M, plan.C, plan.Nb, plan.m) == (variant, M, Cin, B, m)
    assert plan.tile_choice(Nc)[0] == 0
    ld = Nc + pad
    xbuf = torch.zeros(Cin * ld + 8, dtype=torch.float32, device="cuda")
    Xd = xbuf[misalign:misalign + Cin * ld].view(Cin, ld)[:, :Nc]
    Xd.copy_(torch.from_numpy(X))
    ybuf = torch.full((M * ld + 8,), float("nan"), dtype=torch.float32, device="cuda")
    Yd = ybuf[misalign:misalign + M * ld].view(M, ld)[:, :Nc]
    ubp.ubp_spmm(plan, Xd, torch.from_numpy(bias).cuda(), True, out=Yd)
    plan.check()
    if pad:
        assert torch.isnan(ybuf[misalign:misalign + M * ld].view(M, ld)[:, Nc:]).all()
    Yref, A = oracle.masked_matmul(W, mask, X, bias, relu=True)
    Yh = Yd.cpu().numpy()
    assert np.isfinite(Yh).all()
    err = scaled_error(Yh, Yref, A)
    terms = int(mask.sum(axis=1).max()) + 2
    assert err <= 1e-4 and err <= terms * 2.0 ** -24 * 1.5          # pieces of a cut run add a few exact zeros
    # the automatic choice for this orientation: tensor-core kernel when dense and large enough, else this kernel
    auto = ubp.Plan(kblob, 0, kmajor=True)
    dense_enough = (100 - p) >= 3 and M >= 128 and Cin >= 64
    assert auto.variant == (34 if dense_enough else variant)
    Ya = ubp.ubp_spmm(auto, torch.from_numpy(X).cuda(), torch.from_numpy(bias).cuda(), True)
    auto.check()
    assert scaled_error(Ya.cpu().numpy(), Yref, A) <= 1e-4
