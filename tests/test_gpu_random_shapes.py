"""Seeded random layer shapes through the automatic variant and the bf16 tensor-core variants, against the oracle: odd
row / channel / column counts, padded leading dimensions, every block size, 20-97 % sparsity, images of 3 .. 29 pixels,
stride 1 and 2. What the hand-picked cases of test_gpu_parity.py might miss (tile choices change with the shape: plain,
stacked and duplicated-row tiles, one or several tiles per pair, every 3x3 kernel)."""
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
    return torch, ubp


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_1x1_layers(env, seed):
    torch, ubp = env
    rng = np.random.default_rng(seed)
    kernels = set()
    for it in range(40):
        Nb = int(rng.choice([1, 2, 4, 8, 16]))
        M = max(Nb, int(rng.choice([rng.integers(Nb, 130), rng.integers(128, 600), rng.choice([256, 512, 768, 1024, 1000, 520])])))
        C = int(rng.choice([rng.integers(1, 70), rng.integers(64, 300), rng.choice([64, 128, 256, 48])]))
        p = int(rng.integers(20, 98))
        Nc = int(rng.choice([rng.integers(1, 300), rng.integers(300, 6000), rng.choice([4096, 14208, 19201, 30003])]))
        if M * C * Nc > 2e9:
            Nc = max(1, int(2e9 // (M * C)))
        pad = int(rng.choice([0, 0, 0, 1, 2, 4]))
        variant = int(rng.choice([0, 0, 34 + {1: 0, 2: 1, 4: 2, 8: 3, 16: 3}[Nb]]))
        L = ubp_synth.make_layer("f", M, C, Nb, p, 100 * seed + it, Nc=Nc, x_dist="normal", relu=bool(it & 1))
        plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), variant)
        ld = Nc + pad
        xbuf = torch.zeros(C * ld, dtype=torch.float32, device="cuda")
        X = xbuf.view(C, ld)[:, :Nc]
        X.copy_(torch.from_numpy(L.X))
        ybuf = torch.full((M * ld,), float("nan"), dtype=torch.float32, device="cuda")
        Y = ybuf.view(M, ld)[:, :Nc]
        ubp.ubp_spmm(plan, X, torch.from_numpy(L.bias).cuda(), L.relu, out=Y)
        plan.check()
        what = (M, C, Nb, p, Nc, pad, plan.variant, plan.tile_choice(Nc))
        Yh = Y.cpu().numpy()
        assert np.isfinite(Yh).all(), what
        if pad:
            assert torch.isnan(ybuf.view(M, ld)[:, Nc:]).all(), what
        Yref, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias, relu=L.relu)
        assert scaled_error(Yh, Yref, A) <= TOL, what
        kernels.add(plan.tile_choice(Nc)[:2])
    assert len(kernels) >= 3                      # sparse kernel, plain pair tiles, stacked tiles ... all came up


@pytest.mark.parametrize("seed", [21, 22])
def test_random_3x3_layers(env, seed):
    torch, ubp = env
    rng = np.random.default_rng(seed)
    kernels = set()
    for it in range(40):
        Nb = int(rng.choice([1, 2, 4, 8]))
        M = int(rng.choice([rng.integers(max(Nb, 8), 130), rng.integers(129, 400), rng.choice([256, 512, 260])]))
        C = int(rng.choice([16, 32, 48, 64, 24, 20, 128]))
        p = int(rng.integers(30, 92))
        B, H, Wd = int(rng.integers(1, 9)), int(rng.integers(3, 30)), int(rng.integers(3, 30))
        stride = int(rng.choice([1, 1, 2]))
        variant = int(rng.choice([0, 0, 64 + {1: 3, 2: 2, 4: 1, 8: 0}[Nb]]))
        L = ubp_synth.make_layer("f", M, C, Nb, p, 100 * seed + it, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
        plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), variant)
        Y = ubp.ubp_conv3x3_implicit(plan, torch.from_numpy(L.X).cuda(), torch.from_numpy(L.bias).cuda(), True, stride=stride)
        plan.check()
        Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
        Yref, A = Yref[:, :, ::stride, ::stride], A[:, :, ::stride, ::stride]
        what = (M, C, Nb, p, B, H, Wd, stride, plan.variant, plan.tile_choice_conv(B, H, Wd, stride))
        Yh = Y.cpu().numpy()
        assert Yh.shape == Yref.shape and np.isfinite(Yh).all(), what
        assert scaled_error(Yh, Yref, A) <= TOL, what
        kernels.add(plan.tile_choice_conv(B, H, Wd, stride)[0])
    assert len(kernels) >= 3


@pytest.mark.parametrize("seed", [31])
def test_random_stride_two_1x1_layers(env, seed):
    """1x1 with stride 2 on random shapes and both layouts: whichever path the library takes (the CTA-pair kernel reading
    the full-resolution input itself, or the gathered copy first), against the oracle on the subsampled input."""
    torch, ubp = env
    rng = np.random.default_rng(seed)
    paths = set()
    for it in range(40):
        Nb = int(rng.choice([2, 4, 8]))
        M = max(Nb, int(rng.choice([rng.integers(16, 130), rng.integers(129, 600), rng.choice([256, 512, 1024, 768])])))
        C = int(rng.choice([rng.integers(16, 100), rng.integers(64, 300), rng.choice([512, 520, 64, 128])]))
        H = int(rng.choice([4, 8, 12, 14, 16, 28, 56, 7]))
        Wd = int(rng.choice([4, 8, 12, 16, 20, 28, 56, 14, 6]))
        B = int(rng.integers(1, 9))
        if M * C * B * H * Wd // 4 > 1.5e9:
            B = 1
        p = int(rng.integers(30, 95))
        relu = bool(it & 1)
        L = ubp_synth.make_layer("f", M, C, Nb, p, 100 * seed + it, B=B, H=H, Wd=Wd, x_dist="normal")
        plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, Nb), int(rng.choice([0, 34 + {2: 1, 4: 2, 8: 3}[Nb]])))
        layout = str(rng.choice(["CNHW", "NCHW"]))
        x = torch.from_numpy(L.X).cuda()
        if layout == "NCHW":
            x = x.permute(1, 0, 2, 3).contiguous()
        Ho, Wo = (H - 1) // 2 + 1, (Wd - 1) // 2 + 1
        scratch = torch.full((C * B * Ho * Wo,), float("nan"), dtype=torch.float32, device="cuda")
        y = ubp.ubp_conv1x1(plan, x, torch.from_numpy(L.bias).cuda(), relu, stride=2, scratch=scratch, layout=layout)
        torch.cuda.synchronize()
        plan.check()
        paths.add(bool(torch.isnan(scratch).all()))
        y = y.cpu().numpy()
        if layout == "NCHW":
            y = y.transpose(1, 0, 2, 3)
        xs = np.ascontiguousarray(L.X[:, :, ::2, ::2])
        Yref, A = oracle.masked_matmul(L.W, L.mask, xs.reshape(C, -1), L.bias, relu=relu)
        yh = y.reshape(M, -1)
        what = (M, C, Nb, p, B, H, Wd, layout, plan.variant)
        assert yh.shape == Yref.shape and np.isfinite(yh).all(), what
        assert scaled_error(yh, Yref, A) <= TOL, what
    assert paths == {True, False}                 # both the direct and the gathered path came up
