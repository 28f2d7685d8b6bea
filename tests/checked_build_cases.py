"""Cases for the checked build of the library (-DUBP_DEBUG): run as a script with UBP_B200_LIBRARY pointing at
libubp_b200_debug.so (tests/test_gpu_checked_build.py does that in a child process, because a process loads one build).

Every kernel family runs tiny and odd shapes; the results are compared with the oracle and the plan's status word must
stay clear (no index left its extent). Then one plan is damaged on the device in a way the checked build must notice:
an entry's channel index is set to the first channel BEYOND the staged tile (a value the ordinary build would also
survive: that row is the start of the plan group in the same pipeline stage), and the status word must report it.
Prints one line per case and "checked build ok" at the end.
"""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import oracle  # noqa: E402
import ubp_synth  # noqa: E402
import paper_2407_19644_b200 as ubp  # noqa: E402
from paper_2407_19644_b200 import binding  # noqa: E402
from helpers import scaled_error  # noqa: E402

TOL = 1e-4


def spmm_case(M, C, Nb, p, Nc, variant, pad=0, kmajor=False):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 7 * M + C, Nc=Nc, x_dist="normal", relu=(M % 2 == 0))
    if kmajor:
        Lt = ubp_synth.make_layer("t", C, M, Nb, p, 7 * M + C, Nc=8, make_x=False)        # roles exchanged: [C][M]
        W, mask = np.ascontiguousarray(Lt.W[:, :, 0].T), np.ascontiguousarray(Lt.mask.T)  # blocks along the input channels
        plan = ubp.Plan(ubp.ubp_pack_kmajor(W, mask, Nb), variant, kmajor=True)
        X = np.random.default_rng(3).standard_normal((C, Nc)).astype(np.float32)
        Y = ubp.ubp_spmm(plan, torch.from_numpy(X).cuda(), None, False)
        plan.check()
        Yref, A = oracle.masked_matmul(W, mask, X, None, relu=False)
        return scaled_error(Y.cpu().numpy(), Yref, A), plan.variant
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), variant)
    ld = Nc + pad
    xbuf = torch.zeros(L.C * ld, dtype=torch.float32, device="cuda")
    X = xbuf.view(L.C, ld)[:, :Nc]
    X.copy_(torch.from_numpy(L.X))
    ybuf = torch.full((L.M * ld,), float("nan"), dtype=torch.float32, device="cuda")
    Y = ybuf.view(L.M, ld)[:, :Nc]
    ubp.ubp_spmm(plan, X, torch.from_numpy(L.bias).cuda(), L.relu, out=Y)
    plan.check()
    if pad:
        assert torch.isnan(ybuf.view(L.M, ld)[:, Nc:]).all()
    Yref, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias, relu=L.relu)
    return scaled_error(Y.cpu().numpy(), Yref, A), plan.variant


def conv_case(M, C, Nb, p, B, H, Wd, variant, stride=1):
    L = ubp_synth.make_layer("t", M, C, Nb, p, 5 * M + C, B=B, H=H, Wd=Wd, R=9, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), variant)
    x = torch.from_numpy(L.X).cuda()
    Y = ubp.ubp_conv3x3_implicit(plan, x, torch.from_numpy(L.bias).cuda(), True, stride=stride)
    plan.check()
    Yref, A = oracle.masked_conv3x3(L.W, L.mask, L.X, L.bias, relu=True)
    Yref, A = Yref[:, :, ::stride, ::stride], A[:, :, ::stride, ::stride]     # stride s = the stride-1 result at those pixels
    return scaled_error(Y.cpu().numpy(), Yref, A), plan.variant


def s2_case(M, C, Nb, p, B, H, Wd):
    """1x1 with stride 2 read straight from the full-resolution input by the bf16 pair kernel."""
    L = ubp_synth.make_layer("t", M, C, Nb, p, 3 * M + C, B=B, H=H, Wd=Wd, x_dist="normal")
    plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), 36)
    Y = ubp.ubp_conv1x1(plan, torch.from_numpy(L.X).cuda(), torch.from_numpy(L.bias).cuda(), True, stride=2)
    plan.check()
    xs = np.ascontiguousarray(L.X[:, :, ::2, ::2])
    Yref, A = oracle.masked_matmul(L.W, L.mask, xs.reshape(C, -1), L.bias, relu=True)
    return scaled_error(Y.cpu().numpy().reshape(M, -1), Yref, A), plan.variant


def damaged_plan_is_reported():
    """Sparse kernel, one entry's channel index moved one past the staged tile: the checked build skips that panel's
    list and sets the status word; nothing else happens."""
    L = ubp_synth.make_layer("t", 128, 128, 4, 60, 99, Nc=512, x_dist="normal")
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    plan = ubp.Plan(blob, 14)
    img, geom = ubp.plan_image(blob, 14)
    nbk, P, KT, WR = geom["nbk"], geom["panel_rows"], geom["k_tile"], geom["WR"]
    F = P + nbk - 1
    fo_bytes = (2 * (F + 1) + 15) // 16 * 16
    tab = np.frombuffer(img, "<u4", geom["nkt"] * geom["NG"] + 1, 256)
    g0 = int(tab[0]) * 16
    poff = np.frombuffer(img, "<u4", WR + 1, g0)
    so = g0 + int(poff[0])
    n = int(np.frombuffer(img, "<u2", F + 1, so)[F])
    assert n > 0 and int(poff[WR]) >= 1024
    dev_off = plan._dev - plan.buffer.data_ptr() + so + fo_bytes          # jl[0] of panel 0, channel tile 0
    plan.buffer[dev_off:dev_off + 2] = torch.tensor([KT & 0xFF, KT >> 8], dtype=torch.uint8, device="cuda")
    ubp.ubp_spmm(plan, torch.from_numpy(L.X).cuda(), None, False)
    try:
        plan.check()
    except ubp.UbpError as e:
        return e.code
    return 0


def main():
    assert "debug" in os.path.basename(binding.lib_path()), binding.lib_path()
    cases = [
        ("sparse", lambda: spmm_case(64, 64, 4, 50, 256, 0)),
        ("sparse ragged", lambda: spmm_case(100, 70, 4, 60, 520, 3, pad=4)),
        ("sparse Nb=1", lambda: spmm_case(33, 20, 1, 50, 260, 0)),
        ("sparse Nb=3", lambda: spmm_case(37, 45, 3, 40, 132, 0)),
        ("sparse Nb=16", lambda: spmm_case(80, 40, 16, 50, 260, 0)),
        ("sparse tiny", lambda: spmm_case(16, 8, 4, 50, 4, 0)),
        ("K-runs", lambda: spmm_case(96, 160, 4, 70, 516, 71, kmajor=True)),
        ("paper's loop", lambda: spmm_case(100, 70, 4, 60, 300, 60)),
        ("paper's loop, naive", lambda: spmm_case(100, 70, 2, 60, 301, 61)),
        ("pair kernel bf16", lambda: spmm_case(256, 256, 4, 70, 4128, 36)),
        ("pair kernel bf16 ragged", lambda: spmm_case(200, 150, 4, 60, 130, 36, pad=2)),
        ("pair kernel bf16, <= 128 rows", lambda: spmm_case(72, 144, 8, 50, 1028, 37)),
        ("pair kernel bf16, stacked tiles", lambda: spmm_case(512, 64, 4, 60, 2000, 36)),
        ("pair kernel bf16, two chunks per stage, odd chunk count", lambda: spmm_case(256, 520, 4, 70, 1000, 36)),
        ("pair kernel bf16, two chunks per stage, <= 128 rows", lambda: spmm_case(100, 1000, 4, 80, 516, 36, pad=4)),
        ("pair kernel, three pieces", lambda: spmm_case(300, 150, 4, 70, 544, 86)),
        ("pair kernel TF32", lambda: spmm_case(300, 150, 4, 70, 516, 32)),
        ("one-CTA TF32", lambda: spmm_case(128, 128, 4, 60, 388, 32)),
        ("1x1 stride 2, straight from the input", lambda: s2_case(256, 64, 4, 70, 5, 28, 28)),
        ("1x1 stride 2, stacked tiles, two chunks per stage", lambda: s2_case(512, 520, 4, 80, 3, 12, 20)),
        ("3x3 plain", lambda: conv_case(32, 32, 8, 80, 2, 14, 14, 0)),
        ("3x3 padded grid", lambda: conv_case(256, 32, 8, 60, 3, 14, 14, 64)),
        ("3x3 padded grid, odd image", lambda: conv_case(260, 32, 4, 70, 2, 9, 13, 65)),
        ("3x3 per tap", lambda: conv_case(256, 32, 4, 60, 2, 14, 14, 45)),
        ("3x3 stride 2, phase planes", lambda: conv_case(256, 32, 4, 60, 4, 14, 14, 65, stride=2)),
        ("3x3 stride 2, odd image", lambda: conv_case(256, 16, 8, 60, 4, 9, 11, 64, stride=2)),
    ]
    for name, fn in cases:
        err, variant = fn()
        print(f"{name}: variant {variant}, scaled error {err:.2e}", flush=True)
        assert np.isfinite(err) and err <= TOL, (name, err)
    code = damaged_plan_is_reported()
    print(f"damaged plan: status {code}", flush=True)
    assert code != 0, "the checked build did not notice a channel index beyond the staged tile"
    print("checked build ok")


if __name__ == "__main__":
    main()
