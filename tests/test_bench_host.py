"""Host-side logic of bench.py that the multi-GPU run relies on, exercised on CPU with a gloo group of two
processes: per-rank seeds give different batches of the same layer, the step time is the max over ranks, and the
reported value is the whole-job aggregate. The kernels never communicate (columns are independent), so this is
all the N > 1 path adds."""
import os
import socket
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    L = bench.get_layer("fc64", seed_index=rank)
    ms = bench.max_over_ranks(1.0 + rank, dist, torch, "cpu")          # rank 1 is the slow one
    val = bench.aggregate_gflops(2.0 * L.surviving_macs, world, ms)
    out.put((rank, ms, val, float(L.X.sum()), int(L.mask.sum()), L.surviving_macs))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_max_time_and_aggregate_value():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, v0, x0, m0, macs0), (r1, ms1, v1, x1, m1, macs1) = res
    assert ms0 == ms1 == 2.0                                   # max over ranks
    assert macs0 == macs1 and m0 == m1                          # same layer shape and block budget on every rank
    assert x0 != x1                                             # but each rank has its own batch (seed = base + rank)
    assert v0 == v1 == 2 * (2.0 * macs0) / 2.0e-3 / 1e9         # whole-job aggregate at the slowest rank's time


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None, "cpu") == 3.5
    assert abs(bench.aggregate_gflops(1e9, 4, 1.0) - 4000.0) < 1e-9
    L = bench.get_layer("mbv1_pw512")
    assert (L.M, L.C, L.Nc, L.m) == (512, 512, 6272, 19660)
    assert bench.compulsory_bytes(L) == 512 * 6272 * 4 * 2 + 19660 * 4 * 4 + 19660 * 4 + 513 * 4 + 512 * 4
    assert abs(bench.FP32_PEAK_TFLOPS - 74.44992) < 1e-6


def test_added_workloads_are_well_formed():
    sys.path.insert(0, ROOT)
    import bench
    import ubp_synth
    # the other block orientation: every row's runs of ones are whole blocks of KMAJOR_B input channels
    L = bench.get_layer("kmajor_pw512")
    assert (L.M, L.C, L.Nb, L.Nc) == (512, 512, 1, 6272) and L.m == int(L.mask.sum())
    assert L.m == ubp_synth.block_budget(512, 512, 70, bench.KMAJOR_B) * bench.KMAJOR_B
    padded = np.pad(L.mask, ((0, 0), (1, 1))).astype(np.int8)
    d = np.diff(padded, axis=1)
    starts, ends = np.argwhere(d == 1), np.argwhere(d == -1)
    assert ((ends[:, 1] - starts[:, 1]) % bench.KMAJOR_B == 0).all()
    # the chained bottleneck: shapes agree along the chain and only the first layer carries activations
    layers = ubp_synth.config_layers("r50_bottleneck", batch=2)
    assert [(l.M, l.C, l.R) for l in layers] == [(256, 1024, 1), (256, 256, 9), (1024, 256, 1)]
    assert layers[0].X.size and not layers[1].X.size and layers[1].Nc == layers[0].Nc == 2 * 14 * 14
    assert all(a.M == b.C for a, b in zip(layers, layers[1:]))
    # block-selection workloads: the oracle timing extrapolates from a bounded number of rounds
    t, cores, sample = bench.cpu_bed_time(ubp_synth.selection_weights(64, 32, 1, 1), 4, 100, budget_s=0.05)
    assert t > 0 and cores == 1 and ("iterations" in sample or "whole" in sample)
    for name, (M, C, R, Nb, p) in bench.BED_WORKLOADS.items():
        assert name.startswith("bed_") and M % Nb == 0 and 0 < p < 100
