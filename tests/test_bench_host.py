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
    for wname, sp in bench.KMAJOR_WORKLOADS.items():
        L = bench.get_layer(wname)
        assert (L.M, L.C, L.Nb, L.Nc) == (512, 512, 1, 6272) and L.m == int(L.mask.sum())
        assert L.m == ubp_synth.block_budget(512, 512, sp, bench.KMAJOR_B) * bench.KMAJOR_B
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


def test_gpus_flag_without_a_launcher_spawns_the_ranks():
    """`python bench.py --gpus 2` started by hand must not silently measure one rank: it starts two local ranks under
    torch.distributed.run itself. Exercised on CPU through the reference arm (rank 0 times the oracle and prints the
    line, the other rank exits 0 without work)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload",
                        "fc64", "--steps", "1", "--warmup", "3"], capture_output=True, text=True, timeout=600, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(ln) for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                        # rank 0 alone prints
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["config"]["workload"] == "fc64"
    # a launcher that started another number of ranks than --gpus says is an error, not a silent one-GPU run
    env2 = dict(env, WORLD_SIZE="3", RANK="0", LOCAL_RANK="0")
    r2 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload",
                         "fc64", "--steps", "1"], capture_output=True, text=True, timeout=600, env=env2)
    assert r2.returncode != 0 and "rank" in (r2.stderr + r2.stdout)


def test_both_arms_describe_the_same_config():
    sys.path.insert(0, ROOT)
    import bench
    L = bench.get_layer("mbv1_pw512")
    c = bench.workload_config(L, "mbv1_pw512", 1, False)
    assert c["workload"] == "mbv1_pw512" and c["M"] == 512 and c["Nc"] == 6272 and c["blocks"] == 19660
    assert set(bench.EXTRA_CONFIGS) >= {"r50_3x3", "sweep_nb2_p50", "sweep_nb16_p90", "mbv1_L1", "mbv1_L13"}
    assert all(n in bench.WORKLOADS for n in bench.EXTRA_CONFIGS)


def test_error_figures_on_known_values():
    sys.path.insert(0, ROOT)
    import bench
    Yref = np.array([[1.0, -2.0, 0.0], [4.0, 1e-9, 2.0]])
    A = np.array([[2.0, 4.0, 1.0], [8.0, 1.0, 4.0]])
    Y = Yref + np.array([[1e-3, 0.0, 1e-3], [0.0, 1e-3, -2e-3]])
    e = bench.error_figures(Y.astype(np.float64), Yref, A)
    assert abs(e["scaled"] - 1e-3) < 1e-12                       # |d|/A: 5e-4, 0, 1e-3, 0, 1e-3, 5e-4
    assert abs(e["normwise"] - 2e-3 / 4.0) < 1e-12
    assert abs(e["elementwise"] - 1e-3) < 1e-9                   # zeros and the 1e-9 entry are below 1e-3 rms: left out
    assert e["outputs_compared"] == 6
