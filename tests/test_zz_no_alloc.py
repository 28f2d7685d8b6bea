"""ubp_spmm_static: the entry point for callers that cannot allocate device memory (its plan lives in a fixed
array inside the library). Checked against ubp_spmm and against the CPU oracle on two calls in a row -- the
second call finds the first call's plan still in the array and must replace it. Collected last on purpose."""
import numpy as np
import pytest

import oracle
import ubp_synth

pytestmark = pytest.mark.gpu


def test_static_entry_matches_planned_entry_twice():
    import torch
    import paper_2407_19644_b200 as ubp
    assert ubp.static_plan_capacity() == 2 * 1024 * 1024
    layers = [ubp_synth.make_layer("a", 200, 150, 4, 70, 501, Nc=520, x_dist="normal"),
              ubp_synth.make_layer("b", 96, 260, 8, 60, 502, Nc=300, x_dist="normal", relu=False)]
    for L in layers:                                   # two calls in a row, different layers
        blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
        X = torch.from_numpy(L.X).cuda()
        bias = torch.from_numpy(L.bias).cuda()
        want = ubp.ubp_spmm(ubp.Plan(blob), X, bias, L.relu)
        out = torch.full((L.M, L.Nc), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        got = ubp.ubp_spmm_static(blob, X, bias, L.relu, out=out)
        torch.cuda.synchronize()
        # same kernel, same plan bytes, same summation order: within the suite's 1e-4 scaled tolerance
        # (in fact identical)
        scale = (np.abs(L.W[:, :, 0] * L.mask) @ np.abs(L.X) + np.abs(L.bias)[:, None]).astype(np.float64)
        err = np.max(np.abs(got.cpu().numpy().astype(np.float64) - want.cpu().numpy()) / scale)
        assert err <= 1e-4
        assert torch.equal(got, want)
        # and against the definition itself (the oracle), at the same gate
        Yref, A = oracle.masked_matmul(L.W, L.mask, L.X, L.bias, relu=L.relu)
        assert float(np.max(np.abs(got.cpu().numpy() - Yref) / A)) <= 1e-4
    # and the first layer again: the array now holds layer b's plan
    L = layers[0]
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    X = torch.from_numpy(L.X).cuda(); bias = torch.from_numpy(L.bias).cuda()
    assert torch.equal(ubp.ubp_spmm_static(blob, X, bias, L.relu), ubp.ubp_spmm(ubp.Plan(blob), X, bias, L.relu))


def test_static_entry_falls_back_to_the_smaller_plan():
    """512x512 at 70 %: the tensor-core plan (with its dense weight copy) exceeds the 2 MiB array, the sparse plan
    fits, so the call succeeds on the sparse kernel."""
    import torch
    import paper_2407_19644_b200 as ubp
    L = ubp_synth.make_layer("mid", 512, 512, 4, 70, 504, Nc=520, x_dist="normal")
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert ubp.plan_size(blob) > ubp.static_plan_capacity() > ubp.plan_size(blob, 14)
    X = torch.from_numpy(L.X).cuda(); bias = torch.from_numpy(L.bias).cuda()
    got = ubp.ubp_spmm_static(blob, X, bias, True)
    want = ubp.ubp_spmm(ubp.Plan(blob, 14), X, bias, True)
    assert torch.equal(got, want)


def test_static_entry_rejects_oversized_layer():
    import torch
    import paper_2407_19644_b200 as ubp
    L = ubp_synth.make_layer("big", 2048, 2048, 4, 50, 503, Nc=4, make_x=False)
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    assert ubp.plan_size(blob) > ubp.static_plan_capacity()
    X = torch.zeros((2048, 4), device="cuda")
    with pytest.raises(ubp.UbpError) as e:
        ubp.ubp_spmm_static(blob, X)
    assert e.value.code == -8 and "fixed device scratch" in str(e.value)


def test_static_entry_refuses_a_capturing_stream():
    """The upload inside ubp_spmm_static reads a host buffer that lives only for the call, so a captured call would
    replay from freed memory. A capturing stream is refused (UBP_E_UNSUPPORTED) before anything is enqueued: the
    capture ends empty and valid, nothing was launched, and an ordinary call afterwards still works."""
    import torch
    import paper_2407_19644_b200 as ubp
    L = ubp_synth.make_layer("cap", 64, 48, 4, 60, 505, Nc=260, x_dist="normal")
    blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    X = torch.from_numpy(L.X).cuda(); bias = torch.from_numpy(L.bias).cuda()
    out = torch.full((L.M, L.Nc), float("nan"), dtype=torch.float32, device="cuda")
    want = ubp.ubp_spmm_static(blob, X, bias, L.relu).clone()        # first call on the device, outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    marker = torch.zeros(4, device="cuda")
    with torch.cuda.graph(g, stream=s):
        marker.fill_(1.0)                                            # so that the graph is not empty
        with pytest.raises(ubp.UbpError) as e:
            ubp.ubp_spmm_static(blob, X, bias, L.relu, out=out, stream=s)
        assert e.value.code == -6
    g.replay()
    torch.cuda.synchronize()
    assert bool((marker == 1).all())                                 # the capture stayed valid
    assert torch.isnan(out).all()                                    # the refused call recorded nothing
    assert torch.equal(ubp.ubp_spmm_static(blob, X, bias, L.relu, out=out), want)
