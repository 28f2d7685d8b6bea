"""Shared helpers for the test-suite (no arithmetic of the method here)."""
import numpy as np


def plan_to_dense(img: np.ndarray, geom: dict, M: int, C: int, R: int):
    """Replay a plan image on the host: scatter every entry's rows that belong
    to its panel into a dense [M][C][R] array and count how often each
    (row, channel) was written. Independent reader of the image layout."""
    nbk, P, KT, WR, dup = geom["nbk"], geom["panel_rows"], geom["k_tile"], geom["WR"], 2 if geom["dupw"] else 1
    nkt, NP, NG = geom["nkt"], geom["NP"], geom["NG"]
    F = P + nbk - 1
    pad16 = lambda x: (x + 15) // 16 * 16
    fo_bytes = pad16(2 * (F + 1))
    W = np.zeros((M, C, R), np.float32)
    hits = np.zeros((M, C), np.int32)
    tab = np.frombuffer(img, "<u4", nkt * NG + 1, 256)
    n_entries = 0
    for kt in range(nkt):
        for g in range(NG):
            g0 = int(tab[kt * NG + g]) * 16
            g1 = int(tab[kt * NG + g + 1]) * 16
            poff = np.frombuffer(img, "<u4", WR + 1, g0)
            assert g0 + int(poff[WR]) <= g1
            for wr in range(WR):
                p = g * WR + wr
                if poff[wr + 1] == poff[wr]:
                    assert p >= NP
                    continue
                so = g0 + int(poff[wr])
                fo = np.frombuffer(img, "<u2", F + 1, so)
                n = int(fo[F])
                assert (np.diff(fo.astype(np.int64)) >= 0).all() and fo[0] == 0
                jl = np.frombuffer(img, "<u2", n, so + fo_bytes)
                w = np.frombuffer(img, "<f4", n * nbk * R * dup, so + fo_bytes + pad16(2 * (n + 4))).reshape(n, nbk, R, dup)
                assert so + fo_bytes + pad16(2 * (n + 4)) + pad16(4 * (n + 2) * nbk * R * dup) == g0 + int(poff[wr + 1])
                assert not np.frombuffer(img, "<u2", 4, so + fo_bytes + 2 * n).any()      # read-ahead slack is zero
                n_entries += n
                for f in range(F):
                    s = f - (nbk - 1)
                    for e in range(int(fo[f]), int(fo[f + 1])):
                        j = kt * KT + int(jl[e])
                        assert int(jl[e]) < KT and j < C
                        for r in range(nbk):
                            if 0 <= s + r < P:
                                row = p * P + s + r
                                assert row < M
                                W[row, j] = w[e, r, :, 0]
                                if dup == 2:
                                    assert np.array_equal(w[e, r, :, 0].view(np.uint32), w[e, r, :, 1].view(np.uint32))
                                hits[row, j] += 1
    return W, hits, n_entries


def scaled_error(Y: np.ndarray, Yref: np.ndarray, A: np.ndarray) -> float:
    """max |Y - Yref| / A with A = |Wm||X| + |bias| (the error scale of a dot product)."""
    A = np.where(A > 0, A, 1.0)
    return float(np.max(np.abs(Y.astype(np.float64) - Yref) / A))


def krun_plan_to_dense(img: np.ndarray, geom: dict, M: int, C: int):
    """Replay a K-run plan image (entries = runs of nbk consecutive input channels of one output row, filed under
    channel tile / row panel / row inside the panel) into a dense [M][C] array; returns it with the number of entries
    and the number of stored weights that are not zero padding."""
    B, P, KT, WR = geom["nbk"], geom["panel_rows"], geom["k_tile"], geom["WR"]
    nkt, NP, NG = geom["nkt"], geom["NP"], geom["NG"]
    pad16 = lambda x: (x + 15) // 16 * 16
    fo_bytes = pad16(2 * (P + 1))
    W = np.zeros((M, C), np.float64)
    tab = np.frombuffer(img, "<u4", nkt * NG + 1, 256)
    n_entries = 0
    for kt in range(nkt):
        for g in range(NG):
            g0 = int(tab[kt * NG + g]) * 16
            poff = np.frombuffer(img, "<u4", WR + 1, g0)
            for wr in range(WR):
                p = g * WR + wr
                if poff[wr + 1] == poff[wr]:
                    continue
                so = g0 + int(poff[wr])
                fo = np.frombuffer(img, "<u2", P + 1, so)
                n = int(fo[P])
                jl = np.frombuffer(img, "<u2", n, so + fo_bytes)
                w = np.frombuffer(img, "<f4", n * B, so + fo_bytes + pad16(2 * (n + 4))).reshape(n, B)
                n_entries += n
                for r in range(P):
                    for e in range(int(fo[r]), int(fo[r + 1])):
                        ks = int(jl[e])
                        assert 0 <= ks <= KT - B                       # a run lies wholly inside its channel tile
                        row = p * P + r
                        assert row < M
                        for u in range(B):
                            c = kt * KT + ks + u
                            if c < C:
                                W[row, c] += float(w[e, u])
                            else:
                                assert w[e, u] == 0
    return W, n_entries
