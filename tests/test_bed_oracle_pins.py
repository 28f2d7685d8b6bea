"""Pins for the block-selection oracle (scores of Eq. 1, greedy selection of Eq. 3, the dynamic programme of
Eq. 4, block expansion and division of Algorithms 1 and 2) against things that do not come from the oracle:
the paper's eight-weight example, a restatement of expansion by window sums over the remaining kernels,
exhaustive search on tiny inputs, the aligned and the element-wise special cases, and invariants."""
import itertools
import os

import numpy as np
import pytest

import oracle
import ubp_synth
from conftest import GOLDEN, parse_golden

NEG = -np.inf


def ints(v):
    return [int(x) for x in v.split()]


# ---------------------------------------------------------------------------------------------------------
# the worked example of Section 3.2 / Section 4.1
# ---------------------------------------------------------------------------------------------------------

def test_worked_example_greedy_optimal_and_bed():
    g = parse_golden(os.path.join(GOLDEN, "bed_worked_example.txt"))
    N, m = int(g["N"][0]), int(g["m"][0])
    w = np.array(ints(g["w"][0]), np.float32).reshape(-1, 1)
    S = oracle.block_scores(w, N)
    assert S[:-1].tolist() == ints(g["scores"][0]) and S[-1] == NEG
    gi = oracle.greedy_select(S, N, m)
    assert gi.tolist() == ints(g["greedy_order"][0])
    assert float(S[gi].sum()) == float(g["greedy_total"][0])
    oi, tot = oracle.optimal_select(S, N, m)
    assert oi.tolist() == ints(g["optimal"][0]) and tot == float(g["optimal_total"][0])
    Ibar, sc = oracle.bed_expand(S, N, m)
    assert Ibar.tolist() == ints(g["bed_expanded_order"][0])
    assert sc.tolist() == [float(x) for x in g["bed_expanded_scores"][0].split()]
    I = oracle.bed_divide(Ibar, N)
    assert I.tolist() == ints(g["bed_final"][0])
    mask, I2, _ = oracle.bed_select(w, N, m)
    assert mask[:, 0].tolist() == ints(g["mask"][0]) and I2.tolist() == I.tolist()
    # what the text says in words: w0 is kept by expansion although greedy dropped it; w4 is the one to go
    assert mask[0, 0] == 1 and mask[4, 0] == 0 and mask[7, 0] == 0


# ---------------------------------------------------------------------------------------------------------
# Eq. 1
# ---------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("M,C,R,N", [(7, 3, 1, 3), (16, 5, 9, 4), (9, 2, 9, 1), (8, 4, 1, 8)])
def test_scores_are_l1_norms_of_the_blocks_and_minus_infinity_past_the_edge(M, C, R, N):
    W = ubp_synth.selection_weights(M, C, R, seed=5, kind="integer")
    S = oracle.block_scores(W, N).reshape(C, M)          # k = i + M*j: column j is contiguous
    for j in range(C):
        for i in range(M):
            if i + N <= M:
                assert S[j, i] == np.abs(W[i:i + N, j, :]).sum()      # integers: exact
            else:
                assert S[j, i] == NEG
    Wf = ubp_synth.selection_weights(M, C, R, seed=6, kind="trained")
    Sf = oracle.block_scores(Wf, N).reshape(C, M)
    ref = np.array([[np.abs(Wf[i:i + N, j, :].astype(np.float64)).sum() if i + N <= M else NEG
                     for i in range(M)] for j in range(C)])
    fin = np.isfinite(ref)
    assert np.array_equal(np.isfinite(Sf), fin)
    assert np.allclose(Sf[fin], ref[fin], rtol=(N * R + 2) * 2.0 ** -24, atol=0)


# ---------------------------------------------------------------------------------------------------------
# Algorithm 1, restated: every remaining kernel keeps its own l1 norm; a candidate's score is the sum of the
# next N remaining kernels if they all lie in one input channel, else -inf; take the first maximum and
# delete its N kernels. No incremental update anywhere, so a wrong index or sign in the update shows.
# ---------------------------------------------------------------------------------------------------------

def expand_by_window_sums(a, N, m):
    C, M = a.shape
    items = [(j, i, float(a[j, i])) for j in range(C) for i in range(M)]      # list order = k order
    chosen, scores = [], []
    for _ in range(m):
        best, bp = NEG, -1
        for p in range(len(items) - N + 1):
            win = items[p:p + N]
            if all(x[0] == win[0][0] for x in win):
                s = sum(x[2] for x in win)
                if s > best:
                    best, bp = s, p
        if bp < 0:
            break
        chosen.append(items[bp][1] + M * items[bp][0])
        scores.append(best)
        del items[bp:bp + N]
    return chosen, scores, items


@pytest.mark.parametrize("M,C,N,m,seed", [(12, 1, 2, 5, 1), (12, 3, 3, 9, 2), (17, 2, 4, 7, 3), (10, 4, 2, 20, 4),
                                          (9, 3, 3, 9, 5), (16, 2, 8, 3, 6), (11, 2, 1, 13, 7), (6, 5, 5, 5, 8)])
def test_expansion_equals_window_sums_over_remaining_kernels(M, C, N, m, seed):
    W = ubp_synth.selection_weights(M, C, 1, seed=seed, kind="integer")
    W[W == 0] = 1.0                                      # positive norms: fewer accidental ties, still many
    S = oracle.block_scores(W, N)
    Ibar, sc = oracle.bed_expand(S, N, m)
    a = np.abs(W[:, :, 0]).T.copy()
    ref_idx, ref_sc, left = expand_by_window_sums(a, N, m)
    assert Ibar.tolist() == ref_idx
    assert sc.tolist() == ref_sc
    # division gives the runs of removed kernels cut every N rows, which is what decoding the mask gives too
    I = oracle.bed_divide(Ibar, N)
    mask = oracle.starts_to_mask(I, M, C, N)
    kept = np.ones((C, M), np.uint8)
    for (j, i, _) in left:
        kept[j, i] = 0
    assert np.array_equal(mask, kept.T)
    bi, bj = oracle.decode_mask(mask, N)
    assert sorted((bi.astype(np.int64) + M * bj).tolist()) == I.tolist()
    # each chosen score is the mass of the kernels it removed
    assert sum(ref_sc) == float(np.abs(W[:, :, 0])[mask == 1].sum())


def test_expansion_stops_when_nothing_finite_is_left():
    # 7 rows, N = 3: two blocks per column at most, the budget asks for more
    W = ubp_synth.selection_weights(7, 2, 1, seed=11, kind="integer")
    W[W == 0] = 2.0
    S = oracle.block_scores(W, 3)
    Ibar, _ = oracle.bed_expand(S, 3, 10)
    assert Ibar.size == 4
    mask = oracle.starts_to_mask(oracle.bed_divide(Ibar, 3), 7, 2, 3)
    assert mask.sum() == 12 and (mask.sum(axis=0) == 6).all()


# ---------------------------------------------------------------------------------------------------------
# Eq. 4 against exhaustive search; greedy and expansion never beat it
# ---------------------------------------------------------------------------------------------------------

def all_placements(S, N, m):
    """Every set of m candidate indices, pairwise at least N apart, with finite scores."""
    ok = [k for k in range(S.size) if np.isfinite(S[k])]
    for comb in itertools.combinations(ok, m):
        if all(comb[q + 1] - comb[q] >= N for q in range(m - 1)):
            yield comb


@pytest.mark.parametrize("M,C,N,m,seed", [(8, 1, 2, 3, 21), (6, 2, 2, 4, 22), (7, 2, 3, 3, 23), (5, 3, 2, 5, 24),
                                          (9, 1, 4, 2, 25), (6, 2, 3, 4, 26)])
def test_dynamic_programme_is_the_exhaustive_optimum(M, C, N, m, seed):
    W = ubp_synth.selection_weights(M, C, 1, seed=seed, kind="trained")
    S = oracle.block_scores(W, N)
    best = max((float(np.sum(S[list(c)].astype(np.float64))) for c in all_placements(S, N, m)), default=None)
    I, tot = oracle.optimal_select(S, N, m)
    if best is None:
        assert I is None
        return
    assert abs(tot - best) <= 1e-12 * max(1.0, abs(best))
    assert np.all(np.diff(I) >= N) and np.isfinite(S[I]).all()
    assert abs(float(S[I].astype(np.float64).sum()) - best) <= 1e-12 * max(1.0, abs(best))
    a = np.abs(W[:, :, 0]).astype(np.float64)
    for sel in (oracle.greedy_select(S, N, m), oracle.bed_divide(oracle.bed_expand(S, N, m)[0], N)):
        mk = oracle.starts_to_mask(sel, M, C, N)
        assert a[mk == 1].sum() <= best * (1 + 1e-6)


def test_expansion_is_close_to_optimal_and_ahead_of_greedy_on_average():
    """Section 5.2 reports expansion-and-division comparable to the optimum and above greedy; on small random
    layers (where the optimum is computable) the kept l1 mass must rank the same way on average."""
    tot = {"g": 0.0, "b": 0.0, "o": 0.0}
    for seed in range(40):
        M, C, N = 24, 4, 4
        m = oracle.block_budget(M, C, 50, N)
        W = ubp_synth.selection_weights(M, C, 1, seed=100 + seed, kind="trained")
        S = oracle.block_scores(W, N)
        a = np.abs(W[:, :, 0]).astype(np.float64)
        tot["g"] += a[oracle.starts_to_mask(oracle.greedy_select(S, N, m), M, C, N) == 1].sum()
        tot["b"] += a[oracle.bed_select(W, N, m)[0] == 1].sum()
        tot["o"] += oracle.optimal_select(S, N, m)[1]
    assert tot["g"] < tot["b"] <= tot["o"] * (1 + 1e-9)
    assert tot["b"] >= 0.97 * tot["o"]


# ---------------------------------------------------------------------------------------------------------
# special cases that reduce to a sort
# ---------------------------------------------------------------------------------------------------------

def test_block_size_one_is_element_pruning_by_magnitude():
    W = ubp_synth.selection_weights(13, 7, 1, seed=31, kind="trained")
    m = 40
    S = oracle.block_scores(W, 1)
    top = np.sort(np.argsort(-S, kind="stable")[:m])
    assert np.array_equal(np.sort(oracle.greedy_select(S, 1, m)), top)
    assert np.array_equal(oracle.bed_divide(oracle.bed_expand(S, 1, m)[0], 1), top)
    assert np.array_equal(oracle.optimal_select(S, 1, m)[0], top)


@pytest.mark.parametrize("N", [2, 4])
def test_minus_infinity_at_unaligned_starts_gives_aligned_pruning(N):
    """Section 3.1: scores of -inf wherever the start row is not a multiple of N turn the method into aligned
    block-wise pruning, i.e. the m best aligned blocks."""
    M, C, m = 16, 6, 11
    W = ubp_synth.selection_weights(M, C, 1, seed=41, kind="trained")
    S = oracle.block_scores(W, N)
    i = np.arange(M * C) % M
    S[i % N != 0] = NEG
    top = np.sort(np.argsort(-S, kind="stable")[:m])
    assert np.array_equal(np.sort(oracle.greedy_select(S, N, m)), top)
    assert np.array_equal(oracle.bed_divide(oracle.bed_expand(S, N, m)[0], N), top)
    assert np.array_equal(oracle.optimal_select(S, N, m)[0], top)


# ---------------------------------------------------------------------------------------------------------
# invariants at a size closer to a real layer
# ---------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("M,C,R,N,p", [(64, 48, 1, 4, 70), (96, 32, 9, 8, 80), (50, 40, 1, 2, 50), (33, 20, 1, 16, 50)])
def test_selection_invariants(M, C, R, N, p):
    W = ubp_synth.selection_weights(M, C, R, seed=M + N, kind="trained")
    m = oracle.block_budget(M, C, p, N)
    mask, I, Ibar = oracle.bed_select(W, N, m)
    assert I.size == Ibar.size == m                       # Section 3.1: exactly m blocks
    assert np.all(np.diff(I) >= N)                        # Eq. 2: at most one start in any N consecutive candidates
    assert np.all(I % M + N <= M)                         # Eq. 1: no block leaves the weights
    assert int(mask.sum()) == m * N
    bi, bj = oracle.decode_mask(mask, N)                  # runs of ones are whole blocks
    assert np.array_equal(np.sort(bi.astype(np.int64) + M * bj), I)
    # the first choice is the best candidate overall, and chosen scores never increase
    S = oracle.block_scores(W, N)
    _, sc = oracle.bed_expand(S, N, m)
    assert Ibar[0] == int(np.argmax(S)) and np.all(np.diff(sc) <= 0)
    # efficacy (Section 5.2): between aligned pruning (0) and element pruning (1)
    a = np.abs(W.astype(np.float64)).sum(axis=2)
    ep = np.sort(a.ravel())[::-1][:m * N].sum()
    al = a[:M // N * N].reshape(M // N, N, C).sum(axis=1).ravel()
    abp = np.sort(al)[::-1][:m].sum()
    eff = (a[mask == 1].sum() - abp) / (ep - abp)
    assert 0.0 < eff < 1.0
