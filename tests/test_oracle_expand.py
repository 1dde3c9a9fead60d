"""Pins of the oracle's expansion (vocab pass, frontier selection, pool) against
brute force, closed forms and library routines.  CPU only."""
import itertools
import math

import numpy as np
import pytest
import scipy.special

from oracle import radar_oracle as O
from paper_2512_14069_b200 import workloads as W


def rng(seed):
    return np.random.default_rng(seed)


# ---- vocab pass ----------------------------------------------------------------
def test_log_softmax_uniform_closed_form():
    for V in (1, 7, 1000):
        lp = O.log_softmax(np.full(V, 3.25, np.float32))
        assert np.allclose(lp, -math.log(V), atol=1e-14)


def test_log_softmax_matches_scipy_and_sums_to_one():
    z = (rng(0).standard_normal(5000) * 4).astype(np.float32)
    lp = O.log_softmax(z)
    assert np.allclose(lp, scipy.special.log_softmax(z.astype(np.float64)), atol=1e-12)
    assert abs(np.exp(lp).sum() - 1.0) < 1e-12


def test_log_softmax_with_minus_inf():
    z = np.array([0.0, -np.inf, 1.0], np.float32)
    lp = O.log_softmax(z)
    assert lp[1] == -np.inf
    assert abs(np.exp(lp[[0, 2]]).sum() - 1.0) < 1e-14


def test_vocab_topk_vs_python_sort_with_ties():
    g = rng(1)
    for V, k in ((50, 4), (1000, 10), (64, 32)):
        # quantised values force many exact ties: the lowest index must win
        z = np.round(g.standard_normal(V) * 2).astype(np.float32)
        idx, lp = O.vocab_topk(z, k)
        expect = sorted(range(V), key=lambda v: (-float(z[v]), v))[:k]
        assert list(idx) == expect
        full = scipy.special.log_softmax(z.astype(np.float64))
        assert np.allclose(lp, full[expect], atol=1e-12)


def test_vocab_topk_all_equal_takes_first_k():
    idx, _ = O.vocab_topk(np.zeros(20, np.float32), 5)
    assert list(idx) == [0, 1, 2, 3, 4]


def test_vocab_smaller_than_k_is_an_error():
    with pytest.raises(ValueError):
        O.vocab_topk(np.zeros(3, np.float32), 4)


# ---- one expansion ---------------------------------------------------------------
def test_expand_appends_f_major_and_selects_global_topk_bruteforce():
    g = rng(2)
    F, V, k = 3, 12, 3
    logits = g.standard_normal((F, V)).astype(np.float32)
    parent_score = np.array([-0.5, -1.25, -0.75], np.float32)
    parent_idx = np.array([4, 5, 6], np.int32)
    pool = O.Pool(64)
    pool.len = 7
    out = O.expand_step_seq(logits, parent_score, parent_idx, pool, t=2, k=k)
    assert pool.len == 7 + F * k
    full = scipy.special.log_softmax(logits.astype(np.float64), axis=1)
    cands = []
    for f in range(F):
        best = sorted(range(V), key=lambda v: (-float(logits[f, v]), v))[:k]
        for j, v in enumerate(best):
            p = 7 + f * k + j
            assert pool.tok[p] == v and pool.parent[p] == parent_idx[f] and pool.depth[p] == 2
            s = float(parent_score[f]) + full[f, v]
            assert pool.score[p] == np.float32(s)
            cands.append((s, p, f, v))
    # brute force: the k-subset with the largest total score is the frontier (scores are distinct here)
    best_subset = max(itertools.combinations(range(len(cands)), k), key=lambda c: sum(cands[i][0] for i in c))
    assert set(7 + np.array(best_subset)) == set(out["frontier_pool_idx"].tolist())
    # frontier is ordered by score, best first
    assert all(out["frontier_score"][i] >= out["frontier_score"][i + 1] for i in range(k - 1))
    for slot in range(k):
        p = int(out["frontier_pool_idx"][slot])
        s, _, f, v = cands[p - 7]
        assert out["frontier_src_row"][slot] == f and out["frontier_tok"][slot] == v
        assert abs(out["frontier_score"][slot] - s) < 1e-12
        assert pool.draft_row[p] == 1 + (2 - 1) * k + slot


def test_expand_tie_goes_to_lowest_flat_index():
    # two identical rows with identical parents: every candidate score ties pairwise
    row = np.array([3.0, 2.0, 1.0, 0.0], np.float32)
    logits = np.stack([row, row])
    pool = O.Pool(16)
    out = O.expand_step_seq(logits, np.zeros(2, np.float32), np.array([0, 1], np.int32), pool, t=2, k=2)
    assert out["frontier_pool_idx"].tolist() == [0, 2]      # (row0,tok0) then (row1,tok0)
    assert out["frontier_src_row"].tolist() == [0, 1]
    assert out["margin"] == 0.0


def test_walkthrough_structure_k2_two_calls():
    """Appendix walkthrough: the root yields 2 tokens; the second call on both yields 4
    candidates, of which the two kept have different parents, and the same token may
    appear under two parents as two distinct nodes."""
    I, YOU, SAY, DO, SEE = 0, 1, 2, 3, 4
    V = 6
    neg = -20.0
    r0 = np.full(V, neg, np.float32); r0[I], r0[YOU] = 2.0, 1.9
    rI = np.full(V, neg, np.float32); rI[SAY], rI[DO] = 3.0, 0.0
    rYOU = np.full(V, neg, np.float32); rYOU[SEE], rYOU[DO] = 3.0, 0.0
    draft = np.stack([r0, rI, rYOU])
    w = {k: np.zeros_like(v) for k, v in W.gate_weights(W.shrink(W.CONFIGS[1], k=2)).items()}
    w["b2"][:] = [0.0, 1.0]                                  # always continue
    pool, trace = O.run_expansion(draft, k=2, t_max=2, gate_w=w)
    assert [len(trace), pool.len] == [2, 2 + 4]
    assert pool.tok[:6].tolist() == [I, YOU, SAY, DO, SEE, DO]
    assert pool.parent[:6].tolist() == [-1, -1, 0, 0, 1, 1]
    assert trace[1]["frontier_tok"].tolist() == [SAY, SEE]
    assert trace[1]["frontier_src_row"].tolist() == [0, 1]
    assert pool.tok[3] == pool.tok[5] and pool.parent[3] != pool.parent[5]
    # the same structure, read from the fixture that restates the paper's example
    import os
    names = {"I": I, "you": YOU, "say": SAY, "do": DO, "see": SEE}
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "walkthrough_k2.txt"))
            if l.strip() and not l.startswith("#")]
    kept = set(trace[0]["frontier_pool_idx"].tolist()) | set(trace[1]["frontier_pool_idx"].tolist())
    for idx, name, par, keep in rows:
        idx, par, keep = int(idx), int(par), int(keep)
        assert pool.tok[idx] == names[name] and pool.parent[idx] == par and (idx in kept) == bool(keep)


# ---- whole expansion: counts and the score invariant -----------------------------
@pytest.mark.parametrize("cid", [1, 3])
def test_counts_and_path_score_is_sum_of_logprobs(cid):
    cfg = W.CONFIGS[cid]
    if cid == 3:
        cfg = W.shrink(cfg, V=2000)
    k, t_max = cfg.k, cfg.t_max
    draft = W.draft_logits(cfg, 0)
    for force in (1, 2, t_max):
        pool, trace = O.run_expansion(draft, k, t_max, W.gate_weights(cfg), force_calls=force)
        T = len(trace)
        assert T == force
        assert pool.len == k + (T - 1) * k * k
        full = scipy.special.log_softmax(draft.astype(np.float64), axis=1)
        # recompute every pool entry's score by walking to the root through the rows that produced it
        for p in range(pool.len):
            s, q = 0.0, p
            while q != -1:
                t = int(pool.depth[q])
                base = 0 if t == 1 else k + (t - 2) * k * k
                f = (q - base) // k
                row = 0 if t == 1 else 1 + (t - 2) * k + f
                s += full[row, pool.tok[q]]
                if pool.parent[q] != -1:
                    assert pool.draft_row[pool.parent[q]] == row
                q = int(pool.parent[q])
            # storage is float32 at every level: allow one float32 rounding per level
            assert abs(float(pool.score[p]) - s) < 4e-6 * max(1.0, abs(s)) * pool.depth[p]


def test_path_score_exact_in_fp64_single_call():
    cfg = W.CONFIGS[1]
    draft = W.draft_logits(cfg, 0)
    pool = O.Pool(cfg.C)
    out = O.expand_step_seq(draft[0:1], np.zeros(1, np.float32), np.full(1, -1, np.int32), pool, 1, cfg.k)
    full = scipy.special.log_softmax(draft[0].astype(np.float64))
    assert np.allclose(out["frontier_score"], full[out["frontier_tok"]], atol=1e-12)
    assert np.all(out["frontier_score"] <= 0.0)
