"""Pins of the oracle's acceptance step: greedy walk vs brute force over all
root-to-leaf paths, special cases, the chain-rule closed form, the rejection-
sampling marginal over 10^6 seeded draws on a 16-token vocabulary, and the
acceptance-length distribution.  CPU only."""
import ctypes
import os
import subprocess

import numpy as np
import pytest
import scipy.special

from oracle import accept_oracle as A
from oracle import radar_oracle as O
from paper_2512_14069_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)


def _tree(seed, k=3, T=3, t_max=4, V=40, N=12):
    cfg = W.shrink(W.CONFIGS[1], cid=200 + seed, V=V, k=k, t_max=t_max)
    draft = W.draft_logits(cfg, 0)
    pool, _ = O.run_expansion(draft, k, t_max, W.gate_weights(cfg), force_calls=T)
    tree = O.rerank_build_tree(pool, N, 1, 10, t_max)
    return cfg, draft, tree


# ---- greedy ---------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_greedy_equals_bruteforce_over_retrieve_rows(seed):
    cfg, draft, tree = _tree(seed)
    tgt = W.target_logits(W.shrink(cfg, target_sigma=0.7), 0, draft, tree["draft_row"], tree["n_nodes"])
    res = O.verify_greedy(tgt, tree, cfg.t_max)
    a = np.argmax(tgt[: tree["n_nodes"]], axis=1)
    lens = []
    for r in range(tree["n_leaves"]):
        rr = [int(x) for x in tree["retrieve"][r] if x >= 0]
        m = 0
        while m + 1 < len(rr) and tree["tok"][rr[m + 1]] == a[rr[m]]:
            m += 1
        lens.append(m)
    best_len = max(lens)
    assert res["accept_len"] == best_len
    row = tree["retrieve"][res["best_retrieve_row"]]
    assert row[: best_len + 1].tolist() == res["path_nodes"][: best_len + 1].tolist()
    # the first row attaining the maximum is reported
    assert res["best_retrieve_row"] == lens.index(max(lens))
    last = res["path_nodes"][res["accept_len"]]
    assert res["next_token"] == a[last]
    assert res["path_tokens"][0] == tree["tok"][0]
    assert np.all(res["path_nodes"][res["accept_len"] + 1:] == -1)


def test_greedy_target_equals_draft_follows_top1_chain():
    cfg, draft, tree = _tree(3, T=4, N=30)
    tgt = W.target_logits(W.shrink(cfg, target_sigma=0.0), 0, draft, tree["draft_row"], tree["n_nodes"])
    res = O.verify_greedy(tgt, tree, cfg.t_max)
    # with target == draft each expanded node's best child is the target argmax: walk the first-child chain
    cur, depth = 0, 0
    while True:
        kids = O.children_of(tree["parent"], tree["n_nodes"], cur)
        if not kids:
            break
        cur, depth = kids[0], depth + 1
    assert res["accept_len"] == depth and res["path_nodes"][depth] == cur


def test_greedy_argmax_tie_takes_lowest_index():
    tree = {"n_nodes": 2, "tok": np.array([0, 3] + [-1] * 62, np.int32),
            "parent": np.array([-1, 0] + [-1] * 62, np.int32),
            "retrieve": np.array([[0, 1, -1]], np.int32), "n_leaves": 1}
    tgt = np.zeros((2, 8), np.float32)
    tgt[0, [3, 5]] = 2.0
    tgt[1, [6, 7]] = 1.0
    res = O.verify_greedy(tgt, tree, 2)
    assert res["accept_len"] == 1 and res["next_token"] == 6


# ---- stochastic: special cases --------------------------------------------------------
def _stoch(cfg, draft, tree, tgt, seed, T=1.0):
    g = np.random.default_rng(seed)
    ua = g.random(64, dtype=np.float32)
    us = float(g.random(dtype=np.float32))
    return A.verify_stochastic(tgt, draft, tree, ua, us, T, cfg.t_max), ua, us


def test_stochastic_target_equals_draft_accepts_first_child_everywhere():
    cfg, draft, tree = _tree(5, T=4, N=30)
    tgt = W.target_logits(W.shrink(cfg, target_sigma=0.0), 0, draft, tree["draft_row"], tree["n_nodes"])
    for seed in range(20):
        res, _, _ = _stoch(cfg, draft, tree, tgt, seed)
        cur, depth = 0, 0
        while O.children_of(tree["parent"], tree["n_nodes"], cur):
            cur, depth = O.children_of(tree["parent"], tree["n_nodes"], cur)[0], depth + 1
        assert res["accept_len"] == depth and res["path_nodes"][depth] == cur


def test_stochastic_one_hot_target_outside_children_rejects_all():
    cfg, draft, tree = _tree(6)
    kids = [tree["tok"][j] for j in O.children_of(tree["parent"], tree["n_nodes"], 0)]
    other = next(v for v in range(cfg.V) if v not in kids)
    tgt = np.full((64, cfg.V), -1e4, np.float32)
    tgt[:, other] = 0.0
    for seed in range(10):
        res, _, _ = _stoch(cfg, draft, tree, tgt, seed)
        assert res["accept_len"] == 0 and res["next_token"] == other and res["best_retrieve_row"] == 0


def test_stochastic_single_child_is_the_chain_rule_closed_form():
    """One child x: accept iff u < min(1, p(x)/q(x)); else sample norm(max(0, p-q)) by inverse CDF."""
    V = 16
    g = np.random.default_rng(7)
    for trial in range(200):
        tl = g.standard_normal((2, V)).astype(np.float32) * 2
        dl = g.standard_normal((1, V)).astype(np.float32) * 2
        T = [1.0, 0.7][trial % 2]
        p = scipy.special.softmax(tl[0].astype(np.float64) / T)
        q = scipy.special.softmax(dl[0].astype(np.float64) / T)
        x = int(g.integers(V))
        tree = {"n_nodes": 2, "tok": np.array([0, x], np.int32), "parent": np.array([-1, 0], np.int32),
                "draft_row": np.array([0, -1], np.int32), "retrieve": np.array([[0, 1]], np.int32), "n_leaves": 1}
        ua = g.random(64, dtype=np.float32); us = float(g.random(dtype=np.float32))
        res = A.verify_stochastic(tl, dl, tree, ua, us, T, 1)
        if ua[1] < min(1.0, p[x] / q[x]):
            assert res["accept_len"] == 1
            w = scipy.special.softmax(tl[1].astype(np.float64) / T)          # bonus token
        else:
            assert res["accept_len"] == 0
            w = np.maximum(p - q, 0.0)
        cdf = np.cumsum(w)
        assert res["next_token"] == int(np.searchsorted(cdf, us * cdf[-1], side="right"))


# ---- stochastic: Monte-Carlo marginal ---------------------------------------------------
@pytest.fixture(scope="module")
def mc(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("mc") / "libmc.so")
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", out,
                           os.path.join(HERE, "mc_marginal.c"), os.path.join(ROOT, "oracle", "accept_oracle.c"), "-lm"])
    return ctypes.CDLL(out)


def _ptr(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


@pytest.mark.parametrize("n1,n2,T", [(1, 0, 1.0), (2, 0, 1.0), (3, 0, 0.7), (4, 0, 1.0), (2, 2, 1.0), (3, 2, 0.7)])
def test_rejection_sampling_marginal_matches_target(mc, n1, n2, T):
    V, draws = 16, 1_000_000
    g = np.random.default_rng(100 + 10 * n1 + n2)
    tl = (g.standard_normal((1 + n1, V)) * 1.5).astype(np.float32)
    dl = (g.standard_normal((1 + n1, V)) * 1.5).astype(np.float32)
    h1 = np.zeros(V, np.int64); h2 = np.zeros((n1, V), np.int64); hl = np.zeros(3, np.int64)
    mc.mc_marginal.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_long,
                               ctypes.c_uint64] + [ctypes.c_void_p] * 5
    rc = mc.mc_marginal(V, n1, n2, T, draws, 12345 + n1, tl.ctypes.data, dl.ctypes.data,
                        h1.ctypes.data, h2.ctypes.data, hl.ctypes.data)
    assert rc == 0 and h1.sum() == draws
    p = scipy.special.softmax(tl.astype(np.float64) / T, axis=1)
    z = (h1 / draws - p[0]) / np.sqrt(p[0] * (1 - p[0]) / draws)
    assert np.max(np.abs(z)) < 4.5, z
    chi2 = float(np.sum((h1 - draws * p[0]) ** 2 / (draws * p[0])))
    assert chi2 < 60.0                                           # 15 d.o.f.: P(chi2 > 60) ~ 2e-7
    for j in range(n1):
        n = h2[j].sum()
        if n < 1000:
            continue
        pj = p[1 + j]
        zz = (h2[j] / n - pj) / np.sqrt(pj * (1 - pj) / n)
        assert np.max(np.abs(zz)) < 4.5, (j, zz)


def test_marginal_test_detects_a_wrong_rule(mc):
    """Sanity of the pin itself: with children drawn from a distribution other than the one
    handed to the accept routine, the same statistic must fail."""
    V, draws, n1 = 16, 200_000, 2
    g = np.random.default_rng(5)
    tl = (g.standard_normal((1 + n1, V)) * 1.5).astype(np.float32)
    dl = (g.standard_normal((1 + n1, V)) * 1.5).astype(np.float32)
    h1 = np.zeros(V, np.int64); h2 = np.zeros((n1, V), np.int64); hl = np.zeros(3, np.int64)
    mc.mc_marginal.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_long,
                               ctypes.c_uint64] + [ctypes.c_void_p] * 5
    # temperature mismatch: children drawn at T but the comparison is made against softmax(target / 1.3T)
    mc.mc_marginal(V, n1, 0, 1.0, draws, 99, tl.ctypes.data, dl.ctypes.data, h1.ctypes.data, h2.ctypes.data,
                   hl.ctypes.data)
    p_wrong = scipy.special.softmax(tl[0].astype(np.float64) / 1.3)
    z = (h1 / draws - p_wrong) / np.sqrt(p_wrong * (1 - p_wrong) / draws)
    assert np.max(np.abs(z)) > 4.5


# ---- acceptance-length distribution (Eq. 11-13) -----------------------------------------
@pytest.mark.parametrize("seed", range(3))
def test_accept_length_distribution_sums_to_one_and_matches_monte_carlo(mc, seed):
    cfg, draft, tree = _tree(30 + seed, k=3, T=3, t_max=3, V=24, N=14)
    tgt = W.target_logits(W.shrink(cfg, target_sigma=1.0), 0, draft, tree["draft_row"], tree["n_nodes"])
    T = 1.0 if seed != 1 else 0.7
    dist, pacc = A.accept_length_distribution(tgt, draft, tree, T, cfg.t_max)
    assert abs(dist.sum() - 1.0) < 1e-12 and np.all(dist >= -1e-15)
    assert pacc[0] == 1.0
    n = tree["n_nodes"]
    # children's acceptance probabilities never exceed the parent's
    for c in range(n):
        kids = O.children_of(tree["parent"], n, c)
        assert sum(pacc[j] for j in kids) <= pacc[c] + 1e-12
    draws = 400_000
    hl = np.zeros(cfg.t_max + 1, np.int64)
    mc.mc_fixed_tree.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int] + [ctypes.c_void_p] * 5 + \
        [ctypes.c_double, ctypes.c_long, ctypes.c_uint64, ctypes.c_void_p]
    tok = np.ascontiguousarray(tree["tok"][:n]); par = np.ascontiguousarray(tree["parent"][:n])
    drow = np.ascontiguousarray(tree["draft_row"][:n])
    tl = np.ascontiguousarray(tgt[:n]); dl = np.ascontiguousarray(draft)
    rc = mc.mc_fixed_tree(cfg.V, n, cfg.t_max, tok.ctypes.data, par.ctypes.data, drow.ctypes.data,
                          tl.ctypes.data, dl.ctypes.data, T, draws, 777 + seed, hl.ctypes.data)
    assert rc == 0
    freq = hl / draws
    sd = np.sqrt(np.maximum(dist * (1 - dist), 1e-12) / draws)
    assert np.all(np.abs(freq - dist) < 4.5 * sd + 1e-9), (freq, dist)


def test_accept_length_distribution_single_child_closed_form():
    V = 16
    g = np.random.default_rng(9)
    tl = g.standard_normal((2, V)).astype(np.float32); dl = g.standard_normal((1, V)).astype(np.float32)
    x = 5
    tree = {"n_nodes": 2, "tok": np.array([0, x], np.int32), "parent": np.array([-1, 0], np.int32),
            "depth": np.array([0, 1], np.int32), "draft_row": np.array([0, -1], np.int32)}
    dist, pacc = A.accept_length_distribution(tl, dl, tree, 1.0, 1)
    p = scipy.special.softmax(tl[0].astype(np.float64)); q = scipy.special.softmax(dl[0].astype(np.float64))
    a = min(1.0, p[x] / q[x])
    assert np.allclose(dist, [1 - a, a], atol=1e-14) and abs(pacc[1] - a) < 1e-14


# ---- hand-computed edge branches of the accept rule (4-token vocabulary) ---------------------------
# Each case is small enough to follow on paper; the expected values in the comments are worked out from
# Eq. 1-2 and the stated readings (q(x) = 0: accepted iff p(x) > 0; a draft row with no mass left stops
# the sibling loop; the draw is the inverse CDF in token order), not from running the oracle.
def _hand_tree(toks, parents):
    n = len(toks)
    tok = np.full(64, -1, np.int32); tok[:n] = toks
    par = np.full(64, -1, np.int32); par[:n] = parents
    drow = np.full(64, -1, np.int32)
    for i in range(n):
        if any(p == i for p in parents[1:]):
            drow[i] = 0                                   # every internal node reads draft row 0 in these cases
    leaves = [i for i in range(n) if i not in parents[1:]]
    retrieve = np.full((max(len(leaves), 1), 3), -1, np.int32)
    for r, l in enumerate(leaves):
        path = [l]
        while par[path[-1]] >= 0:
            path.append(int(par[path[-1]]))
        retrieve[r, :len(path)] = path[::-1]
    return {"n_nodes": n, "tok": tok, "parent": par, "draft_row": drow, "retrieve": retrieve, "n_leaves": len(leaves)}


NEG = -np.inf


def _logs(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, np.float64)).astype(np.float32)


def test_accept_when_draft_probability_is_zero_and_target_positive():
    # q(x) = 0, p(x) = 1/4 > 0: the ratio is +inf, the child is accepted whatever u is.
    tree = _hand_tree([9, 2], [-1, 0])
    target = np.stack([_logs([.25, .25, .25, .25]), _logs([.1, .2, .3, .4])])
    draft = _logs([1 / 3, 1 / 3, 0, 1 / 3])[None]
    ua = np.full(64, 0.999, np.float32)
    r = A.verify_stochastic(target, draft, tree, ua, 0.55, 1.0, 2)
    assert r["accept_len"] == 1 and r["path_nodes"][:2].tolist() == [0, 1]
    # leaf reached: bonus token from softmax(target[1]) = (.1, .2, .3, .4); CDF .1 .3 .6 1: first step above .55 is token 2
    assert r["next_token"] == 2


def test_reject_when_both_probabilities_are_zero():
    # q(x) = 0 and p(x) = 0: rejected.  p = (1/3, 1/3, 0, 1/3), q = (1/4, 1/4, 0, 1/2):
    # residual max(0, p - q) = (1/12, 1/12, 0, 0) -> (1/2, 1/2, 0, 0); u = .7 -> token 1.
    tree = _hand_tree([9, 2], [-1, 0])
    target = np.stack([_logs([1 / 3, 1 / 3, 0, 1 / 3]), _logs([.25, .25, .25, .25])])
    draft = _logs([.25, .25, 0, .5])[None]
    ua = np.zeros(64, np.float32)                         # u = 0 would accept anything with a positive ratio
    r = A.verify_stochastic(target, draft, tree, ua, 0.7, 1.0, 2)
    assert r["accept_len"] == 0 and r["next_token"] == 1
    r = A.verify_stochastic(target, draft, tree, ua, 0.3, 1.0, 2)
    assert r["next_token"] == 0


def test_draft_row_with_all_mass_on_the_rejected_token_stops_the_sibling_loop():
    # q = (0, 1, 0, 0); children x1 = token 1, x2 = token 0.  p = (.4, .1, .3, .2): ratio for x1 = .1 < u = .5 -> reject.
    # Residual max(0, p - q) = (.4, 0, .3, .2) / .9.  Removing token 1 leaves q with no mass: nothing is left to
    # propose, so x2 is NOT tried (it would be accepted, its q being 0 and its p positive) and the next token is
    # drawn from the residual: CDF 4/9, 4/9, 7/9, 1: u = .5 -> token 2, u = .4 -> token 0.
    tree = _hand_tree([9, 1, 0], [-1, 0, 0])
    target = np.stack([_logs([.4, .1, .3, .2]), _logs([.25] * 4), _logs([.25] * 4)])
    draft = _logs([0, 1, 0, 0])[None]
    ua = np.full(64, 0.5, np.float32)
    r = A.verify_stochastic(target, draft, tree, ua, 0.5, 1.0, 2)
    assert r["accept_len"] == 0 and r["next_token"] == 2
    assert A.verify_stochastic(target, draft, tree, ua, 0.4, 1.0, 2)["next_token"] == 0
    # Eq. 13 on the same tree: P_acc(x1) = .1, P_acc(x2) = 0 (never tried), P_stop(root) = .9
    dist, pacc = A.accept_length_distribution(target, draft, dict(tree, depth=np.array([0, 1, 1] + [0] * 61, np.int32)), 1.0, 2)
    assert abs(pacc[1] - 0.1) < 1e-7 and pacc[2] == 0.0           # the logits are float32: ln(.1) is rounded
    assert abs(dist[0] - 0.9) < 1e-7 and abs(dist[1] - 0.1) < 1e-7


def test_second_sibling_is_tried_on_the_residual_and_the_renormalised_draft():
    # The ordinary multi-draft step, by hand: p = (.4, .1, .3, .2), q = (.1, .6, .2, .1); x1 = token 1, x2 = token 2.
    # x1: ratio 1/6 < u = .5 -> reject.  p' = max(0, p - q) = (.3, 0, .1, .1) / .5 = (.6, 0, .2, .2);
    # q' = (.1, 0, .2, .1) / .4 = (.25, 0, .5, .25).  x2: ratio .2 / .5 = .4 < .5 -> reject.
    # p'' = max(0, p' - q') = (.35, 0, 0, 0) / .35 = (1, 0, 0, 0): next token 0 for every u.
    tree = _hand_tree([9, 1, 2], [-1, 0, 0])
    target = np.stack([_logs([.4, .1, .3, .2]), _logs([.25] * 4), _logs([.25] * 4)])
    draft = _logs([.1, .6, .2, .1])[None]
    r = A.verify_stochastic(target, draft, tree, np.full(64, 0.5, np.float32), 0.9, 1.0, 2)
    assert r["accept_len"] == 0 and r["next_token"] == 0
    assert abs(r["accept_margin"] - 0.1) < 1e-6                      # |u - ratio| of the closer test (x2)
    # with u = .3 the second sibling (ratio .4) is accepted; it is a leaf: bonus token from its uniform target row
    ua = np.full(64, 0.5, np.float32); ua[2] = 0.3
    r = A.verify_stochastic(target, draft, tree, ua, 0.6, 1.0, 2)
    assert r["accept_len"] == 1 and r["path_nodes"][:2].tolist() == [0, 2] and r["next_token"] == 2


def test_inverse_cdf_upper_end_returns_the_last_token_with_mass():
    # u = 1 is outside [0, 1) but defined: no step of the CDF lies above u * total, and the draw falls back to the
    # last token with positive weight (token 2 here, not the zero-weight token 3).
    tree = _hand_tree([9], [-1])
    target = _logs([.2, .3, .5, 0])[None]
    draft = _logs([.25] * 4)[None]
    r = A.verify_stochastic(target, draft, tree, np.zeros(64, np.float32), 1.0, 1.0, 2)
    assert r["accept_len"] == 0 and r["next_token"] == 2
    # just below the top step the ordinary rule applies: largest float32 below 1
    assert A.verify_stochastic(target, draft, tree, np.zeros(64, np.float32), np.float32(1) - np.float32(2 ** -24), 1.0, 2)["next_token"] == 2
    assert A.verify_stochastic(target, draft, tree, np.zeros(64, np.float32), 0.4999, 1.0, 2)["next_token"] == 1
