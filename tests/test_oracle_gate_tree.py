"""Pins of the oracle's prediction model, call schedule, rerank and tree
serialisation.  CPU only."""
import itertools

import numpy as np
import pytest
import torch

from oracle import radar_oracle as O
from paper_2512_14069_b200 import workloads as W


# ---- prediction model ---------------------------------------------------------------
def _torch_gate(w, k):
    H = O.GATE_HIDDEN
    lstm = torch.nn.LSTM(input_size=k, hidden_size=H, num_layers=1).double()
    fc1 = torch.nn.Linear(H + k, H).double()
    fc2 = torch.nn.Linear(H, 2).double()
    with torch.no_grad():
        lstm.weight_ih_l0.copy_(torch.from_numpy(w["w_ih"]).double())
        lstm.weight_hh_l0.copy_(torch.from_numpy(w["w_hh"]).double())
        lstm.bias_ih_l0.copy_(torch.from_numpy(w["b_ih"]).double())
        lstm.bias_hh_l0.copy_(torch.from_numpy(w["b_hh"]).double())
        fc1.weight.copy_(torch.from_numpy(w["w1"]).double()); fc1.bias.copy_(torch.from_numpy(w["b1"]).double())
        fc2.weight.copy_(torch.from_numpy(w["w2"]).double()); fc2.bias.copy_(torch.from_numpy(w["b2"]).double())
    return lstm, fc1, fc2


@pytest.mark.parametrize("k", [4, 10])
def test_gate_matches_torch_lstm_and_linear_over_a_sequence(k):
    cfg = W.shrink(W.CONFIGS[2], k=k)
    w = W.gate_weights(cfg)
    # scale up so that the nonlinearities are exercised away from their linear range
    w = {n: (v * 6).astype(np.float32) for n, v in w.items()}
    lstm, fc1, fc2 = _torch_gate(w, k)
    g = np.random.default_rng(3)
    H = O.GATE_HIDDEN
    h = np.zeros(H); c = np.zeros(H)
    th = (torch.zeros(1, 1, H).double(), torch.zeros(1, 1, H).double())
    for _ in range(5):
        x = g.random(k)
        y, h, c = O.gate_step(x, h, c, w)
        with torch.no_grad():
            out, th = lstm(torch.from_numpy(x).view(1, 1, k), th)
            ty = fc2(torch.relu(fc1(torch.cat([out.view(-1), torch.from_numpy(x)]))))
        assert np.allclose(y, ty.numpy(), atol=1e-12)
        assert np.allclose(h, th[0].view(-1).numpy(), atol=1e-12)
        assert np.allclose(c, th[1].view(-1).numpy(), atol=1e-12)


def test_gate_with_a_wide_input_matches_torch_lstm():
    """The hidden-state variant of Table 3 is the same network with another input size."""
    d_in, H = 48, O.GATE_HIDDEN
    g = np.random.default_rng(11)
    u = lambda *shape: g.uniform(-0.5, 0.5, size=shape).astype(np.float32)
    w = {"w_ih": u(4 * H, d_in), "w_hh": u(4 * H, H), "b_ih": u(4 * H), "b_hh": u(4 * H),
         "w1": u(H, H + d_in), "b1": u(H), "w2": u(2, H), "b2": u(2)}
    lstm, fc1, fc2 = _torch_gate(w, d_in)
    h = np.zeros(H); c = np.zeros(H)
    th = (torch.zeros(1, 1, H).double(), torch.zeros(1, 1, H).double())
    for _ in range(4):
        x = g.standard_normal(d_in)
        y, h, c = O.gate_step(x, h, c, w)
        with torch.no_grad():
            out, th = lstm(torch.from_numpy(x).view(1, 1, d_in), th)
            ty = fc2(torch.relu(fc1(torch.cat([out.view(-1), torch.from_numpy(x)]))))
        assert np.allclose(y, ty.numpy(), atol=1e-12)
        assert np.allclose(h, th[0].view(-1).numpy(), atol=1e-12)


def _mlp_weights(k, seed=5, scale=2.0):
    g = np.random.default_rng(seed)
    H = O.GATE_HIDDEN
    u = lambda *shape: g.uniform(-scale, scale, size=shape).astype(np.float32)
    return {"w1": u(H, k), "b1": u(H), "w2": u(2, H), "b2": u(2)}


@pytest.mark.parametrize("k", [4, 10])
def test_mlp_gate_matches_torch_sequential(k):
    w = _mlp_weights(k)
    net = torch.nn.Sequential(torch.nn.Linear(k, O.GATE_HIDDEN), torch.nn.ReLU(), torch.nn.Linear(O.GATE_HIDDEN, 2)).double()
    with torch.no_grad():
        net[0].weight.copy_(torch.from_numpy(w["w1"]).double()); net[0].bias.copy_(torch.from_numpy(w["b1"]).double())
        net[2].weight.copy_(torch.from_numpy(w["w2"]).double()); net[2].bias.copy_(torch.from_numpy(w["b2"]).double())
    g = np.random.default_rng(9)
    for _ in range(5):
        x = g.random(k)
        with torch.no_grad():
            ty = net(torch.from_numpy(x))
        assert np.allclose(O.gate_step_mlp(x, w), ty.numpy(), atol=1e-12)


def test_mlp_gate_is_the_lstm_gate_with_the_recurrent_columns_cut():
    """With the head's columns for the LSTM output zeroed, the paper's model no longer sees its state and
    must equal the memoryless policy on the remaining columns; and zero weights give the output bias."""
    cfg = W.shrink(W.CONFIGS[2], k=6)
    w = {n: (v * 5).astype(np.float32) for n, v in W.gate_weights(cfg).items()}
    H = O.GATE_HIDDEN
    w["w1"][:, :H] = 0
    wm = {"w1": w["w1"][:, H:].copy(), "b1": w["b1"], "w2": w["w2"], "b2": w["b2"]}
    g = np.random.default_rng(2)
    h = np.zeros(H); c = np.zeros(H)
    for _ in range(4):
        x = g.random(6)
        y, h, c = O.gate_step(x, h, c, w)
        assert np.allclose(y, O.gate_step_mlp(x, wm), atol=1e-12)
    wz = {n: np.zeros_like(v) for n, v in wm.items()}
    wz["b2"][:] = [0.5, -2.0]
    assert O.gate_step_mlp(np.ones(6), wz).tolist() == [0.5, -2.0]


def test_policy_variants_drive_the_expansion():
    cfg = W.CONFIGS[1]
    draft = W.draft_logits(cfg, 0)
    k, t_max, H = cfg.k, cfg.t_max, O.GATE_HIDDEN
    # memoryless policy: a bias that always continues runs to t_max, one that always stops makes one call
    wm = {n: np.zeros_like(v) for n, v in _mlp_weights(k).items()}
    wm["b2"][:] = [0.0, 1.0]
    _, trace = O.run_expansion(draft, k, t_max, wm, policy="mlp_scores")
    assert len(trace) == t_max and not any(tr["h"].any() for tr in trace)      # no recurrent state is kept
    wm["b2"][:] = [1.0, 0.0]
    _, trace = O.run_expansion(draft, k, t_max, wm, policy="mlp_scores")
    assert len(trace) == 1
    # hidden-state policy: the gate sees features[t-1] at call t and nothing of the scores
    d_in = 24
    g = np.random.default_rng(4)
    u = lambda *shape: g.uniform(-0.3, 0.3, size=shape).astype(np.float32)
    w = {"w_ih": u(4 * H, d_in), "w_hh": u(4 * H, H), "b_ih": u(4 * H), "b_hh": u(4 * H),
         "w1": u(H, H + d_in), "b1": u(H), "w2": u(2, H), "b2": u(2)}
    feats = g.standard_normal((t_max - 1, d_in)).astype(np.float32)
    _, trace = O.run_expansion(draft, k, t_max, w, policy="lstm_hidden", features=feats, force_calls=3)
    h = np.zeros(H); c = np.zeros(H)
    for t, tr in enumerate(trace[:2], start=1):
        y, h, c = O.gate_step(feats[t - 1].astype(np.float64), h, c, w)
        h, c = h.astype(np.float32), c.astype(np.float32)
        assert np.allclose(tr["gate_logits"], y, atol=1e-12)


def test_gate_zero_weights_returns_output_bias():
    w = {n: np.zeros_like(v) for n, v in W.gate_weights(W.CONFIGS[1]).items()}
    w["b2"][:] = [0.25, -1.5]
    y, h, c = O.gate_step(np.ones(4), np.zeros(128), np.zeros(128), w)
    assert y.tolist() == [0.25, -1.5] and not h.any() and not c.any()
    assert O.gate_decision(y) is False
    assert O.gate_decision(np.array([0.0, 0.0])) is False      # tie stops
    assert O.gate_decision(np.array([0.0, 1e-9])) is True


def test_gate_schedule_first_call_always_and_never_after_tmax():
    cfg = W.CONFIGS[1]
    draft = W.draft_logits(cfg, 0)
    w = {n: np.zeros_like(v) for n, v in W.gate_weights(cfg).items()}
    w["b2"][:] = [1.0, 0.0]                                   # always stop
    pool, trace = O.run_expansion(draft, cfg.k, cfg.t_max, w)
    assert len(trace) == 1 and "gate_logits" in trace[0]
    w["b2"][:] = [0.0, 1.0]                                   # always continue
    pool, trace = O.run_expansion(draft, cfg.k, cfg.t_max, w)
    assert len(trace) == cfg.t_max
    assert all("gate_logits" in tr for tr in trace[:-1]) and "gate_logits" not in trace[-1]
    assert trace[-1]["cont"] is False


def test_gate_input_is_exp_of_frontier_scores_descending():
    cfg = W.CONFIGS[1]
    draft = W.draft_logits(cfg, 0)
    seen = []
    orig = O.gate_step

    def spy(x, h, c, w):
        seen.append(np.array(x))
        return orig(x, h, c, w)
    O.gate_step = spy
    try:
        pool, trace = O.run_expansion(draft, cfg.k, cfg.t_max, W.gate_weights(cfg), force_calls=3)
    finally:
        O.gate_step = orig
    for x, tr in zip(seen, trace):
        assert np.all(x >= 0) and np.all(x <= 1) and np.all(np.diff(x) <= 0)
        assert np.allclose(x, np.exp(tr["frontier_score"]), rtol=1e-6)


# ---- rerank / tree ---------------------------------------------------------------
def _random_pool(seed, k=3, T=3, t_max=4, V=40):
    cfg = W.shrink(W.CONFIGS[1], cid=100 + seed, V=V, k=k, t_max=t_max)
    draft = W.draft_logits(cfg, 0)
    pool, _ = O.run_expansion(draft, k, t_max, W.gate_weights(cfg), force_calls=T)
    return pool


def _ancestors(parent, i):
    out = set()
    while i != -1:
        out.add(i)
        i = int(parent[i])
    return out


@pytest.mark.parametrize("seed", range(6))
def test_mask_is_exactly_ancestors_and_self(seed):
    pool = _random_pool(seed)
    tree = O.rerank_build_tree(pool, N=10 + seed, root_tok=5, prefix_len=77, t_max=4)
    M = tree["n_nodes"]
    assert M == min(10 + seed, pool.len) + 1
    for i in range(M):
        anc = _ancestors(tree["parent"], i)
        bits = {t for t in range(64) if (int(tree["mask"][i]) >> t) & 1}
        assert bits == anc
        assert bin(int(tree["mask"][i])).count("1") == tree["depth"][i] + 1
        assert int(tree["mask"][i]) < 2 ** (i + 1) and int(tree["mask"][i]) & 1
        assert tree["pos"][i] == 77 + tree["depth"][i]
        if i:
            assert tree["parent"][i] < i
            assert tree["tok"][i] == pool.tok[tree["pool_idx"][i]]
            assert tree["score"][i] == pool.score[tree["pool_idx"][i]]
    assert tree["tok"][0] == 5 and tree["parent"][0] == -1 and tree["depth"][0] == 0
    assert all(tree["mask"][i] == 0 for i in range(M, 64))
    # serialisation is in ascending pool index
    assert np.all(np.diff(tree["pool_idx"][1:M]) > 0)


def test_rerank_is_the_best_subset_and_ancestor_closed_bruteforce():
    pool = _random_pool(11, k=2, T=3, t_max=3)               # 2 + 4 + 4 = 10 candidates
    assert pool.len == 10
    for N in (1, 3, 5, 9, 10, 14):
        tree = O.rerank_build_tree(pool, N, 0, 0, 3)
        n_eff = min(N, pool.len)
        kept = set(tree["pool_idx"][1:tree["n_nodes"]].tolist())
        best = max(itertools.combinations(range(pool.len), n_eff),
                   key=lambda c: sum(float(pool.score[i]) for i in c))
        assert kept == set(best)
        for p in kept:
            assert pool.parent[p] == -1 or int(pool.parent[p]) in kept


def test_rerank_tie_keeps_lowest_pool_index():
    pool = O.Pool(8)
    pool.len = 4
    pool.tok[:4] = [9, 8, 7, 6]
    pool.parent[:4] = -1
    pool.depth[:4] = 1
    pool.score[:4] = [-1.0, -2.0, -2.0, -2.0]
    tree = O.rerank_build_tree(pool, 2, 0, 0, 2)
    assert tree["pool_idx"][1:3].tolist() == [0, 1] and tree["margin"] == 0.0


@pytest.mark.parametrize("seed", range(4))
def test_retrieve_rows_are_all_root_to_leaf_paths(seed):
    pool = _random_pool(20 + seed, k=3, T=4, t_max=4)
    N = 14
    tree = O.rerank_build_tree(pool, N, 1, 10, 4)
    M = tree["n_nodes"]
    kids = {i: [j for j in range(M) if tree["parent"][j] == i] for i in range(M)}
    paths = []

    def dfs(i, acc):
        if not kids[i]:
            paths.append(acc + [i])
        for j in kids[i]:
            dfs(j, acc + [i])
    dfs(0, [])
    paths.sort(key=lambda p: p[-1])                           # leaves in ascending node index
    assert tree["n_leaves"] == len(paths)
    for r, p in enumerate(paths):
        row = tree["retrieve"][r]
        assert row[: len(p)].tolist() == p and np.all(row[len(p):] == -1)
    assert np.all(tree["retrieve"][len(paths):] == -1)
    # draft_row is set exactly on nodes that have children
    for i in range(M):
        assert (tree["draft_row"][i] >= 0) == bool(kids[i])


def test_single_call_tree_is_a_star():
    cfg = W.CONFIGS[1]
    pool, _ = O.run_expansion(W.draft_logits(cfg, 0), cfg.k, cfg.t_max, W.gate_weights(cfg), force_calls=1)
    tree = O.rerank_build_tree(pool, cfg.N, 3, 128, cfg.t_max)
    assert tree["n_nodes"] == cfg.k + 1 and tree["n_leaves"] == cfg.k
    assert np.all(tree["depth"][1:cfg.k + 1] == 1) and np.all(tree["parent"][1:cfg.k + 1] == 0)
    assert tree["draft_row"][0] == 0
