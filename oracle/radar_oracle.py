"""Plain fp64 oracle of one RADAR speculative step (numpy, per-sequence loops).

TEST INFRASTRUCTURE ONLY: never imported by the product path.

Every function states the passage of the paper it follows.  Inputs arrive in the
precision of the library's buffers (float32 arrays; bf16 data is widened exactly
to float32 by the caller) and every computation is carried out in float64.
Values that cross a call boundary of the library as float32 buffers (path
scores, the gate's recurrent state) are rounded to float32 by the *driver*
`run_expansion` when it chains calls, exactly as the buffers would.

Selections use (value descending, index ascending): the lowest index wins ties.
Each float-keyed selection also reports its *margin* (the smallest gap that
would have to close for the decision to change) so that a parity test can tell
a rounding-order difference from a bug.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

M_MAX = 64          # tree rows (root + draft nodes) fit one 64-bit ancestor mask
GATE_HIDDEN = 128   # App. "Implementation Details": hidden_size = 128

# Readings of the paper where its text leaves a choice (each is one named switch).
GATE_INPUT_CUMULATIVE = True   # the gate sees exp(cumulative path log-prob) of the k survivors
GATE_TIE_STOPS = True          # equal logits -> action 0 (stop)
N_COUNTS_ROOT = False          # the rerank size N counts draft nodes only


# --------------------------------------------------------------------------
# a1: vocabulary pass
# --------------------------------------------------------------------------
def log_softmax(z) -> np.ndarray:
    """log of the softmax probabilities of one logits row.

    The draft model's confidence score of a token is its softmax probability
    (Sec. 4.2, state definition: c_i in [0,1]); the tree works with its log.
    """
    z = np.asarray(z, dtype=np.float64)
    m = np.max(z)
    return z - m - np.log(np.sum(np.exp(z - m)))


def order_desc(values) -> np.ndarray:
    """Indices sorted by (value descending, index ascending)."""
    v = np.asarray(values, dtype=np.float64)
    return np.argsort(-v, kind="stable")


def vocab_topk(z, k: int):
    """Top-k tokens of one row and their log-probabilities (Sec. 4.2, state s_t).

    The order is taken on the raw logits: log-softmax is strictly monotone, so
    it is the same order, and it does not depend on how the normaliser is
    summed.
    """
    z = np.asarray(z)
    if z.shape[0] < k:
        raise ValueError("vocabulary smaller than k")
    idx = order_desc(z)[:k]
    return idx.astype(np.int32), log_softmax(z)[idx]


# --------------------------------------------------------------------------
# D1: candidate pool (every node any draft call has produced)
# --------------------------------------------------------------------------
@dataclass
class Pool:
    capacity: int
    tok: np.ndarray = field(init=False)
    parent: np.ndarray = field(init=False)     # pool index of the parent, -1 = root
    score: np.ndarray = field(init=False)      # cumulative log-prob, float32 storage
    depth: np.ndarray = field(init=False)      # 1-based draft call that produced it
    draft_row: np.ndarray = field(init=False)  # row of the next call's logits where it is expanded, -1 = never
    len: int = 0

    def __post_init__(self):
        c = self.capacity
        self.tok = np.full(c, -1, np.int32)
        self.parent = np.full(c, -1, np.int32)
        self.score = np.zeros(c, np.float32)
        self.depth = np.zeros(c, np.int32)
        self.draft_row = np.full(c, -1, np.int32)


def pool_capacity(k: int, t_max: int) -> int:
    """k candidates from the first call (one row), k*k from each later call."""
    return k + (t_max - 1) * k * k


# --------------------------------------------------------------------------
# a1 + a2: one draft call's expansion for one sequence
# --------------------------------------------------------------------------
def expand_step_seq(logits, parent_score, parent_pool_idx, pool: Pool, t: int, k: int):
    """One expansion (App. "Inference Pipeline Walkthrough").

    Every frontier row yields its k most probable tokens; a child's score is its
    parent's path score plus its own log-probability; all F*k children enter
    the pool; the k best of them (over all parents together, as in the
    walkthrough where the two survivors have different parents) form the next
    frontier.

    logits [F,V] float32, parent_score [F] float32, parent_pool_idx [F] int.
    Returns a dict; `margin` is the smallest gap between neighbours among the
    best k+1 candidate scores (frontier order and membership both depend on it).
    """
    logits = np.asarray(logits)
    F, V = logits.shape
    topk_tok = np.zeros((F, k), np.int32)
    topk_logp = np.zeros((F, k), np.float64)
    for f in range(F):
        topk_tok[f], topk_logp[f] = vocab_topk(logits[f], k)
    cand = np.asarray(parent_score, np.float64)[:, None] + topk_logp      # [F,k]
    base = pool.len
    if base + F * k > pool.capacity:
        raise ValueError("pool overflow")
    for f in range(F):
        for j in range(k):
            p = base + f * k + j
            pool.tok[p] = topk_tok[f, j]
            pool.parent[p] = parent_pool_idx[f]
            pool.score[p] = np.float32(cand[f, j])
            pool.depth[p] = t
    pool.len = base + F * k
    flat = cand.reshape(-1)
    order = order_desc(flat)
    sel = order[:k]
    head = flat[order[: min(k + 1, flat.size)]]
    gaps = -np.diff(head)
    gaps = gaps[np.isfinite(gaps)]
    margin = float(np.min(gaps)) if gaps.size else np.inf
    for slot, s in enumerate(sel):
        pool.draft_row[base + s] = 1 + (t - 1) * k + slot
    return {
        "topk_tok": topk_tok,
        "topk_logp": topk_logp,
        "frontier_tok": topk_tok.reshape(-1)[sel].astype(np.int32),
        "frontier_score": flat[sel],
        "frontier_local_logp": topk_logp.reshape(-1)[sel],
        "frontier_pool_idx": (base + sel).astype(np.int32),
        "frontier_src_row": (sel // k).astype(np.int32),
        "margin": margin,
        # which candidates the margin is about (reporting only): pool indices and scores of the best k+1
        "head_pool_idx": (base + order[: min(k + 1, flat.size)]).astype(np.int64),
        "head_score": head.copy(),
    }


# --------------------------------------------------------------------------
# a3: prediction model (single-layer LSTM + two-layer MLP head)
# --------------------------------------------------------------------------
def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def gate_step(x, h, c, w):
    """One call of the prediction model (Sec. 4.2 and App. "Implementation Details").

    x: the k confidence scores in [0,1]; (h, c): recurrent state, zero at the
    first call of a speculative step.  Textbook LSTM cell with gate blocks in the
    order input, forget, cell, output and two bias vectors; the LSTM output is
    concatenated with x and sent through Linear(H+k -> H), ReLU, Linear(H -> 2).
    Dropout is the identity at inference.  Returns (y[2], h', c').
    Action 1 = continue, action 0 = stop (action space of the MDP).
    """
    x = np.asarray(x, np.float64)
    h = np.asarray(h, np.float64)
    c = np.asarray(c, np.float64)
    W_ih, W_hh = np.asarray(w["w_ih"], np.float64), np.asarray(w["w_hh"], np.float64)
    b_ih, b_hh = np.asarray(w["b_ih"], np.float64), np.asarray(w["b_hh"], np.float64)
    W1, b1 = np.asarray(w["w1"], np.float64), np.asarray(w["b1"], np.float64)
    W2, b2 = np.asarray(w["w2"], np.float64), np.asarray(w["b2"], np.float64)
    H = h.shape[0]
    pre = W_ih @ x + b_ih + W_hh @ h + b_hh
    i = _sigmoid(pre[0:H])
    f = _sigmoid(pre[H:2 * H])
    g = np.tanh(pre[2 * H:3 * H])
    o = _sigmoid(pre[3 * H:4 * H])
    c_new = f * c + i * g
    h_new = o * np.tanh(c_new)
    hidden = np.maximum(W1 @ np.concatenate([h_new, x]) + b1, 0.0)
    y = W2 @ hidden + b2
    return y, h_new, c_new


def gate_step_mlp(x, w):
    """The memoryless policy of the ablation (Table 3, "MLP / scores"; Sec. 4.2: it uses only the
    confidence scores as its state).  The paper gives no layer sizes for it; the reading taken here is
    the prediction model's own two-layer head without the LSTM in front: Linear(k -> H), ReLU,
    Linear(H -> 2), with w["w1"] of shape [H, k].  Returns y[2]."""
    x = np.asarray(x, np.float64)
    W1, b1 = np.asarray(w["w1"], np.float64), np.asarray(w["b1"], np.float64)
    W2, b2 = np.asarray(w["w2"], np.float64), np.asarray(w["b2"], np.float64)
    assert W1.shape[1] == x.shape[0]
    return W2 @ np.maximum(W1 @ x + b1, 0.0) + b2


def gate_decision(y) -> bool:
    """Deterministic reading of the binary control signal: continue iff logit 1 wins."""
    return bool(y[1] > y[0]) if GATE_TIE_STOPS else bool(y[1] >= y[0])


# --------------------------------------------------------------------------
# a4 loop: dynamic expansion for one sequence
# --------------------------------------------------------------------------
def run_expansion(draft_logits, k: int, t_max: int, gate_w, force_calls: int | None = None,
                  policy: str = "lstm_scores", features=None):
    """Draft-tree expansion for one sequence (Sec. 4.1; Eq. for T_pred).

    draft_logits [1+(t_max-1)k, V] float32: row 0 feeds call 1, rows
    1+(t-2)k .. 1+(t-1)k-1 feed call t >= 2 (one row per frontier slot).
    The gate runs after every call except call t_max (the paper drops that call
    because generation terminates anyway).  `force_calls` overrides the gate
    (used for workloads whose depth the harness fixes).
    `policy` selects the ablation variants of Table 3: "lstm_scores" (the paper's model),
    "mlp_scores" (gate_step_mlp; no recurrent state) and "lstm_hidden" (the same LSTM + head fed
    with the draft model's hidden state of the call instead of the scores: `features`
    [t_max-1, d_in] float32, row t-1 for call t; which hidden vector that is - the paper does not
    say - is the caller's choice).
    Returns (pool, trace) where trace holds per-call outputs and margins.
    """
    assert policy in ("lstm_scores", "mlp_scores", "lstm_hidden")
    H = GATE_HIDDEN
    pool = Pool(pool_capacity(k, t_max))
    h = np.zeros(H, np.float32)
    c = np.zeros(H, np.float32)
    parent_score = np.zeros(1, np.float32)
    parent_pool_idx = np.full(1, -1, np.int32)
    trace = []
    t = 1
    while True:
        rows = draft_logits[0:1] if t == 1 else draft_logits[1 + (t - 2) * k: 1 + (t - 1) * k]
        out = expand_step_seq(rows, parent_score, parent_pool_idx, pool, t, k)
        out["t"] = t
        cont = False
        if t < t_max:
            scores = out["frontier_score"] if GATE_INPUT_CUMULATIVE else out["frontier_local_logp"]
            x = np.exp(np.asarray(scores, np.float32).astype(np.float64))
            if policy == "mlp_scores":
                y = gate_step_mlp(x, gate_w)
            else:
                inp = x if policy == "lstm_scores" else np.asarray(features[t - 1], np.float32).astype(np.float64)
                y, h_new, c_new = gate_step(inp, h, c, gate_w)
                h, c = h_new.astype(np.float32), c_new.astype(np.float32)
            out["gate_logits"] = y
            out["gate_margin"] = float(abs(y[1] - y[0]))
            cont = gate_decision(y)
            if force_calls is not None:
                cont = t < force_calls
        out["cont"] = cont
        out["h"], out["c"] = h.copy(), c.copy()
        trace.append(out)
        if not cont:
            break
        parent_score = out["frontier_score"].astype(np.float32)
        parent_pool_idx = out["frontier_pool_idx"]
        t += 1
    return pool, trace


# --------------------------------------------------------------------------
# a4: rerank + serialise the tree
# --------------------------------------------------------------------------
def rerank_build_tree(pool: Pool, N: int, root_tok: int, prefix_len: int, t_max: int):
    """Top-N rerank of every candidate and serialisation for one masked pass.

    (Sec. 1: the candidates are organised as a tree that is serialised and
    verified through masked attention in one pass; Sec. 2.3: nodes are reordered
    and pruned by confidence.)  Keep the N best pool entries by path score, lay
    them out after the root in ascending pool index (parents precede children,
    siblings stay in descending probability), and derive parent, depth,
    ancestor mask, position id, leaves and root-to-leaf retrieve rows.
    """
    L = pool.len
    n_eff = min(N - 1 if N_COUNTS_ROOT else N, L)
    if n_eff + 1 > M_MAX:
        raise ValueError("tree does not fit a 64-bit mask")
    order = order_desc(pool.score[:L])
    margin = np.inf
    cut_pair = None                     # the last kept and the first dropped entry (reporting only)
    if n_eff < L and n_eff > 0:
        margin = float(np.float64(pool.score[order[n_eff - 1]]) - np.float64(pool.score[order[n_eff]]))
        cut_pair = (int(order[n_eff - 1]), int(order[n_eff]))
    kept = np.sort(order[:n_eff])
    M = n_eff + 1
    node_of = {-1: 0}
    for r, p in enumerate(kept):
        node_of[int(p)] = r + 1
    tok = np.full(M_MAX, -1, np.int32)
    parent = np.full(M_MAX, -1, np.int32)
    depth = np.zeros(M_MAX, np.int32)
    pos = np.zeros(M_MAX, np.int32)
    pidx = np.full(M_MAX, -1, np.int32)
    score = np.zeros(M_MAX, np.float32)
    drow = np.full(M_MAX, -1, np.int32)
    mask = np.zeros(M_MAX, np.uint64)
    tok[0], pos[0], mask[0], drow[0] = root_tok, prefix_len, np.uint64(1), 0
    for r, p in enumerate(kept):
        i = r + 1
        pp = int(pool.parent[p])
        if pp not in node_of:
            raise AssertionError("kept set is not ancestor-closed")
        tok[i] = pool.tok[p]
        parent[i] = node_of[pp]
        depth[i] = depth[parent[i]] + 1
        if depth[i] != pool.depth[p]:
            raise AssertionError("depth mismatch")
        pos[i] = prefix_len + depth[i]
        pidx[i] = p
        score[i] = pool.score[p]
        drow[i] = pool.draft_row[p]
        mask[i] = mask[parent[i]] | (np.uint64(1) << np.uint64(i))
    has_child = np.zeros(M, bool)
    for i in range(1, M):
        has_child[parent[i]] = True
    for i in range(M):
        if not has_child[i]:
            drow[i] = -1                      # a node without children consults no draft row
    leaves = [i for i in range(M) if not has_child[i]]
    if M == 1:
        leaves = []                           # a root-only tree has no draft path to retrieve
    retrieve = np.full((N, t_max + 1), -1, np.int32)
    for l, leaf in enumerate(leaves):
        chain = []
        i = leaf
        while i != -1:
            chain.append(i)
            i = int(parent[i])
        chain.reverse()
        retrieve[l, : len(chain)] = chain
    return {
        "n_nodes": M, "tok": tok, "parent": parent, "depth": depth, "pos": pos,
        "pool_idx": pidx, "score": score, "draft_row": drow, "mask": mask,
        "retrieve": retrieve, "n_leaves": len(leaves), "margin": margin, "cut_pair": cut_pair,
    }


# --------------------------------------------------------------------------
# a5: tree-masked verification attention
# --------------------------------------------------------------------------
def tree_attention_head(q, k_prefix, v_prefix, k_tree, v_tree, mask, n_nodes, scale):
    """Masked softmax attention of the tree's queries for one (sequence, q-head).

    (Sec. 3: the target model scores the whole draft in one parallel pass;
    Sec. 1: the tree is verified via masked attention.)  Node i attends to every
    prefix position and to tree position t iff bit t of mask[i] is set.
    q [M,d]; k_prefix, v_prefix [P,d]; k_tree, v_tree [M,d] -> out [n_nodes,d],
    lse [n_nodes] (natural-log normaliser of the scaled scores).
    """
    q = np.asarray(q, np.float64)[:n_nodes]
    K = np.concatenate([np.asarray(k_prefix, np.float64), np.asarray(k_tree, np.float64)[:n_nodes]], 0)
    Vv = np.concatenate([np.asarray(v_prefix, np.float64), np.asarray(v_tree, np.float64)[:n_nodes]], 0)
    P = k_prefix.shape[0]
    s = (q @ K.T) * scale                                   # [n,P+n]
    allowed = np.ones_like(s, dtype=bool)
    for i in range(n_nodes):
        for t in range(n_nodes):
            allowed[i, P + t] = bool((int(mask[i]) >> t) & 1)
    s = np.where(allowed, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    den = e.sum(axis=1, keepdims=True)
    out = (e / den) @ Vv
    return out, (m + np.log(den))[:, 0]


def tree_attention(Q, Kc, Vc, Kt, Vt, mask, n_nodes, prefix_len, scale=None, pairs=None):
    """All (sequence, head) pairs, or only those listed in `pairs`.

    Q [B,64,Hq,d]; Kc,Vc: list of per-sequence prefix caches [P_b,Hkv,d];
    Kt,Vt [B,64,Hkv,d]; mask [B,64] uint64.  KV head of q-head h is h // (Hq/Hkv).
    Returns O [B,64,Hq,d] (rows >= n_nodes left at 0) and lse [B,Hq,64].
    """
    B, _, Hq, d = Q.shape
    Hkv = Kt.shape[2]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    O = np.zeros((B, M_MAX, Hq, d), np.float64)
    lse = np.zeros((B, Hq, M_MAX), np.float64)
    todo = pairs if pairs is not None else [(b, h) for b in range(B) for h in range(Hq)]
    for b, h in todo:
        n = int(n_nodes[b])
        P = int(prefix_len[b])
        g = h // G
        o, l = tree_attention_head(Q[b, :, h], Kc[b][:P, g], Vc[b][:P, g], Kt[b, :, g], Vt[b, :, g],
                                   mask[b], n, scale)
        O[b, :n, h] = o
        lse[b, h, :n] = l
    return O, lse


# --------------------------------------------------------------------------
# a6: greedy acceptance (temperature 0)
# --------------------------------------------------------------------------
def children_of(parent, n_nodes, c):
    return [j for j in range(1, n_nodes) if parent[j] == c]


def best_retrieve_row(retrieve, n_leaves, path):
    for r in range(n_leaves):
        if all(retrieve[r, d] == path[d] for d in range(len(path))):
            return r
    return -1


def verify_greedy(target_logits, tree, t_max: int):
    """Longest path whose tokens the target model would itself have produced.

    (Temperature-0 rows of the temperature study; Sec. 3 with a deterministic
    target.)  At the current node take the target's argmax (lowest index on
    ties); move to the child carrying that token, else stop.  The argmax at the
    last accepted node is the next token.  target_logits [>=n_nodes, V].
    """
    n = tree["n_nodes"]
    a = [int(np.argmax(np.asarray(target_logits[i]))) for i in range(n)]
    cur, path = 0, [0]
    while True:
        nxt = [j for j in children_of(tree["parent"], n, cur) if tree["tok"][j] == a[cur]]
        if not nxt:
            break
        cur = nxt[0]
        path.append(cur)
    path_nodes = np.full(t_max + 1, -1, np.int32)
    path_tokens = np.full(t_max + 1, -1, np.int32)
    path_nodes[: len(path)] = path
    path_tokens[: len(path)] = tree["tok"][path]
    return {
        "accept_len": len(path) - 1, "path_nodes": path_nodes, "path_tokens": path_tokens,
        "next_token": a[cur], "best_retrieve_row": best_retrieve_row(tree["retrieve"], tree["n_leaves"], path),
        "argmax": np.asarray(a, np.int32),
    }
