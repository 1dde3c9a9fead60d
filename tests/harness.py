"""Shared test harness: draws one workload with the seeded generators, runs the CPU oracle
on it and (on a GPU machine) the CUDA library on the same bits, and compares.  Inputs flow
generator -> {oracle, CUDA}; nothing the CUDA path produces is ever fed to the oracle.
"""
from __future__ import annotations

import numpy as np

from oracle import accept_oracle as A
from oracle import radar_oracle as O
from paper_2512_14069_b200 import workloads as W

TAU_SCORE = 1e-5        # margin below which a float-keyed selection is declared a near-tie
TAU_PROB = 1e-9         # same, for accept tests / inverse-CDF draws (both sides evaluate them in fp64)
TOL_SCORE = 1e-5        # log-prob scores and gate logits (fp32 path)
TOL_ATTN = {"f32": 1e-5, "bf16": 2e-2}


def make_inputs(cfg: W.Config, with_attention=True, with_kv=True):
    B = cfg.B
    inp = {
        "draft": np.stack([W.draft_logits(cfg, b) for b in range(B)]),
        "gate": W.gate_weights(cfg),
        "force_calls": W.forced_calls(cfg),
        "n_keep": np.minimum(W.keep_sizes(cfg), cfg.N).astype(np.int32),
        "root_tok": W.root_tokens(cfg),
        "prefix_len": W.prefix_lens(cfg),
    }
    if with_attention:
        inp["Q"] = np.stack([W.attn_q(cfg, b) for b in range(B)])
        kt, vt = zip(*[W.attn_tree_kv(cfg, b) for b in range(B)])
        inp["Kt"], inp["Vt"] = np.stack(kt), np.stack(vt)
        if with_kv:
            kc, vc = zip(*[W.attn_prefix_kv(cfg, b, int(inp["prefix_len"][b])) for b in range(B)])
            inp["Kc"], inp["Vc"] = list(kc), list(vc)
    ua, us = W.accept_uniforms(cfg)
    inp["u_accept"], inp["u_sample"] = ua, us
    return inp


def oracle_expand_and_tree(cfg: W.Config, inp):
    pools, traces, trees = [], [], []
    for b in range(cfg.B):
        fc = None if inp["force_calls"] is None else int(inp["force_calls"][b])
        pool, trace = O.run_expansion(inp["draft"][b], cfg.k, cfg.t_max, inp["gate"], force_calls=fc)
        tree = O.rerank_build_tree(pool, int(inp["n_keep"][b]), int(inp["root_tok"][b]), int(inp["prefix_len"][b]),
                                   cfg.t_max)
        pools.append(pool)
        traces.append(trace)
        trees.append(tree)
    return pools, traces, trees


def make_target(cfg: W.Config, inp, trees):
    return np.stack([W.target_logits(cfg, b, inp["draft"][b], trees[b]["draft_row"], trees[b]["n_nodes"])
                     for b in range(cfg.B)])


def oracle_accept(cfg: W.Config, inp, trees, target):
    out = []
    for b in range(cfg.B):
        if cfg.mode == "greedy":
            out.append(O.verify_greedy(target[b], trees[b], cfg.t_max))
        else:
            out.append(A.verify_stochastic(target[b], inp["draft"][b], trees[b], inp["u_accept"][b],
                                           float(inp["u_sample"][b]), float(np.float32(cfg.temperature)), cfg.t_max))
    return out


def oracle_attention(cfg: W.Config, inp, trees, pairs=None):
    n_nodes = np.array([t["n_nodes"] for t in trees])
    mask = np.stack([t["mask"] for t in trees])
    w = lambda x: W.widen(cfg, x)
    need = set(range(cfg.B)) if pairs is None else {b for b, _ in pairs}     # widen only what will be read
    wide = lambda xs: [w(x) if b in need else x[:0] for b, x in enumerate(xs)]
    return O.tree_attention(w(inp["Q"]), wide(inp["Kc"]), wide(inp["Vc"]), w(inp["Kt"]),
                            w(inp["Vt"]), mask, n_nodes, inp["prefix_len"], pairs=pairs)


# ---- CUDA side ---------------------------------------------------------------------------
def to_dev(x, bf16=False):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x))
    if bf16 or x.dtype == np.uint16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


class CudaRun:
    """Uploads a workload and drives the library through `SpecStep`."""

    def __init__(self, cfg: W.Config, inp, ctx=None, max_prefix_len=None, logits_bf16=False):
        import torch
        from paper_2512_14069_b200 import binding as rb
        from paper_2512_14069_b200.pipeline import SpecStep
        self.torch, self.rb, self.cfg, self.inp = torch, rb, cfg, inp
        self.ctx = ctx or rb.Context(0)
        kvdt = torch.float32 if cfg.kv_dtype == "f32" else torch.bfloat16
        mode = rb.RADAR_GREEDY if cfg.mode == "greedy" else rb.RADAR_STOCHASTIC
        mpl = int(max(inp["prefix_len"])) if max_prefix_len is None else max_prefix_len
        self.step = SpecStep(self.ctx, B=cfg.B, V=cfg.V, k=cfg.k, t_max=cfg.t_max, N=cfg.N, Hq=cfg.Hq, Hkv=cfg.Hkv,
                             d=cfg.d, kv_dtype=kvdt, max_prefix_len=mpl, mode=mode,
                             temperature=float(np.float32(cfg.temperature)))
        self.draft = to_dev(inp["draft"])
        if logits_bf16:
            self.draft = self.draft.to(torch.bfloat16)
        self.gate = {n: to_dev(v) for n, v in inp["gate"].items()}
        self.force = None if inp["force_calls"] is None else to_dev(inp["force_calls"])
        self.n_keep = to_dev(inp["n_keep"])
        self.root_tok = to_dev(inp["root_tok"])
        self.prefix_len = to_dev(inp["prefix_len"])

    def expand_and_tree(self):
        s = self.step
        s.run_expansion(self.draft, self.gate, self.force)
        s.build_tree(self.root_tok, self.prefix_len, self.n_keep)
        self.ctx.check_device_status()

    def upload_attention(self, page_size=None, spare_pages=3):
        """Contiguous (packed) prefix cache, or with `page_size` a paged one: the same K/V rows scattered
        over shuffled pages, a block table per sequence, unused table entries -1, and NaN in every cache
        row that belongs to no token (page tails, spare pages), so that a read of them cannot go unnoticed."""
        inp, torch = self.inp, self.torch
        self.Q, self.Kt, self.Vt = to_dev(inp["Q"]), to_dev(inp["Kt"]), to_dev(inp["Vt"])
        self.block_table, self.page_size = None, 0
        if page_size is None:
            self.Kc = to_dev(np.concatenate(inp["Kc"], 0))
            self.Vc = to_dev(np.concatenate(inp["Vc"], 0))
            start = np.concatenate([[0], np.cumsum(inp["prefix_len"])[:-1]]).astype(np.int64)
            self.kv_start = to_dev(start)
            return
        ps = page_size
        need = [(int(p) + ps - 1) // ps for p in inp["prefix_len"]]
        n_pages = sum(need) + spare_pages
        order = np.random.default_rng(1000 + ps).permutation(n_pages)
        max_pages = max(max(need), 1) + 1
        table = np.full((self.cfg.B, max_pages), -1, np.int32)
        sample = inp["Kc"][0]
        nan = np.uint16(0x7FC0) if sample.dtype == np.uint16 else np.float32(np.nan)
        Kc = np.full((n_pages * ps,) + sample.shape[1:], nan, sample.dtype)
        Vc = np.full_like(Kc, nan)
        nxt = 0
        for b in range(self.cfg.B):
            for p in range(need[b]):
                page = int(order[nxt]); nxt += 1
                table[b, p] = page
                rows = inp["Kc"][b][p * ps:(p + 1) * ps]
                Kc[page * ps:page * ps + len(rows)] = rows
                Vc[page * ps:page * ps + len(rows)] = inp["Vc"][b][p * ps:(p + 1) * ps]
        self.Kc, self.Vc = to_dev(Kc), to_dev(Vc)
        self.kv_start = None
        self.block_table, self.page_size = to_dev(table), ps

    def attention(self, trees=None):
        """With `trees` (oracle trees) the masks come from the generator side, so attention can be
        checked independently of the CUDA tree build."""
        s = self.step
        if trees is not None:
            mask = to_dev(np.stack([t["mask"] for t in trees]).view(np.int64))
            n_nodes = to_dev(np.array([t["n_nodes"] for t in trees], np.int32))
        else:
            mask = n_nodes = None
        s.attention(self.Q, self.Kc, self.Vc, self.kv_start, self.prefix_len, self.Kt, self.Vt, mask, n_nodes,
                    block_table=self.block_table, page_size=self.page_size)
        self.ctx.check_device_status()
        return s.O.float().cpu().numpy(), s.lse.cpu().numpy()

    def accept(self, target):
        s = self.step
        tl = to_dev(target)
        if self.draft.dtype != tl.dtype:
            tl = tl.to(self.draft.dtype)
        s.accept(tl, self.draft, to_dev(self.inp["u_accept"]), to_dev(self.inp["u_sample"]))
        self.ctx.check_device_status()


# ---- comparisons -------------------------------------------------------------------------------
def _same_bits_siblings(inp, b, pool, p, q):
    """Pool entries p and q are children of one parent whose logits are bit-identical: both sides then hold
    exactly equal scores for them (the same function of the same inputs) and order them by index."""
    if pool.parent[p] != pool.parent[q]:
        return False
    par = int(pool.parent[p])
    row = 0 if par < 0 else int(pool.draft_row[par])
    z = inp["draft"][b][row]
    return z[pool.tok[p]].tobytes() == z[pool.tok[q]].tobytes()


def check_margins(cfg, traces, trees, accepts=None, inp=None, pools=None):
    """The seeds must not put any float-keyed decision within rounding distance of a tie.  With `inp` and
    `pools`, a gap of exactly zero between siblings whose logits are bit-identical is not a near-tie (low
    precision logits collide often): it is decided by index on both sides."""
    def gap_ok(b, gap, p, q):
        if gap > TAU_SCORE:
            return True
        return gap == 0.0 and inp is not None and _same_bits_siblings(inp, b, pools[b], int(p), int(q))

    for b in range(cfg.B):
        for tr in traces[b]:
            hp, hs = tr["head_pool_idx"], tr["head_score"]
            for a in range(len(hp) - 1):
                gap = float(hs[a] - hs[a + 1])
                assert not np.isfinite(gap) or gap_ok(b, gap, hp[a], hp[a + 1]), ("frontier near-tie", b, tr["t"], gap)
            if "gate_margin" in tr:
                assert tr["gate_margin"] > TAU_SCORE, ("gate near-tie", b, tr["t"], tr["gate_margin"])
        if trees[b]["cut_pair"] is not None:
            assert gap_ok(b, trees[b]["margin"], *trees[b]["cut_pair"]), ("rerank near-tie", b, trees[b]["margin"])
        if accepts is not None and "accept_margin" in accepts[b]:
            assert accepts[b]["accept_margin"] > TAU_PROB and accepts[b]["sample_margin"] > TAU_PROB, (b, accepts[b])


def compare_expansion(cfg, gpu: CudaRun, pools, traces):
    s = gpu.step
    g = lambda t: t.cpu().numpy()
    k = cfg.k
    ft, fs, fp, fr = g(s.frontier_tok), g(s.frontier_score), g(s.frontier_pool_idx), g(s.frontier_src_row)
    tt, tl, tt1, tl1 = g(s.topk_tok), g(s.topk_logp), g(s.topk_tok1), g(s.topk_logp1)
    gl, ch = g(s.gate_logits), g(s.cont_hist)
    ptok, ppar, pdep, pdr, psc, plen = g(s.pool_tok), g(s.pool_parent), g(s.pool_depth), g(s.pool_draft_row), \
        g(s.pool_score), g(s.pool_len)
    hh, cc = g(s.h), g(s.c)
    for b in range(cfg.B):
        pool, trace = pools[b], traces[b]
        for tr in trace:
            i = tr["t"] - 1
            ttok, tlp = (tt1[b], tl1[b]) if tr["t"] == 1 else (tt[i, b], tl[i, b])
            assert np.array_equal(ttok, tr["topk_tok"]), ("topk tokens", b, tr["t"])
            assert np.max(np.abs(tlp - tr["topk_logp"])) <= TOL_SCORE
            assert np.array_equal(ft[i, b], tr["frontier_tok"]), ("frontier tokens", b, tr["t"])
            assert np.array_equal(fp[i, b], tr["frontier_pool_idx"])
            assert np.array_equal(fr[i, b], tr["frontier_src_row"])
            assert np.max(np.abs(fs[i, b] - tr["frontier_score"])) <= TOL_SCORE
            assert bool(ch[i, b]) == tr["cont"], ("continue/stop", b, tr["t"])
            if "gate_logits" in tr:
                assert np.max(np.abs(gl[i, b] - tr["gate_logits"])) <= TOL_SCORE, ("gate logits", gl[i, b], tr["gate_logits"])
        L = pool.len
        assert plen[b] == L
        assert np.array_equal(ptok[b, :L], pool.tok[:L]) and np.array_equal(ppar[b, :L], pool.parent[:L])
        assert np.array_equal(pdep[b, :L], pool.depth[:L]) and np.array_equal(pdr[b, :L], pool.draft_row[:L])
        assert np.max(np.abs(psc[b, :L].astype(np.float64) - pool.score[:L])) <= TOL_SCORE
        assert np.max(np.abs(hh[b] - trace[-1]["h"])) <= TOL_SCORE and np.max(np.abs(cc[b] - trace[-1]["c"])) <= TOL_SCORE
        # calls after the stop must not have touched anything of this sequence
        for i in range(len(trace), cfg.t_max):
            assert ch[i, b] == 0


def compare_tree(cfg, gpu: CudaRun, trees):
    s = gpu.step
    g = lambda t: t.cpu().numpy()
    for b in range(cfg.B):
        t = trees[b]
        assert g(s.n_nodes)[b] == t["n_nodes"] and g(s.n_leaves)[b] == t["n_leaves"]
        assert np.array_equal(g(s.tree_tok)[b], t["tok"]) and np.array_equal(g(s.tree_parent)[b], t["parent"])
        assert np.array_equal(g(s.tree_depth)[b], t["depth"]) and np.array_equal(g(s.tree_pos)[b], t["pos"])
        assert np.array_equal(g(s.tree_pool_idx)[b], t["pool_idx"])
        assert np.array_equal(g(s.tree_draft_row)[b], t["draft_row"])
        assert np.array_equal(g(s.tree_mask)[b].view(np.uint64), t["mask"])
        assert np.max(np.abs(g(s.tree_score)[b].astype(np.float64) - t["score"])) <= TOL_SCORE
        rows = t["retrieve"].shape[0]                     # the oracle was given this sequence's own N
        assert np.array_equal(g(s.retrieve)[b, :rows], t["retrieve"]) and np.all(g(s.retrieve)[b, rows:] == -1)


def compare_accept(cfg, gpu: CudaRun, accepts):
    s = gpu.step
    g = lambda t: t.cpu().numpy()
    for b in range(cfg.B):
        a = accepts[b]
        assert g(s.accept_len)[b] == a["accept_len"], ("accept_len", b, g(s.accept_len)[b], a["accept_len"])
        assert np.array_equal(g(s.path_nodes)[b], a["path_nodes"]) and np.array_equal(g(s.path_tokens)[b], a["path_tokens"])
        assert g(s.next_token)[b] == a["next_token"], ("next_token", b, g(s.next_token)[b], a["next_token"])
        assert g(s.best_retrieve_row)[b] == a["best_retrieve_row"]


def compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees, pairs=None):
    tol = TOL_ATTN[cfg.kv_dtype]
    todo = pairs if pairs is not None else [(b, h) for b in range(cfg.B) for h in range(cfg.Hq)]
    worst = 0.0
    for b, h in todo:
        n = trees[b]["n_nodes"]
        worst = max(worst, float(np.max(np.abs(O_gpu[b, :n, h] - O_ref[b, :n, h]))))
        assert np.max(np.abs(lse_gpu[b, h, :n] - lse_ref[b, h, :n])) <= max(tol, 1e-4)
    assert worst <= tol, ("attention max-abs error", worst, tol)
    return worst
