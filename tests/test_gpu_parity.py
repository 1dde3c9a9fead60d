"""Parity of the CUDA library (through the C ABI) against the CPU oracle on the same seeded
inputs.  Needs a B200.  Sizes: the two small paper configurations in full, the batched ones
reduced so that the oracle finishes in seconds while every kernel still spans several tiles,
chunks and a ragged tail."""
import numpy as np
import pytest

import harness as H
from paper_2512_14069_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2512_14069_b200 import binding as rb
    c = rb.Context(0)
    yield c
    c.close()


def small(cid):
    """Reduced copies of the batched configurations (same head layout, dtype, k, t_max, N, mode)."""
    cfg = W.CONFIGS[cid]
    if cid == 3:
        return W.shrink(cfg, B=3, Hq=8, Hkv=8, P=(1500, 1500), V=32000)
    if cid == 4:
        return W.shrink(cfg, B=3, Hq=16, Hkv=2, P=(1100, 1100), V=20011)       # odd V: unaligned rows
    if cid == 5:
        return W.shrink(cfg, B=4, Hq=8, Hkv=2, P=(300, 2100), V=30002)
    return cfg


@pytest.mark.parametrize("cid", [1, 2, 3, 4, 5])
def test_whole_step_matches_oracle(ctx, cid):
    cfg = small(cid)
    inp = H.make_inputs(cfg)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    target = H.make_target(cfg, inp, trees)
    accepts = H.oracle_accept(cfg, inp, trees, target)
    H.check_margins(cfg, traces, trees, accepts)

    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    H.compare_tree(cfg, g, trees)

    g.upload_attention()
    O_gpu, lse_gpu = g.attention()                      # masks from the CUDA tree build
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)

    g.accept(target)
    H.compare_accept(cfg, g, accepts)


@pytest.mark.parametrize("name", ["fixed_depth_greedy", "chain_greedy", "chain_stochastic"])
def test_regression_workloads_match_oracle(ctx, name):
    """The fixed schedule the paper compares with (gate off, every sequence makes all t_max calls) and
    chain drafts (k = 1: the tree is a path, its mask is causal, and stochastic acceptance is the
    single-draft rule of Eq. 1-2)."""
    if name == "fixed_depth_greedy":
        cfg = W.shrink(W.CONFIGS[2], B=3, V=9001, P=(700, 700), depth_plan="fixed_tmax")
    elif name == "chain_greedy":
        cfg = W.shrink(W.CONFIGS[2], B=3, V=9001, P=(700, 700), k=1, N=7, depth_plan="fixed_tmax")
    else:
        cfg = W.shrink(W.CONFIGS[3], B=3, Hq=8, Hkv=8, V=9001, P=(700, 700), k=1, t_max=6, N=5, depth_plan="fixed_tmax")
    inp = H.make_inputs(cfg)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    assert all(len(t) == cfg.t_max for t in traces)
    if cfg.k == 1:
        for t in trees:                                   # a path: node i's ancestors are 0..i
            assert all(int(t["mask"][i]) == (1 << (i + 1)) - 1 for i in range(t["n_nodes"]))
    target = H.make_target(cfg, inp, trees)
    accepts = H.oracle_accept(cfg, inp, trees, target)
    H.check_margins(cfg, traces, trees, accepts)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    H.compare_tree(cfg, g, trees)
    g.upload_attention()
    O_gpu, lse_gpu = g.attention()
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)
    g.accept(target)
    H.compare_accept(cfg, g, accepts)


@pytest.mark.parametrize("policy,feat_dim", [("mlp_scores", 0), ("lstm_hidden", 64), ("lstm_hidden", 4096)])
def test_policy_variants_match_oracle(ctx, policy, feat_dim):
    """The policy networks of the ablation (Table 3): memoryless MLP on the scores, and the LSTM fed with
    a hidden-state vector (a small one and one of the draft model's width).  Same comparisons as the
    paper's model: every call's outputs, gate logits within 1e-5, continue/stop bit-exact, final h and c."""
    from oracle import radar_oracle as O
    from paper_2512_14069_b200 import binding as rb
    cfg = W.shrink(W.CONFIGS[2], B=5, V=9001, depth_plan="gate")
    inp = H.make_inputs(cfg, with_attention=False)
    w = W.policy_weights(cfg, policy, feat_dim)
    feats = W.gate_features(cfg, feat_dim) if feat_dim else None
    pools, traces = [], []
    for b in range(cfg.B):
        pool, trace = O.run_expansion(inp["draft"][b], cfg.k, cfg.t_max, w, policy=policy,
                                      features=None if feats is None else feats[:, b])
        pools.append(pool)
        traces.append(trace)
        for tr in trace:
            assert tr["margin"] > H.TAU_SCORE and tr.get("gate_margin", 1.0) > H.TAU_SCORE
    assert len({len(t) for t in traces}) > 1 or policy == "mlp_scores"      # the hidden-state gate stops at different depths
    g = H.CudaRun(cfg, inp, ctx)
    code = rb.RADAR_POLICY_MLP_SCORES if policy == "mlp_scores" else rb.RADAR_POLICY_LSTM_HIDDEN
    g.step.run_expansion(g.draft, {n: H.to_dev(v) for n, v in w.items()}, None, policy=code,
                         features=None if feats is None else H.to_dev(feats))
    ctx.check_device_status()
    H.compare_expansion(cfg, g, pools, traces)


@pytest.mark.parametrize("cid,temperature", [(1, 1.0), (3, 1.0), (5, 0.7), (2, 0.5)])
def test_accept_length_distribution_matches_oracle(ctx, cid, temperature):
    """Eq. 11-13 for every tree of the batch: p_0..p_tmax and P_acc of every row against the fp64 oracle.
    Both sides work in fp64 and differ only in summation order: 1e-9 absolute is generous."""
    import torch
    from oracle import accept_oracle as A
    from paper_2512_14069_b200 import binding as rb
    cfg = small(cid) if cid != 2 else W.shrink(W.CONFIGS[2], V=30011)
    inp = H.make_inputs(cfg, with_attention=False)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    target = H.make_target(cfg, inp, trees)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_tree(cfg, g, trees)
    s = g.step
    dist = torch.full((cfg.B, cfg.t_max + 1), -1.0, dtype=torch.float64, device="cuda")
    pacc = torch.full((cfg.B, 64), -1.0, dtype=torch.float64, device="cuda")
    wb = rb.radar_acclen_workspace_bytes(ctx, cfg.B, cfg.V)
    ws = torch.zeros(wb + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    rb.radar_accept_length_distribution(
        ctx, B=cfg.B, V=cfg.V, t_max=cfg.t_max, temperature=float(np.float32(temperature)), target_logits=H.to_dev(target),
        tree_tok=s.tree_tok, tree_parent=s.tree_parent, tree_depth=s.tree_depth, tree_draft_row=s.tree_draft_row,
        n_nodes=s.n_nodes, draft_logits=g.draft, R=s.R, dist=dist, p_acc_node=pacc, workspace=ws[off:off + wb])
    ctx.check_device_status()
    dist, pacc = dist.cpu().numpy(), pacc.cpu().numpy()
    for b in range(cfg.B):
        d_ref, p_ref = A.accept_length_distribution(target[b], inp["draft"][b], trees[b], float(np.float32(temperature)),
                                                    cfg.t_max)
        n = trees[b]["n_nodes"]
        assert np.max(np.abs(dist[b] - d_ref)) < 1e-9, (b, dist[b], d_ref)
        assert np.max(np.abs(pacc[b, :n] - p_ref)) < 1e-9 and not pacc[b, n:].any()
        assert abs(dist[b].sum() - 1.0) < 1e-9


@pytest.mark.parametrize("cid,mode", [(1, "greedy"), (3, "greedy"), (1, "stochastic"), (3, "stochastic")])
def test_bf16_logits_with_many_ties(ctx, cid, mode):
    """bf16 logits collide often: token order must still be (value desc, id asc) bit for bit, and the whole
    expansion, the tree, both acceptance modes and Eq. 11-13 must match the oracle on bf16 logits.  Equal logits
    under one parent give exactly equal scores on both sides (decided by index), so such zero gaps are not
    near-ties; every other float-keyed decision must still clear the margin."""
    import torch
    from oracle import accept_oracle as A
    from paper_2512_14069_b200 import binding as rb
    cfg = W.shrink(small(cid), mode=mode)
    inp = H.make_inputs(cfg, with_attention=False)
    inp["draft"] = W.bf16_bits_to_f32(W.f32_to_bf16_bits(inp["draft"])).reshape(inp["draft"].shape)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    target = H.make_target(cfg, inp, trees)
    target = W.bf16_bits_to_f32(W.f32_to_bf16_bits(target)).reshape(target.shape)
    accepts = H.oracle_accept(cfg, inp, trees, target)
    H.check_margins(cfg, traces, trees, accepts, inp=inp, pools=pools)
    assert any(tr["margin"] == 0.0 for b in range(cfg.B) for tr in traces[b]), "the case is meant to contain exact ties"

    g = H.CudaRun(cfg, inp, ctx, logits_bf16=True)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    H.compare_tree(cfg, g, trees)
    g.accept(target)
    H.compare_accept(cfg, g, accepts)
    if mode == "stochastic":
        # Eq. 11-13 on the same bf16 logits
        s = g.step
        T = float(np.float32(cfg.temperature))
        dist = torch.full((cfg.B, cfg.t_max + 1), -1.0, dtype=torch.float64, device="cuda")
        pacc = torch.full((cfg.B, 64), -1.0, dtype=torch.float64, device="cuda")
        wb = rb.radar_acclen_workspace_bytes(ctx, cfg.B, cfg.V)
        ws = torch.zeros(wb + 256, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 256
        rb.radar_accept_length_distribution(
            ctx, B=cfg.B, V=cfg.V, t_max=cfg.t_max, temperature=T, target_logits=H.to_dev(target).to(torch.bfloat16),
            tree_tok=s.tree_tok, tree_parent=s.tree_parent, tree_depth=s.tree_depth, tree_draft_row=s.tree_draft_row,
            n_nodes=s.n_nodes, draft_logits=g.draft, R=s.R, dist=dist, p_acc_node=pacc, workspace=ws[off:off + wb])
        ctx.check_device_status()
        dist, pacc = dist.cpu().numpy(), pacc.cpu().numpy()
        for b in range(cfg.B):
            d_ref, p_ref = A.accept_length_distribution(target[b], inp["draft"][b], trees[b], T, cfg.t_max)
            n = trees[b]["n_nodes"]
            assert np.max(np.abs(dist[b] - d_ref)) < 1e-9 and np.max(np.abs(pacc[b, :n] - p_ref)) < 1e-9


def test_attention_with_oracle_masks_and_ragged_trees(ctx):
    """Attention alone, masks and tree sizes taken from the oracle: ragged prefixes and trees,
    a root-only tree, a prefix shorter than one tile, GQA with G = 4."""
    cfg = W.shrink(W.CONFIGS[5], B=5, Hq=8, Hkv=2, P=(1, 900), V=2000, k=4, t_max=5, N=40)
    inp = H.make_inputs(cfg)
    inp["prefix_len"][0] = 1
    inp["Kc"][0], inp["Vc"][0] = inp["Kc"][0][:1], inp["Vc"][0][:1]
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    trees[1] = dict(trees[1]); trees[1]["n_nodes"] = 1                        # root only
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention()
    O_gpu, lse_gpu = g.attention(trees)
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)


@pytest.mark.parametrize("Hq,Hkv,d", [(8, 8, 64), (8, 4, 64), (16, 1, 128), (6, 3, 128), (24, 8, 128)])
def test_attention_bf16_head_layouts(ctx, Hq, Hkv, d):
    """bf16 tensor-core path at head_dim 64 and 128, G = 1, 2 and 16 (eight row blocks), and G = 3, which the
    tensor-core path does not take (falls to the FMA kernel): ragged prefixes incl. an empty one, ragged trees."""
    cfg = W.shrink(W.CONFIGS[5], cid=80 + Hq + d, B=4, Hq=Hq, Hkv=Hkv, d=d, P=(0, 700), V=2000, k=4, t_max=5, N=50)
    inp = H.make_inputs(cfg)
    inp["prefix_len"][0] = 0
    inp["Kc"][0], inp["Vc"][0] = inp["Kc"][0][:0], inp["Vc"][0][:0]
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    trees[2] = dict(trees[2]); trees[2]["n_nodes"] = 1
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention()
    O_gpu, lse_gpu = g.attention(trees)
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)


@pytest.mark.parametrize("page_size,Hq,Hkv,dtype", [(16, 8, 2, "bf16"), (64, 8, 8, "bf16"), (128, 16, 2, "bf16"),
                                                    (256, 8, 2, "bf16"), (32, 6, 3, "bf16"), (16, 4, 2, "f32")])
def test_attention_paged_prefix_cache(ctx, page_size, Hq, Hkv, dtype):
    """The prefix K/V scattered over shuffled pages (16 to 256 tokens) and read through a block table: same
    outputs as the oracle computes from the logical rows.  Ragged prefixes, one empty, one shorter than a page,
    one ending exactly on a page boundary; rows of the cache that belong to no token hold NaN.
    (6 query / 3 KV heads and fp32 take the FMA kernel, the others the tensor-core kernel.)"""
    base = W.CONFIGS[5] if dtype == "bf16" else W.CONFIGS[1]
    cfg = W.shrink(base, cid=120 + page_size + Hq, B=5, Hq=Hq, Hkv=Hkv, d=128 if dtype == "bf16" else 64,
                   P=(200, 1500), V=2000, k=4, t_max=5, N=50)
    inp = H.make_inputs(cfg)
    for b, plen in ((0, 0), (1, 5), (2, 4 * page_size)):
        inp["prefix_len"][b] = plen
        inp["Kc"][b], inp["Vc"][b] = W.attn_prefix_kv(cfg, b, plen) if plen else (inp["Kc"][b][:0], inp["Vc"][b][:0])
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention(page_size=page_size)
    O_gpu, lse_gpu = g.attention(trees)
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)


def test_attention_paged_reports_bad_page(ctx):
    """A block-table entry outside the cache is reported on the device status word; nothing faults."""
    import torch
    from paper_2512_14069_b200 import binding as rb
    cfg = W.shrink(W.CONFIGS[5], cid=97, B=2, Hq=8, Hkv=2, P=(300, 300), V=2000, k=4, t_max=4, N=30)
    inp = H.make_inputs(cfg)
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention(page_size=64)
    table = g.block_table.cpu().numpy().copy()
    table[1, 2] = 10 ** 6
    g.block_table = H.to_dev(table)
    s = g.step
    mask = H.to_dev(np.stack([t["mask"] for t in trees]).view(np.int64))
    n_nodes = H.to_dev(np.array([t["n_nodes"] for t in trees], np.int32))
    s.attention(g.Q, g.Kc, g.Vc, None, g.prefix_len, g.Kt, g.Vt, mask, n_nodes, block_table=g.block_table, page_size=64)
    torch.cuda.synchronize()
    assert ctx.read_device_status() == -1
    assert ctx.read_device_status() == rb.RADAR_OK


def test_attention_long_prefix_many_segments(ctx):
    """One long and three short sequences: the long one's units are cut across many CTAs (partials + combine),
    the short ones share CTAs with it."""
    cfg = W.shrink(W.CONFIGS[5], cid=99, B=4, Hq=8, Hkv=2, P=(100, 100), V=2000, k=4, t_max=5, N=60)
    inp = H.make_inputs(cfg)
    long_len = 40000
    inp["prefix_len"][1] = long_len
    kc, vc = W.attn_prefix_kv(cfg, 1, long_len)
    inp["Kc"][1], inp["Vc"][1] = kc, vc
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention()
    O_gpu, lse_gpu = g.attention(trees)
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)


@pytest.mark.parametrize("kind", ["bf16_tensor_core", "f32_fma", "bf16_fma"])
def test_attention_reports_prefix_beyond_cache(ctx, kind):
    """A prefix that would read past the cache is refused on the device status word by both kernels (the
    tensor-core one, and the FMA one for fp32 and for bf16 head ratios the tensor path does not take); the
    sequence is skipped before anything of the cache is read, so nothing faults, and the other sequence's
    output is still right."""
    import torch
    from paper_2512_14069_b200 import binding as rb
    if kind == "f32_fma":
        cfg = W.shrink(W.CONFIGS[1], cid=97, B=2, Hq=4, Hkv=2, P=(300, 300), V=2000, k=4, t_max=4, N=30)
    else:
        Hq = 8 if kind == "bf16_tensor_core" else 6
        cfg = W.shrink(W.CONFIGS[5], cid=98, B=2, Hq=Hq, Hkv=2, P=(300, 300), V=2000, k=4, t_max=4, N=30)
    inp = H.make_inputs(cfg)
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx, max_prefix_len=4096)
    g.upload_attention()
    g.prefix_len = H.to_dev(np.array([300, 4000], np.int32))          # sequence 1 claims more rows than the cache holds
    s = g.step
    mask = H.to_dev(np.stack([t["mask"] for t in trees]).view(np.int64))
    n_nodes = H.to_dev(np.array([t["n_nodes"] for t in trees], np.int32))
    path = rb.radar_tree_attention_path(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, Q=g.Q, Kc=g.Kc, Vc=g.Vc, kv_start=g.kv_start,
                                        prefix_len=g.prefix_len, max_prefix_len=4096, Kt=g.Kt, Vt=g.Vt, mask=mask,
                                        n_nodes=n_nodes, O=s.O, workspace=s.ws_attn)
    assert path == (rb.RADAR_ATTN_PATH_TENSOR_CORE if kind == "bf16_tensor_core" else rb.RADAR_ATTN_PATH_FMA)
    s.attention(g.Q, g.Kc, g.Vc, g.kv_start, g.prefix_len, g.Kt, g.Vt, mask, n_nodes)
    torch.cuda.synchronize()
    assert ctx.read_device_status() == -1
    assert ctx.read_device_status() == rb.RADAR_OK
    O_ref, _ = H.oracle_attention(cfg, inp, trees, pairs=[(0, h) for h in range(cfg.Hq)])
    n0 = trees[0]["n_nodes"]
    assert np.max(np.abs(s.O.float().cpu().numpy()[0, :n0] - O_ref[0, :n0])) <= H.TOL_ATTN[cfg.kv_dtype]


def test_attention_fp32_head_dim_64_and_128(ctx):
    for d in (64, 128):
        cfg = W.shrink(W.CONFIGS[1], cid=40 + d, B=2, Hq=4, Hkv=2, d=d, P=(257, 257))
        inp = H.make_inputs(cfg)
        _, _, trees = H.oracle_expand_and_tree(cfg, inp)
        g = H.CudaRun(cfg, inp, ctx)
        g.upload_attention()
        O_gpu, lse_gpu = g.attention(trees)
        O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
        H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)


@pytest.mark.parametrize("k,V", [(1, 77), (32, 4099), (7, 33), (32, 32003)])
def test_expansion_edge_sizes(ctx, k, V):
    """k = 1, k = 32 (the limit) and a vocabulary barely larger than k; k = 32 at V = 32003 is the size at which
    the staged chunk records no longer fit next to the gate weights, so the unstaged merge has to take over."""
    t_max = 3 if k == 32 else 4
    cfg = W.shrink(W.CONFIGS[1], cid=60 + k, V=V, k=k, t_max=t_max, N=min(63, 3 * k), B=2, gate_b2_offset=5.0)
    inp = H.make_inputs(cfg, with_attention=False)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    H.check_margins(cfg, traces, trees)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    H.compare_tree(cfg, g, trees)


@pytest.mark.parametrize("B", [2, 20])
def test_gate_with_and_without_helper_blocks(ctx, B):
    """The select + gate kernel runs as a cluster of four blocks per sequence while 8 B blocks fit the device (three
    of them hold W_hh in shared memory and deliver W_hh h into the first), and as one block per sequence beyond
    that.  B = 2 takes the first form, B = 20 the second; gate state and decisions must match the oracle in both."""
    cfg = W.shrink(W.CONFIGS[1], cid=80 + B, B=B, V=5003, k=6, t_max=6, N=30, gate_b2_offset=0.5)   # every call runs
    inp = H.make_inputs(cfg, with_attention=False)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    H.check_margins(cfg, traces, trees)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    H.compare_tree(cfg, g, trees)


def test_minus_inf_logits_and_nan_status(ctx):
    import torch
    cfg = W.shrink(W.CONFIGS[1], cid=70, B=1)
    inp = H.make_inputs(cfg, with_attention=False)
    inp["draft"][0, :, 5:200] = -np.inf
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_expansion(cfg, g, pools, traces)
    # a NaN is reported through the status word, nothing faults
    inp["draft"][0, 0, 17] = np.nan
    g2 = H.CudaRun(cfg, inp, ctx)
    g2.step.run_expansion(g2.draft, g2.gate, g2.force)
    from paper_2512_14069_b200 import binding as rb
    assert ctx.read_device_status() == -6
    assert ctx.read_device_status() == rb.RADAR_OK          # reading clears it
    torch.cuda.synchronize()


def test_host_side_argument_errors(ctx):
    import torch
    from paper_2512_14069_b200 import binding as rb
    cfg = W.CONFIGS[1]
    inp = H.make_inputs(cfg, with_attention=False)
    g = H.CudaRun(cfg, inp, ctx)
    s = g.step
    with pytest.raises(rb.RadarError) as e:
        s.k = 33
        s.expand(1, g.draft, g.gate)
    assert e.value.status == -2
    s.k = cfg.k
    with pytest.raises(rb.RadarError) as e:
        ws = s.ws_expand
        s.ws_expand = ws[:16]
        s.expand(1, g.draft, g.gate)
    assert e.value.status == -3
    s.ws_expand = ws
    with pytest.raises(rb.RadarError) as e:
        s.d = 96
        s.attention(s.O, s.O, s.O, torch.zeros(1, dtype=torch.int64, device="cuda"), g.prefix_len, s.O, s.O)
    assert e.value.status == -2
    s.d = cfg.d
    # a tensor that does not start on a 16-byte boundary is refused on the host by either kernel (nothing is launched)
    qbuf = torch.zeros(s.O.numel() + 4, dtype=s.O.dtype, device="cuda")
    q_off = qbuf[2:2 + s.O.numel()].view(s.O.shape)                  # 8 bytes past an aligned address (fp32)
    kvz = torch.zeros(cfg.B * 64, cfg.Hkv, cfg.d, dtype=s.O.dtype, device="cuda")
    with pytest.raises(rb.RadarError) as e:
        s.attention(q_off, kvz, kvz, torch.zeros(cfg.B, dtype=torch.int64, device="cuda"), g.prefix_len, kvz.view(cfg.B, 64, cfg.Hkv, cfg.d),
                    kvz.view(cfg.B, 64, cfg.Hkv, cfg.d))
    assert e.value.status == -1
    # policy variants: an unknown policy, a hidden-state policy without features or with a ragged feature width
    for kw in (dict(policy=7), dict(policy=rb.RADAR_POLICY_LSTM_HIDDEN),
               dict(policy=rb.RADAR_POLICY_LSTM_HIDDEN, features=torch.zeros(cfg.t_max - 1, cfg.B, 6, device="cuda"))):
        with pytest.raises(rb.RadarError) as e:
            s.expand(1, g.draft, g.gate, **kw)
        assert e.value.status == -1
    # the memoryless policy needs only its own four tensors
    mlp = {n: H.to_dev(v) for n, v in W.policy_weights(cfg, "mlp_scores").items()}
    s.expand(1, g.draft, mlp, policy=rb.RADAR_POLICY_MLP_SCORES)
    # paged cache: a page size that is neither 16/32/64 nor a multiple of 128, and a table too short for the prefix
    kv = torch.zeros(512, cfg.Hkv, cfg.d, device="cuda")
    table = torch.zeros(cfg.B, 1, dtype=torch.int32, device="cuda")
    for ps in (48, 64):
        with pytest.raises(rb.RadarError) as e:
            s.attention(s.O, kv, kv, None, g.prefix_len, s.O[:, :, :cfg.Hkv], s.O[:, :, :cfg.Hkv], block_table=table, page_size=ps)
        assert e.value.status == -1, ps
    torch.cuda.synchronize()
    assert ctx.read_device_status() == 0


def test_stochastic_acceptance_with_minus_inf_logits(ctx):
    """-inf logits are legal (probability 0).  The accept call alone, on trees built from clean inputs, with
    draft / target logits edited so that the walk meets: a child whose draft probability is 0 but whose target
    probability is positive (accepted whatever the uniform), a child with both 0 (rejected), a draft row whose
    whole mass sits on the rejected child (the sibling loop stops, the residual is sampled), and -inf scattered
    over a fifth of both tensors."""
    cfg = small(3)
    assert cfg.mode == "stochastic"
    inp = H.make_inputs(cfg, with_attention=False)
    pools, traces, trees = H.oracle_expand_and_tree(cfg, inp)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    H.compare_tree(cfg, g, trees)
    target = H.make_target(cfg, inp, trees).copy()
    draft = inp["draft"].copy()
    rng = np.random.Generator(np.random.Philox(4242))
    for b in range(cfg.B):
        draft[b][rng.random(draft[b].shape) < 0.2] = -np.inf
        target[b][rng.random(target[b].shape) < 0.2] = -np.inf
        t = trees[b]
        kids = [j for j in range(1, t["n_nodes"]) if t["parent"][j] == 0]
        x1, row = int(t["tok"][kids[0]]), int(t["draft_row"][0])
        for j in kids:                                   # the root's children start from finite logits on both sides
            draft[b, row, t["tok"][j]] = inp["draft"][b, row, t["tok"][j]]
            target[b, 0, t["tok"][j]] = 0.0
        if b == 0:
            draft[b, row, x1] = -np.inf                  # q(x1) = 0 < p(x1): accepted
        elif b == 1:
            draft[b, row, x1] = -np.inf                  # q(x1) = p(x1) = 0: rejected, the siblings follow
            target[b, 0, x1] = -np.inf
        else:
            keep = draft[b, row, x1]
            draft[b, row, :] = -np.inf                   # all draft mass on x1 ...
            draft[b, row, x1] = keep
            target[b, 0, x1] = -40.0                     # ... which the target all but excludes: rejected, nothing left to propose
    inp2 = dict(inp, draft=draft)
    accepts = H.oracle_accept(cfg, inp2, trees, target)
    assert accepts[0]["accept_len"] >= 1 and accepts[2]["accept_len"] == 0
    for b in range(cfg.B):
        assert accepts[b]["accept_margin"] > H.TAU_PROB and accepts[b]["sample_margin"] > H.TAU_PROB, (b, accepts[b])
    g.draft = H.to_dev(draft)
    g.inp = inp2
    g.accept(target)
    H.compare_accept(cfg, g, accepts)


@pytest.mark.parametrize("kind", ["bf16_tensor_core", "bf16_two_row_blocks", "f32_fma"])
def test_attention_several_layers_in_one_call(ctx, kind):
    """The multi-layer form: L sets of Q / K / V that share one tree per sequence, every layer against the oracle.
    On the tensor-core path all layers run in one persistent launch (units of a layer repeat per layer and the
    ranges of the CTAs run across layer boundaries); the FMA path goes layer by layer."""
    import torch
    from paper_2512_14069_b200 import binding as rb
    L = 3
    if kind == "f32_fma":
        base = W.shrink(W.CONFIGS[1], cid=150, B=2, Hq=4, Hkv=2, P=(100, 400), V=2000, k=4, t_max=4, N=30)
    elif kind == "bf16_two_row_blocks":
        base = W.shrink(W.CONFIGS[5], cid=151, B=3, Hq=16, Hkv=2, P=(200, 1500), V=2000, k=4, t_max=5, N=50)
    else:
        base = W.shrink(W.CONFIGS[5], cid=152, B=4, Hq=8, Hkv=8, P=(0, 900), V=2000, k=4, t_max=5, N=40)
    inp0 = H.make_inputs(base)
    if kind == "bf16_tensor_core":
        inp0["prefix_len"][0] = 0
    _, _, trees = H.oracle_expand_and_tree(base, inp0)
    plen = inp0["prefix_len"]
    layers = []
    for l in range(L):                                  # every layer draws its own Q / K / V (another stream id), same lengths
        c = W.shrink(base, cid=base.cid + 10 * (l + 1))
        inp = {"Q": np.stack([W.attn_q(c, b) for b in range(c.B)]), "prefix_len": plen}
        kt, vt = zip(*[W.attn_tree_kv(c, b) for b in range(c.B)])
        inp["Kt"], inp["Vt"] = np.stack(kt), np.stack(vt)
        kc, vc = zip(*[W.attn_prefix_kv(c, b, int(plen[b])) for b in range(c.B)])
        inp["Kc"], inp["Vc"] = list(kc), list(vc)
        layers.append(inp)
    stack = lambda name: H.to_dev(np.stack([inp[name] for inp in layers]))
    Q, Kt, Vt = stack("Q"), stack("Kt"), stack("Vt")
    Kc = H.to_dev(np.stack([np.concatenate(inp["Kc"], 0) for inp in layers]))
    Vc = H.to_dev(np.stack([np.concatenate(inp["Vc"], 0) for inp in layers]))
    kv_start = H.to_dev(np.concatenate([[0], np.cumsum(plen)[:-1]]).astype(np.int64))
    mask = H.to_dev(np.stack([t["mask"] for t in trees]).view(np.int64))
    n_nodes = H.to_dev(np.array([t["n_nodes"] for t in trees], np.int32))
    O = torch.zeros_like(Q)
    lse = torch.zeros(L, base.B, base.Hq, 64, device="cuda")
    maxp = int(max(plen))
    wb = rb.radar_attn_workspace_bytes(ctx, base.B, base.Hq, base.Hkv, base.d, rb.dtype_code(Q), maxp)
    ws = torch.zeros(wb + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    kw = dict(B=base.B, Hq=base.Hq, Hkv=base.Hkv, d=base.d, Q=Q, Kc=Kc, Vc=Vc, kv_start=kv_start, prefix_len=H.to_dev(plen),
              max_prefix_len=maxp, Kt=Kt, Vt=Vt, mask=mask, n_nodes=n_nodes, O=O, lse=lse, workspace=ws[off:off + wb], n_layers=L)
    assert rb.radar_tree_attention_path(**kw) == (rb.RADAR_ATTN_PATH_FMA if kind == "f32_fma" else rb.RADAR_ATTN_PATH_TENSOR_CORE)
    rb.radar_tree_attention(ctx, **kw)
    ctx.check_device_status()
    O_gpu, lse_gpu = O.float().cpu().numpy(), lse.cpu().numpy()
    for l in range(L):
        O_ref, lse_ref = H.oracle_attention(base, layers[l], trees)
        H.compare_attention(base, O_gpu[l], lse_gpu[l], O_ref, lse_ref, trees)
    # rows past a tree's end stay untouched in every layer
    for b in range(base.B):
        assert not O_gpu[:, b, trees[b]["n_nodes"]:].any()


@pytest.mark.parametrize("Hq,Hkv,P", [(8, 2, (6000, 9000)), (4, 4, (5000, 7000)), (16, 2, (9000, 14000))])
def test_attention_scores_far_above_the_running_maximum(ctx, Hq, Hkv, P):
    """Keys that score 100 to 300 doublings above everything their row has seen before, one in almost every tile
    (each aimed at another query row, at varying places of the tile), plus: both column halves of one tile for
    one row, the same row in consecutive tiles with growing size, the last prefix key and the tree tile.  The
    running maximum of a row then jumps again and again, by far more than the lazy-rescaling threshold, and
    everything accumulated before has to be scaled away exactly.  Long prefixes, so that a CTA runs several
    tiles of a unit; units with two live row blocks and with one."""
    cfg = W.shrink(W.CONFIGS[5], cid=140 + Hq, B=3, Hq=Hq, Hkv=Hkv, d=128, P=P, V=2000, k=4, t_max=5, N=50)
    inp = H.make_inputs(cfg)
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    G = Hq // Hkv

    def plant(b, key, node, head, alpha, tree=False):
        q = W.bf16_bits_to_f32(inp["Q"][b][node, head])
        dst = inp["Kt"][b] if tree else inp["Kc"][b]
        dst[key, head // G] = W.f32_to_bf16_bits(alpha * q)

    for b in range(cfg.B):
        Pb, n = int(inp["prefix_len"][b]), trees[b]["n_nodes"]
        assert Pb >= 5000 and n >= 4
        for t in range(1, Pb // 128):
            if t % 7 == 3:
                continue                                       # some tiles stay ordinary
            plant(b, t * 128 + (37 * t + 5 * b) % 128, t % n, (3 * t + b) % Hq, 8.0 + t % 3)
        plant(b, 10 * 128 + 10, 3, 1, 14.0)                    # both halves of one tile, one row
        plant(b, 10 * 128 + 70, 3, 1, 19.0)
        plant(b, 11 * 128 + 40, 3, 1, 25.0)                    # and the same row again in the next tile
        plant(b, Pb - 1, 0, Hq // 2, 16.0)                     # the last prefix key
        plant(b, 0, n - 1, 0, 30.0, tree=True)                 # the root's key in the tree tile: every row sees it
    g = H.CudaRun(cfg, inp, ctx)
    g.upload_attention()
    O_gpu, lse_gpu = g.attention(trees)
    assert ctx.read_device_status() == 0
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees)
    assert float(np.max(lse_ref)) > 100.0                      # the planted keys do dominate their rows
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees)
