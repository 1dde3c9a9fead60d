"""Parity at the full sizes of the batched configurations, in the launch configuration the benchmark
times (same `SpecStep`, same workspaces, same grid plans).  The expansion, the tree and the
acceptance are compared in full (the oracle handles them in seconds even at V = 128256); the
attention output is compared on sampled (sequence, query head) pairs that the oracle computes one
by one, chosen to cover the first and last sequence, the longest and the shortest prefix and
both ends of the head range."""
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


def sampled_pairs(cfg, prefix_len, n_random=6):
    B, Hq = cfg.B, cfg.Hq
    longest, shortest = int(np.argmax(prefix_len)), int(np.argmin(prefix_len))
    pairs = {(0, 0), (B - 1, Hq - 1), (longest, Hq // 2), (shortest, 1 % Hq), (longest, Hq - 1), (shortest, 0)}
    g = np.random.Generator(np.random.Philox(1234 + cfg.cid))
    while len(pairs) < 6 + n_random:
        pairs.add((int(g.integers(0, B)), int(g.integers(0, Hq))))
    return sorted(pairs)


@pytest.mark.parametrize("cid", [3, 4, 5])
def test_full_size_step_matches_oracle(ctx, cid):
    import torch
    cfg = W.CONFIGS[cid]
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
    O_gpu, lse_gpu = g.attention()
    pairs = sampled_pairs(cfg, inp["prefix_len"])
    O_ref, lse_ref = H.oracle_attention(cfg, inp, trees, pairs=pairs)
    H.compare_attention(cfg, O_gpu, lse_gpu, O_ref, lse_ref, trees, pairs=pairs)
    # every live output row is finite and rows past a tree's end were left alone (the buffer starts at zero)
    for b in range(cfg.B):
        n = trees[b]["n_nodes"]
        assert np.isfinite(O_gpu[b, :n]).all()
        assert not O_gpu[b, n:].any()

    g.accept(target)
    H.compare_accept(cfg, g, accepts)
    del g
    torch.cuda.empty_cache()
