"""The workspace-free greedy acceptance entry point against the regular one.

Some hosts of the library cannot allocate device memory when they get to the acceptance step:
a serving engine that has given every free byte of the GPU to its own cache pool, or a decode
loop that must not pay cudaMalloc's device-wide synchronisation.  For them the library carries a
fixed 1 MiB scratch array of its own.  This test drives that entry point through the C ABI twice
in a row (the second call finds the first call's records still in the array) with different
inputs and requires bit-identical results to radar_verify_accept, which gets a caller workspace,
and to the CPU oracle's greedy walk; it also checks that a call leaves the amount of free device
memory as it found it (the context's creation has already made the driver load what the path needs).
It is collected last so that a stop-at-first-failure run has already covered everything else.
"""
import numpy as np
import pytest

import harness as H
from paper_2512_14069_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _outputs(step):
    return [t.clone() for t in (step.accept_len, step.path_nodes, step.path_tokens, step.next_token,
                                step.best_retrieve_row)]


def test_noalloc_greedy_accept_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2512_14069_b200 import binding as rb
    ctx = rb.Context(0)
    cfg = W.shrink(W.CONFIGS[4], B=3, Hq=8, Hkv=2, P=(64, 64), V=20011)
    inp = H.make_inputs(cfg, with_attention=False)
    g = H.CudaRun(cfg, inp, ctx)
    g.expand_and_tree()
    s = g.step
    n_nodes = s.n_nodes.cpu().numpy()
    drow = s.tree_draft_row.cpu().numpy()
    # two different sets of target logits: the second call must not be influenced by the first one's records
    targets = []
    for sigma in (1.0, 0.05):
        c = W.shrink(cfg, target_sigma=sigma)
        targets.append(H.to_dev(np.stack([W.target_logits(c, b, inp["draft"][b], drow[b], int(n_nodes[b]))
                                          for b in range(cfg.B)])))
    from oracle import radar_oracle as O
    _, _, trees = H.oracle_expand_and_tree(cfg, inp)
    expected = []
    for tl in targets:
        s.accept(tl)
        torch.cuda.synchronize()
        expected.append(_outputs(s))
        for b in range(cfg.B):                                  # the regular entry point itself against the oracle
            ref = O.verify_greedy(tl[b].cpu().numpy(), trees[b], cfg.t_max)
            assert int(s.accept_len[b]) == ref["accept_len"] and int(s.next_token[b]) == ref["next_token"]
            assert np.array_equal(s.path_nodes[b].cpu().numpy(), ref["path_nodes"])
    assert not torch.equal(expected[0][0], expected[1][0]) or not torch.equal(expected[0][3], expected[1][3])

    for it, (tl, exp) in enumerate(zip(targets, expected)):     # two calls in a row on the shared scratch
        for t in (s.accept_len, s.path_nodes, s.path_tokens, s.next_token, s.best_retrieve_row):
            t.fill_(-7)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rb.radar_verify_accept_greedy_noalloc(
            ctx, B=cfg.B, V=cfg.V, t_max=cfg.t_max, N=cfg.N, target_logits=tl, tree_tok=s.tree_tok,
            tree_parent=s.tree_parent, n_nodes=s.n_nodes, retrieve=s.retrieve, n_leaves=s.n_leaves,
            accept_len=s.accept_len, path_nodes=s.path_nodes, path_tokens=s.path_tokens, next_token=s.next_token,
            best_retrieve_row=s.best_retrieve_row)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        for got, want in zip(_outputs(s), exp):
            assert torch.equal(got, want)                       # integer outputs: exact
        for b in range(cfg.B):                                  # and directly against the oracle
            ref = O.verify_greedy(tl[b].cpu().numpy(), trees[b], cfg.t_max)
            assert int(s.accept_len[b]) == ref["accept_len"] and int(s.next_token[b]) == ref["next_token"]
            assert int(s.best_retrieve_row[b]) == ref["best_retrieve_row"]
    assert ctx.read_device_status() == 0

    # a batch whose records cannot fit the fixed array is refused on the host, nothing is launched
    assert rb.radar_noalloc_scratch_bytes() == 1 << 20
    with pytest.raises(rb.RadarError) as e:
        rb.radar_verify_accept_greedy_noalloc(
            ctx, B=4096, V=128256, t_max=cfg.t_max, N=cfg.N, target_logits=None, tree_tok=None, tree_parent=None,
            n_nodes=None, retrieve=None, n_leaves=None, accept_len=None, path_nodes=None, path_tokens=None,
            next_token=None, best_retrieve_row=None)
    assert e.value.status == -2
    ctx.close()
