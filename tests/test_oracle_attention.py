"""Pins of the oracle's tree attention against library attention and closed-form
special cases.  CPU only."""
import numpy as np
import torch
import torch.nn.functional as F

from oracle import radar_oracle as O


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _chain_mask(n):
    m = np.zeros(64, np.uint64)
    for i in range(n):
        m[i] = np.uint64((1 << (i + 1)) - 1)
    return m


def test_chain_tree_equals_causal_sdpa_with_gqa():
    B, Hq, Hkv, d, P, n = 2, 4, 2, 16, 9, 6
    Q = _rand((B, 64, Hq, d), 0)
    Kc = [_rand((P + b, Hkv, d), 10 + b) for b in range(B)]
    Vc = [_rand((P + b, Hkv, d), 20 + b) for b in range(B)]
    Kt, Vt = _rand((B, 64, Hkv, d), 1), _rand((B, 64, Hkv, d), 2)
    mask = np.stack([_chain_mask(n)] * B)
    plen = np.array([P, P + 1])
    Oo, lse = O.tree_attention(Q, Kc, Vc, Kt, Vt, mask, np.array([n, n]), plen)
    for b in range(B):
        Pb = plen[b]
        Kall = torch.from_numpy(np.concatenate([Kc[b], Kt[b, :n]], 0)).double()      # [Pb+n,Hkv,d]
        Vall = torch.from_numpy(np.concatenate([Vc[b], Vt[b, :n]], 0)).double()
        Kall = Kall.repeat_interleave(Hq // Hkv, dim=1).permute(1, 0, 2)              # [Hq,L,d]
        Vall = Vall.repeat_interleave(Hq // Hkv, dim=1).permute(1, 0, 2)
        q = torch.from_numpy(Q[b, :n]).double().permute(1, 0, 2)                      # [Hq,n,d]
        allow = torch.ones(n, Pb + n, dtype=torch.bool)
        allow[:, Pb:] = torch.tril(torch.ones(n, n, dtype=torch.bool))
        ref = F.scaled_dot_product_attention(q, Kall, Vall, attn_mask=allow)           # [Hq,n,d]
        assert np.allclose(Oo[b, :n], ref.permute(1, 0, 2).numpy(), atol=1e-12)
        s = torch.einsum("hnd,hld->hnl", q, Kall) / np.sqrt(d)
        s = s.masked_fill(~allow, float("-inf"))
        assert np.allclose(lse[b, :, :n], torch.logsumexp(s, -1).numpy(), atol=1e-12)
    assert not Oo[:, n:].any()


def test_branching_mask_each_node_sees_only_its_ancestors():
    # root -> {1, 2}; 1 -> {3}; 2 -> {4}.  Node 3 must ignore tree keys 2 and 4.
    d, P = 8, 5
    parent = [-1, 0, 0, 1, 2]
    mask = np.zeros(64, np.uint64)
    for i, p in enumerate(parent):
        mask[i] = (mask[p] if p >= 0 else np.uint64(0)) | np.uint64(1 << i)
    q = _rand((64, d), 3); kp = _rand((P, d), 4); vp = _rand((P, d), 5)
    kt = _rand((64, d), 6); vt = _rand((64, d), 7)
    out, _ = O.tree_attention_head(q, kp, vp, kt, vt, mask, 5, 0.5)
    for i in range(5):
        anc = [t for t in range(5) if (int(mask[i]) >> t) & 1]
        K = np.concatenate([kp, kt[anc]], 0).astype(np.float64)
        Vv = np.concatenate([vp, vt[anc]], 0).astype(np.float64)
        s = K @ q[i].astype(np.float64) * 0.5
        w = np.exp(s - s.max()); w /= w.sum()
        assert np.allclose(out[i], w @ Vv, atol=1e-12)
    # changing a non-ancestor's key/value must not move node 3's output
    kt2, vt2 = kt.copy(), vt.copy()
    kt2[[2, 4]] += 100.0; vt2[[2, 4]] -= 50.0
    out2, _ = O.tree_attention_head(q, kp, vp, kt2, vt2, mask, 5, 0.5)
    assert np.array_equal(out[3], out2[3]) and np.array_equal(out[1], out2[1])
    assert not np.allclose(out[4], out2[4])


def test_root_only_is_plain_decode_attention():
    d, P = 16, 33
    q = _rand((64, d), 1); kp = _rand((P, d), 2); vp = _rand((P, d), 3)
    kt = _rand((64, d), 4); vt = _rand((64, d), 5)
    mask = np.zeros(64, np.uint64); mask[0] = 1
    out, _ = O.tree_attention_head(q, kp, vp, kt, vt, mask, 1, 1 / np.sqrt(d))
    K = torch.from_numpy(np.concatenate([kp, kt[:1]])).double()[None]
    Vv = torch.from_numpy(np.concatenate([vp, vt[:1]])).double()[None]
    ref = F.scaled_dot_product_attention(torch.from_numpy(q[:1]).double()[None], K, Vv)
    assert np.allclose(out, ref[0].numpy(), atol=1e-12)


def test_equal_values_and_zero_query_closed_forms():
    d, P, n = 8, 7, 4
    q = _rand((64, d), 1); kp = _rand((P, d), 2); kt = _rand((64, d), 3)
    row = _rand((d,), 4)
    vp = np.tile(row, (P, 1)); vt = np.tile(row, (64, 1))
    mask = _chain_mask(n)
    out, _ = O.tree_attention_head(q, kp, vp, kt, vt, mask, n, 0.3)
    assert np.allclose(out, row[None].astype(np.float64), atol=1e-12)       # convex combination of equal rows
    vp = _rand((P, d), 5); vt = _rand((64, d), 6)
    out, lse = O.tree_attention_head(np.zeros((64, d), np.float32), kp, vp, kt, vt, mask, n, 0.3)
    for i in range(n):
        allowed = np.concatenate([vp, vt[: i + 1]]).astype(np.float64)
        assert np.allclose(out[i], allowed.mean(0), atol=1e-12)            # uniform weights
        assert abs(lse[i] - np.log(P + i + 1)) < 1e-12


def test_empty_prefix():
    d, n = 8, 3
    q = _rand((64, d), 1); kt = _rand((64, d), 3); vt = _rand((64, d), 4)
    out, _ = O.tree_attention_head(q, np.zeros((0, d), np.float32), np.zeros((0, d), np.float32), kt, vt,
                                   _chain_mask(n), n, 1.0)
    assert np.allclose(out[0], vt[0].astype(np.float64), atol=1e-12)         # the root sees only itself
