"""Device buffers and the launch sequence of one speculative step.

`SpecStep` owns the torch tensors one step needs (pool, frontier, tree, attention output,
acceptance output, workspaces) and issues the library calls in order on the current
stream: t_max expansion calls (sequences the prediction model has stopped are skipped on
the device, so no decision ever returns to the host), rerank + tree build, tree
attention, acceptance.  The expansion calls are issued as two overlapping chains: the
bandwidth-bound vocabulary passes run ahead on a side stream while the latency-bound
select + gate blocks follow on the main stream (the pass of call t+1 skips the sequences
that had stopped before call t; one that stops at call t is read once in vain).
It contains no arithmetic of the method.
"""
from __future__ import annotations

import torch

from . import binding as rb


class SpecStep:
    def __init__(self, ctx: rb.Context, *, B, V, k, t_max, N, Hq, Hkv, d, kv_dtype, max_prefix_len,
                 mode=rb.RADAR_GREEDY, temperature=1.0, logits_dtype=torch.float32, device="cuda:0"):
        self.ctx = ctx
        self.B, self.V, self.k, self.t_max, self.N = B, V, k, t_max, N
        self.Hq, self.Hkv, self.d = Hq, Hkv, d
        self.kv_dtype, self.logits_dtype = kv_dtype, logits_dtype
        self.max_prefix_len = max_prefix_len
        self.mode, self.temperature = mode, float(temperature)
        self.C = k + (t_max - 1) * k * k
        self.R = 1 + (t_max - 1) * k
        dev = torch.device(device)
        self.dev = dev
        i32, f32, u8, i64 = torch.int32, torch.float32, torch.uint8, torch.int64
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
        H, M = rb.RADAR_GATE_HIDDEN, rb.RADAR_MAX_NODES
        # expansion state
        self.active = z((B,), u8)
        self.cont = z((B,), u8)
        self.h, self.c = z((B, H), f32), z((B, H), f32)
        self.pool_tok, self.pool_parent = z((B, self.C), i32), z((B, self.C), i32)
        self.pool_depth, self.pool_draft_row = z((B, self.C), i32), z((B, self.C), i32)
        self.pool_score, self.pool_len = z((B, self.C), f32), z((B,), i32)
        self.root_score, self.root_pool_idx = z((B, 1), f32), torch.full((B, 1), -1, dtype=i32, device=dev)
        # per-call outputs, one slot per draft call so that a whole step can be inspected afterwards
        T = t_max
        self.frontier_tok, self.frontier_score = z((T, B, k), i32), z((T, B, k), f32)
        self.frontier_pool_idx, self.frontier_src_row = z((T, B, k), i32), z((T, B, k), i32)
        self.topk_tok, self.topk_logp = z((T, B, k, k), i32), z((T, B, k, k), f32)
        self.topk_tok1, self.topk_logp1 = z((B, 1, k), i32), z((B, 1, k), f32)      # call 1 has one row
        self.gate_logits, self.cont_hist = z((T, B, 2), f32), z((T, B), u8)
        # tree
        self.tree_tok, self.tree_parent, self.tree_depth = z((B, M), i32), z((B, M), i32), z((B, M), i32)
        self.tree_pos, self.tree_pool_idx, self.tree_draft_row = z((B, M), i32), z((B, M), i32), z((B, M), i32)
        self.tree_score, self.tree_mask = z((B, M), f32), z((B, M), i64)
        self.n_nodes, self.n_leaves = z((B,), i32), z((B,), i32)
        self.retrieve = z((B, N, t_max + 1), i32)
        # attention + acceptance outputs
        self.O = z((B, M, Hq, d), kv_dtype)
        self.lse = z((B, Hq, M), f32)
        self.accept_len, self.next_token, self.best_retrieve_row = z((B,), i32), z((B,), i32), z((B,), i32)
        self.path_nodes, self.path_tokens = z((B, t_max + 1), i32), z((B, t_max + 1), i32)
        # workspaces
        wb = max(rb.radar_expand_workspace_bytes(ctx, B, 1, V, k), rb.radar_expand_workspace_bytes(ctx, B, k, V, k))
        self.ws_expand = z((wb + 255,), u8)
        self.ws_expand2 = z((wb + 255,), u8)          # consecutive calls alternate, so a pass can run ahead of the select
        self.ws_attn = z((rb.radar_attn_workspace_bytes(ctx, B, Hq, Hkv, d, rb.dtype_code(self.O), max_prefix_len) + 255,), u8)
        self.ws_accept = z((rb.radar_accept_workspace_bytes(ctx, B, V, mode) + 255,), u8)
        self.side = torch.cuda.Stream(dev)            # the vocabulary passes of the pipelined expansion
        for n in ("ws_expand", "ws_expand2", "ws_attn", "ws_accept"):
            t = getattr(self, n)
            off = (-t.data_ptr()) % 256
            setattr(self, n, t[off:off + t.numel() - 255])

    # ---- expansion -------------------------------------------------------------------
    def expand(self, t, draft_logits, gate, force_calls=None, policy=rb.RADAR_POLICY_LSTM_SCORES, features=None,
               phase=rb.RADAR_EXPAND_ALL, vocab_mask=None, workspace=None, stream=None):
        """Draft call t (1-based) on draft_logits [B,R,V]: row 0 for t = 1, rows 1+(t-2)k.. for t >= 2.
        `features` [t_max-1, B, feat_dim] feeds the hidden-state policy (row t-1 at call t).  `phase`, `vocab_mask`
        (the mask a RADAR_EXPAND_VOCAB call reads rows by), `workspace` and `stream` serve the pipelined form."""
        k, B, V = self.k, self.B, self.V
        F = 1 if t == 1 else k
        row0 = 0 if t == 1 else 1 + (t - 2) * k
        s = t - 1
        rb.radar_expand_step(
            self.ctx, B=B, F=F, V=V, k=k, t=t, t_max=self.t_max, logits=draft_logits,
            logits_row_stride=V, logits_seq_stride=self.R * V, logits_offset_elems=row0 * V,
            parent_score=self.root_score if t == 1 else self.frontier_score[s - 1],
            parent_pool_idx=self.root_pool_idx if t == 1 else self.frontier_pool_idx[s - 1],
            active=vocab_mask if phase == rb.RADAR_EXPAND_VOCAB else self.active, force_calls=force_calls, gate=gate, h=self.h, c=self.c,
            pool_capacity=self.C, pool_tok=self.pool_tok, pool_parent=self.pool_parent, pool_depth=self.pool_depth,
            pool_draft_row=self.pool_draft_row, pool_score=self.pool_score, pool_len=self.pool_len,
            frontier_tok=self.frontier_tok[s], frontier_score=self.frontier_score[s],
            frontier_pool_idx=self.frontier_pool_idx[s], frontier_src_row=self.frontier_src_row[s],
            topk_tok=self.topk_tok1 if t == 1 else self.topk_tok[s],
            topk_logp=self.topk_logp1 if t == 1 else self.topk_logp[s],
            gate_logits=self.gate_logits[s], cont=self.cont_hist[s], workspace=self.ws_expand if workspace is None else workspace,
            policy=policy, features=None if features is None or t >= self.t_max else features[s], phase=phase, stream=stream)

    def run_expansion(self, draft_logits, gate, force_calls=None, policy=rb.RADAR_POLICY_LSTM_SCORES, features=None,
                      pipelined=True):
        if not pipelined:
            for t in range(1, self.t_max + 1):      # call 1 restarts the state on the device
                self.expand(t, draft_logits, gate, force_calls, policy, features)
            return
        # Two chains.  The vocabulary pass of call t (side stream, workspace t % 2) needs the select + gate block
        # of call t - 2 done: that block wrote the mask the pass skips rows by (cont of call t - 2; nothing for
        # t <= 2) and was the last reader of the same workspace.  The select + gate block of call t (main stream)
        # needs its pass and the block of call t - 1, which precedes it on the stream.
        main, side = torch.cuda.current_stream(), self.side
        ws = (self.ws_expand, self.ws_expand2)
        args = (draft_logits, gate, force_calls, policy, features)
        side.wait_stream(main)                      # fork: whatever produced the inputs is done
        sel_done = {}
        for t in range(1, self.t_max + 1):
            if t - 2 in sel_done:
                side.wait_event(sel_done[t - 2])
            mask = self.cont_hist[t - 3] if t >= 3 else None
            self.expand(t, *args, phase=rb.RADAR_EXPAND_VOCAB, vocab_mask=mask, workspace=ws[t % 2], stream=side)
            voc = torch.cuda.Event()
            voc.record(side)
            main.wait_event(voc)
            self.expand(t, *args, phase=rb.RADAR_EXPAND_SELECT, workspace=ws[t % 2], stream=main)
            sel_done[t] = torch.cuda.Event()
            sel_done[t].record(main)
        main.wait_stream(side)                      # join (the last pass has been waited for already)

    # ---- tree, attention, acceptance ------------------------------------------------------
    def build_tree(self, root_tok, prefix_len, n_keep=None):
        rb.radar_rerank_build_tree(
            self.ctx, B=self.B, N=self.N, t_max=self.t_max, pool_capacity=self.C, pool_tok=self.pool_tok,
            pool_parent=self.pool_parent, pool_depth=self.pool_depth, pool_draft_row=self.pool_draft_row,
            pool_score=self.pool_score, pool_len=self.pool_len, n_keep=n_keep, root_tok=root_tok,
            prefix_len=prefix_len, tree_tok=self.tree_tok, tree_parent=self.tree_parent, tree_depth=self.tree_depth,
            tree_pos=self.tree_pos, tree_pool_idx=self.tree_pool_idx, tree_draft_row=self.tree_draft_row,
            tree_score=self.tree_score, tree_mask=self.tree_mask, n_nodes=self.n_nodes, retrieve=self.retrieve,
            n_leaves=self.n_leaves)

    def attention(self, Q, Kc, Vc, kv_start, prefix_len, Kt, Vt, mask=None, n_nodes=None, block_table=None, page_size=0):
        rb.radar_tree_attention(
            self.ctx, B=self.B, Hq=self.Hq, Hkv=self.Hkv, d=self.d, Q=Q, Kc=Kc, Vc=Vc, kv_start=kv_start,
            prefix_len=prefix_len, max_prefix_len=self.max_prefix_len, Kt=Kt, Vt=Vt,
            mask=self.tree_mask if mask is None else mask, n_nodes=self.n_nodes if n_nodes is None else n_nodes,
            O=self.O, lse=self.lse, workspace=self.ws_attn, block_table=block_table, page_size=page_size)

    def accept(self, target_logits, draft_logits=None, u_accept=None, u_sample=None):
        rb.radar_verify_accept(
            self.ctx, B=self.B, V=self.V, t_max=self.t_max, N=self.N, mode=self.mode, temperature=self.temperature,
            target_logits=target_logits, tree_tok=self.tree_tok, tree_parent=self.tree_parent,
            tree_draft_row=self.tree_draft_row, n_nodes=self.n_nodes, retrieve=self.retrieve, n_leaves=self.n_leaves,
            draft_logits=draft_logits, R=self.R, u_accept=u_accept, u_sample=u_sample, accept_len=self.accept_len,
            path_nodes=self.path_nodes, path_tokens=self.path_tokens, next_token=self.next_token,
            best_retrieve_row=self.best_retrieve_row, workspace=self.ws_accept)
