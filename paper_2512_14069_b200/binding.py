"""Thin ctypes binding of libradar_b200.so: same names as include/radar.h, argument
marshalling only.  torch tensors are used for device memory and streams; every step of
the path runs in the library's CUDA kernels.  There is no CPU fallback: if the library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libradar_b200.so")

RADAR_MAX_NODES = 64
RADAR_GATE_HIDDEN = 128
RADAR_F32, RADAR_BF16 = 0, 1
RADAR_GREEDY, RADAR_STOCHASTIC = 0, 1
RADAR_POLICY_LSTM_SCORES, RADAR_POLICY_MLP_SCORES, RADAR_POLICY_LSTM_HIDDEN = 0, 1, 2
RADAR_OK = 0
RADAR_EXPAND_ALL, RADAR_EXPAND_VOCAB, RADAR_EXPAND_SELECT = 0, 1, 2
RADAR_ATTN_PATH_FMA, RADAR_ATTN_PATH_TENSOR_CORE = 0, 1

_c_int, _c_i64, _c_f, _vp, _sz = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t


class ExpandArgs(ctypes.Structure):
    _fields_ = [
        ("B", _c_int), ("F", _c_int), ("V", _c_int), ("k", _c_int), ("t", _c_int), ("t_max", _c_int),
        ("logits", _vp), ("logits_dtype", _c_int), ("logits_row_stride", _c_i64), ("logits_seq_stride", _c_i64),
        ("parent_score", _vp), ("parent_pool_idx", _vp), ("active", _vp), ("force_calls", _vp),
        ("w_ih", _vp), ("w_hh", _vp), ("b_ih", _vp), ("b_hh", _vp),
        ("w1", _vp), ("b1", _vp), ("w2", _vp), ("b2", _vp),
        ("h", _vp), ("c", _vp),
        ("pool_capacity", _c_int),
        ("pool_tok", _vp), ("pool_parent", _vp), ("pool_depth", _vp), ("pool_draft_row", _vp),
        ("pool_score", _vp), ("pool_len", _vp),
        ("frontier_tok", _vp), ("frontier_score", _vp), ("frontier_pool_idx", _vp), ("frontier_src_row", _vp),
        ("topk_tok", _vp), ("topk_logp", _vp), ("gate_logits", _vp), ("cont", _vp),
        ("workspace", _vp), ("workspace_bytes", _sz),
        ("policy", _c_int), ("feat_dim", _c_int), ("features", _vp), ("phase", _c_int),
    ]


class TreeArgs(ctypes.Structure):
    _fields_ = [
        ("B", _c_int), ("N", _c_int), ("t_max", _c_int), ("pool_capacity", _c_int),
        ("pool_tok", _vp), ("pool_parent", _vp), ("pool_depth", _vp), ("pool_draft_row", _vp),
        ("pool_score", _vp), ("pool_len", _vp), ("n_keep", _vp), ("root_tok", _vp), ("prefix_len", _vp),
        ("tree_tok", _vp), ("tree_parent", _vp), ("tree_depth", _vp), ("tree_pos", _vp), ("tree_pool_idx", _vp),
        ("tree_draft_row", _vp), ("tree_score", _vp), ("tree_mask", _vp), ("n_nodes", _vp), ("retrieve", _vp),
        ("n_leaves", _vp),
    ]


class AttnArgs(ctypes.Structure):
    _fields_ = [
        ("B", _c_int), ("Hq", _c_int), ("Hkv", _c_int), ("d", _c_int), ("dtype", _c_int),
        ("Q", _vp), ("Kc", _vp), ("Vc", _vp), ("kv_start", _vp), ("prefix_len", _vp), ("max_prefix_len", _c_int),
        ("cache_rows", _c_i64), ("Kt", _vp), ("Vt", _vp), ("mask", _vp), ("n_nodes", _vp), ("scale", _c_f), ("O", _vp), ("lse", _vp),
        ("workspace", _vp), ("workspace_bytes", _sz),
        ("block_table", _vp), ("page_size", _c_int), ("max_pages", _c_int),
        ("n_layers", _c_int), ("q_layer_stride", _c_i64), ("cache_layer_stride", _c_i64),
        ("tree_kv_layer_stride", _c_i64), ("o_layer_stride", _c_i64), ("lse_layer_stride", _c_i64),
    ]


class AcceptArgs(ctypes.Structure):
    _fields_ = [
        ("B", _c_int), ("V", _c_int), ("t_max", _c_int), ("N", _c_int), ("mode", _c_int), ("temperature", _c_f),
        ("target_logits", _vp), ("logits_dtype", _c_int),
        ("tree_tok", _vp), ("tree_parent", _vp), ("tree_draft_row", _vp), ("n_nodes", _vp), ("retrieve", _vp),
        ("n_leaves", _vp), ("draft_logits", _vp), ("R", _c_int), ("u_accept", _vp), ("u_sample", _vp),
        ("accept_len", _vp), ("path_nodes", _vp), ("path_tokens", _vp), ("next_token", _vp),
        ("best_retrieve_row", _vp), ("workspace", _vp), ("workspace_bytes", _sz),
    ]


class AccLenArgs(ctypes.Structure):
    _fields_ = [
        ("B", _c_int), ("V", _c_int), ("t_max", _c_int), ("temperature", _c_f),
        ("target_logits", _vp), ("logits_dtype", _c_int),
        ("tree_tok", _vp), ("tree_parent", _vp), ("tree_depth", _vp), ("tree_draft_row", _vp), ("n_nodes", _vp),
        ("draft_logits", _vp), ("R", _c_int), ("dist", _vp), ("p_acc_node", _vp),
        ("workspace", _vp), ("workspace_bytes", _sz),
    ]


class TrainArgs(ctypes.Structure):
    _fields_ = [
        ("n", _c_int), ("k", _c_int), ("t_max", _c_int),
        ("log_states", _vp), ("dists", _vp), ("u_action", _vp), ("u_length", _vp),
        ("alpha", _c_f), ("gamma", _c_f), ("T_o", _c_f), ("T_d", _c_f), ("T_p", _c_f),
        ("lr", _c_f), ("beta1", _c_f), ("beta2", _c_f), ("eps", _c_f), ("step", _c_int),
        ("theta", _vp), ("adam_m", _vp), ("adam_v", _vp), ("grad", _vp), ("loss", _vp),
        ("calls", _vp), ("l_acc", _vp), ("actions", _vp),
        ("workspace", _vp), ("workspace_bytes", _sz),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libradar_b200.so is missing: build it with `python -m paper_2512_14069_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.radar_create.restype = _c_int
        L.radar_create.argtypes = [ctypes.POINTER(_vp), _c_int]
        L.radar_destroy.restype = _c_int
        L.radar_destroy.argtypes = [_vp]
        L.radar_status_string.restype = ctypes.c_char_p
        L.radar_status_string.argtypes = [_c_int]
        L.radar_read_device_status.restype = _c_int
        L.radar_read_device_status.argtypes = [_vp, _vp]
        L.radar_expand_workspace_bytes.restype = _sz
        L.radar_expand_workspace_bytes.argtypes = [_vp, _c_int, _c_int, _c_int, _c_int]
        L.radar_expand_step.restype = _c_int
        L.radar_expand_step.argtypes = [_vp, ctypes.POINTER(ExpandArgs), _vp]
        L.radar_rerank_build_tree.restype = _c_int
        L.radar_rerank_build_tree.argtypes = [_vp, ctypes.POINTER(TreeArgs), _vp]
        L.radar_attn_workspace_bytes.restype = _sz
        L.radar_attn_workspace_bytes.argtypes = [_vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int]
        L.radar_tree_attention.restype = _c_int
        L.radar_tree_attention.argtypes = [_vp, ctypes.POINTER(AttnArgs), _vp]
        L.radar_accept_workspace_bytes.restype = _sz
        L.radar_accept_workspace_bytes.argtypes = [_vp, _c_int, _c_int, _c_int]
        L.radar_verify_accept.restype = _c_int
        L.radar_verify_accept.argtypes = [_vp, ctypes.POINTER(AcceptArgs), _vp]
        L.radar_acclen_workspace_bytes.restype = _sz
        L.radar_acclen_workspace_bytes.argtypes = [_vp, _c_int, _c_int]
        L.radar_accept_length_distribution.restype = _c_int
        L.radar_accept_length_distribution.argtypes = [_vp, ctypes.POINTER(AccLenArgs), _vp]
        L.radar_profile_begin.restype = _c_int
        L.radar_profile_begin.argtypes = [_vp, _c_int]
        L.radar_profile_end.restype = _c_int
        L.radar_profile_end.argtypes = [_vp]
        L.radar_kernel_count.restype = _c_int
        L.radar_kernel_name.restype = ctypes.c_char_p
        L.radar_kernel_name.argtypes = [_c_int]
        L.radar_kernel_stats.restype = _c_int
        L.radar_kernel_stats.argtypes = [_vp, _c_int, ctypes.POINTER(ctypes.c_longlong),
                                         ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong)]
        L.radar_reset_launch_counts.restype = _c_int
        L.radar_reset_launch_counts.argtypes = [_vp]
        _lib = L
    return _lib


class RadarError(RuntimeError):
    def __init__(self, where: str, status: int):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, lib().radar_status_string(status).decode(), status))


def _check(where: str, status: int):
    if status != RADAR_OK:
        raise RadarError(where, status)


def _ptr(t, dtype=None):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return RADAR_F32
    if t.dtype == torch.bfloat16:
        return RADAR_BF16
    raise ValueError("unsupported dtype %s" % t.dtype)


class Context:
    """radar_create / radar_destroy."""

    def __init__(self, device: int = 0):
        h = _vp()
        _check("radar_create", lib().radar_create(ctypes.byref(h), device))
        self.handle = h
        self.device = device

    def close(self):
        if self.handle:
            lib().radar_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def read_device_status(self, stream=None) -> int:
        return lib().radar_read_device_status(self.handle, _stream(stream))

    def check_device_status(self, stream=None):
        _check("device status", self.read_device_status(stream))

    # ---- measurement helpers ----
    def profile_begin(self, max_records: int):
        _check("radar_profile_begin", lib().radar_profile_begin(self.handle, max_records))

    def profile_end(self):
        _check("radar_profile_end", lib().radar_profile_end(self.handle))

    def reset_launch_counts(self):
        _check("radar_reset_launch_counts", lib().radar_reset_launch_counts(self.handle))

    def kernel_stats(self) -> dict:
        """{kernel name: (launches since reset, event-timed ms, event-timed launches)}"""
        out = {}
        for i in range(lib().radar_kernel_count()):
            n, ms, tn = ctypes.c_longlong(), ctypes.c_double(), ctypes.c_longlong()
            _check("radar_kernel_stats", lib().radar_kernel_stats(self.handle, i, ctypes.byref(n), ctypes.byref(ms),
                                                                  ctypes.byref(tn)))
            out[lib().radar_kernel_name(i).decode()] = (n.value, ms.value, tn.value)
        return out


def radar_expand_workspace_bytes(ctx: Context, B, F, V, k) -> int:
    return int(lib().radar_expand_workspace_bytes(ctx.handle, B, F, V, k))


def radar_attn_workspace_bytes(ctx: Context, B, Hq, Hkv, d, dtype, max_prefix_len) -> int:
    return int(lib().radar_attn_workspace_bytes(ctx.handle, B, Hq, Hkv, d, dtype, max_prefix_len))


def radar_accept_workspace_bytes(ctx: Context, B, V, mode) -> int:
    return int(lib().radar_accept_workspace_bytes(ctx.handle, B, V, mode))


def radar_expand_step(ctx: Context, *, B, F, V, k, t, t_max, logits, logits_row_stride, logits_seq_stride,
                      logits_offset_elems=0, parent_score, parent_pool_idx, active, force_calls=None, gate,
                      h, c, pool_capacity, pool_tok, pool_parent, pool_depth, pool_draft_row, pool_score, pool_len,
                      frontier_tok, frontier_score, frontier_pool_idx, frontier_src_row, topk_tok, topk_logp,
                      gate_logits, cont, workspace, stream=None, policy=RADAR_POLICY_LSTM_SCORES, features=None,
                      phase=RADAR_EXPAND_ALL):
    """One draft call's expansion.  `logits` is a CUDA tensor; the rows of this call start
    `logits_offset_elems` elements into it.  `gate` is a dict of the weight tensors (all eight for the
    LSTM policies; w1, b1, w2, b2 for RADAR_POLICY_MLP_SCORES); `features` [B, feat_dim] float32 is the
    input of RADAR_POLICY_LSTM_HIDDEN."""
    f32, i32, u8 = torch.float32, torch.int32, torch.uint8
    a = ExpandArgs()
    a.B, a.F, a.V, a.k, a.t, a.t_max = B, F, V, k, t, t_max
    a.logits = _ptr(logits) + logits_offset_elems * logits.element_size()
    a.logits_dtype = dtype_code(logits)
    a.logits_row_stride, a.logits_seq_stride = logits_row_stride, logits_seq_stride
    a.parent_score, a.parent_pool_idx = _ptr(parent_score, f32), _ptr(parent_pool_idx, i32)
    a.active, a.force_calls = _ptr(active, u8), _ptr(force_calls, i32)
    for n in ("w_ih", "w_hh", "b_ih", "b_hh", "w1", "b1", "w2", "b2"):
        setattr(a, n, _ptr(gate.get(n), f32))
    a.policy, a.phase = policy, phase
    if features is not None:
        a.features, a.feat_dim = _ptr(features, f32), features.shape[-1]
    a.h, a.c = _ptr(h, f32), _ptr(c, f32)
    a.pool_capacity = pool_capacity
    a.pool_tok, a.pool_parent, a.pool_depth = _ptr(pool_tok, i32), _ptr(pool_parent, i32), _ptr(pool_depth, i32)
    a.pool_draft_row, a.pool_score, a.pool_len = _ptr(pool_draft_row, i32), _ptr(pool_score, f32), _ptr(pool_len, i32)
    a.frontier_tok, a.frontier_score = _ptr(frontier_tok, i32), _ptr(frontier_score, f32)
    a.frontier_pool_idx, a.frontier_src_row = _ptr(frontier_pool_idx, i32), _ptr(frontier_src_row, i32)
    a.topk_tok, a.topk_logp = _ptr(topk_tok, i32), _ptr(topk_logp, f32)
    a.gate_logits, a.cont = _ptr(gate_logits, f32), _ptr(cont, u8)
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    _check("radar_expand_step", lib().radar_expand_step(ctx.handle, ctypes.byref(a), _stream(stream)))


def radar_rerank_build_tree(ctx: Context, *, B, N, t_max, pool_capacity, pool_tok, pool_parent, pool_depth,
                            pool_draft_row, pool_score, pool_len, n_keep=None, root_tok, prefix_len, tree_tok,
                            tree_parent, tree_depth, tree_pos, tree_pool_idx, tree_draft_row, tree_score, tree_mask,
                            n_nodes, retrieve, n_leaves, stream=None):
    f32, i32 = torch.float32, torch.int32
    a = TreeArgs()
    a.B, a.N, a.t_max, a.pool_capacity = B, N, t_max, pool_capacity
    a.pool_tok, a.pool_parent, a.pool_depth = _ptr(pool_tok, i32), _ptr(pool_parent, i32), _ptr(pool_depth, i32)
    a.pool_draft_row, a.pool_score, a.pool_len = _ptr(pool_draft_row, i32), _ptr(pool_score, f32), _ptr(pool_len, i32)
    a.n_keep, a.root_tok, a.prefix_len = _ptr(n_keep, i32), _ptr(root_tok, i32), _ptr(prefix_len, i32)
    a.tree_tok, a.tree_parent, a.tree_depth = _ptr(tree_tok, i32), _ptr(tree_parent, i32), _ptr(tree_depth, i32)
    a.tree_pos, a.tree_pool_idx, a.tree_draft_row = _ptr(tree_pos, i32), _ptr(tree_pool_idx, i32), _ptr(tree_draft_row, i32)
    a.tree_score, a.tree_mask = _ptr(tree_score, f32), _ptr(tree_mask, torch.int64)
    a.n_nodes, a.retrieve, a.n_leaves = _ptr(n_nodes, i32), _ptr(retrieve, i32), _ptr(n_leaves, i32)
    _check("radar_rerank_build_tree", lib().radar_rerank_build_tree(ctx.handle, ctypes.byref(a), _stream(stream)))


def _attn_args(*, B, Hq, Hkv, d, Q, Kc, Vc, kv_start, prefix_len, max_prefix_len, Kt, Vt, mask, n_nodes, O, workspace,
               lse=None, scale=0.0, block_table=None, page_size=0, n_layers=1):
    """With n_layers > 1 every tensor carries a leading layer dimension: Q, O [L, B, 64, Hq, d]; Kt, Vt [L, B, 64, Hkv, d];
    Kc, Vc [L, cache_rows, Hkv, d]; lse [L, B, Hq, 64]."""
    a = AttnArgs()
    if n_layers > 1:
        a.n_layers = n_layers
        a.q_layer_stride, a.o_layer_stride = Q[0].numel(), O[0].numel()
        a.tree_kv_layer_stride = Kt[0].numel()
        a.cache_layer_stride = 0 if Kc is None else Kc[0].numel()
        a.lse_layer_stride = 0 if lse is None else lse[0].numel()
    a.B, a.Hq, a.Hkv, a.d, a.dtype = B, Hq, Hkv, d, dtype_code(Q)
    for t in (Kc, Vc, Kt, Vt, O):
        if t is not None and t.dtype != Q.dtype:
            raise ValueError("Q, K, V and O must share one dtype")
    a.Q, a.Kc, a.Vc = _ptr(Q), _ptr(Kc), _ptr(Vc)
    a.kv_start, a.prefix_len = _ptr(kv_start, torch.int64), _ptr(prefix_len, torch.int32)
    a.max_prefix_len = max_prefix_len
    a.cache_rows = 0 if Kc is None else min(Kc.numel(), Vc.numel()) // (Hkv * d * max(n_layers, 1))   # token rows [Hkv][d] per layer
    a.Kt, a.Vt, a.mask, a.n_nodes = _ptr(Kt), _ptr(Vt), _ptr(mask, torch.int64), _ptr(n_nodes, torch.int32)
    a.scale, a.O, a.lse = scale, _ptr(O), _ptr(lse, torch.float32)
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    if block_table is not None:
        a.block_table, a.page_size, a.max_pages = _ptr(block_table, torch.int32), page_size, block_table.shape[-1]
    return a


def radar_tree_attention(ctx: Context, *, stream=None, **kw):
    """Arguments as in `_attn_args` (the fields of radar_attn_args as tensors).  `block_table` [B, max_pages] int32
    with `page_size` selects the paged prefix cache (kv_start may then be None)."""
    a = _attn_args(**kw)
    _check("radar_tree_attention", lib().radar_tree_attention(ctx.handle, ctypes.byref(a), _stream(stream)))


def radar_tree_attention_path(**kw) -> int:
    """RADAR_ATTN_PATH_TENSOR_CORE or RADAR_ATTN_PATH_FMA for the same keyword arguments as radar_tree_attention."""
    L = lib()
    L.radar_tree_attention_path.restype = _c_int
    L.radar_tree_attention_path.argtypes = [ctypes.POINTER(AttnArgs)]
    a = _attn_args(**kw)
    return int(L.radar_tree_attention_path(ctypes.byref(a)))


def radar_verify_accept(ctx: Context, *, B, V, t_max, N, mode, target_logits, tree_tok, tree_parent, tree_draft_row,
                        n_nodes, retrieve, n_leaves, accept_len, path_nodes, path_tokens, next_token,
                        best_retrieve_row, workspace, temperature=1.0, draft_logits=None, R=0, u_accept=None,
                        u_sample=None, stream=None):
    i32, f32 = torch.int32, torch.float32
    a = AcceptArgs()
    a.B, a.V, a.t_max, a.N, a.mode, a.temperature = B, V, t_max, N, mode, temperature
    a.target_logits, a.logits_dtype = _ptr(target_logits), dtype_code(target_logits)
    if draft_logits is not None and draft_logits.dtype != target_logits.dtype:
        raise ValueError("target and draft logits must share one dtype")
    a.tree_tok, a.tree_parent, a.tree_draft_row = _ptr(tree_tok, i32), _ptr(tree_parent, i32), _ptr(tree_draft_row, i32)
    a.n_nodes, a.retrieve, a.n_leaves = _ptr(n_nodes, i32), _ptr(retrieve, i32), _ptr(n_leaves, i32)
    a.draft_logits, a.R = _ptr(draft_logits), R
    a.u_accept, a.u_sample = _ptr(u_accept, f32), _ptr(u_sample, f32)
    a.accept_len, a.path_nodes, a.path_tokens = _ptr(accept_len, i32), _ptr(path_nodes, i32), _ptr(path_tokens, i32)
    a.next_token, a.best_retrieve_row = _ptr(next_token, i32), _ptr(best_retrieve_row, i32)
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    _check("radar_verify_accept", lib().radar_verify_accept(ctx.handle, ctypes.byref(a), _stream(stream)))


def radar_acclen_workspace_bytes(ctx: Context, B, V) -> int:
    return int(lib().radar_acclen_workspace_bytes(ctx.handle, B, V))


def radar_accept_length_distribution(ctx: Context, *, B, V, t_max, temperature, target_logits, tree_tok, tree_parent,
                                     tree_depth, tree_draft_row, n_nodes, draft_logits, R, dist, p_acc_node, workspace,
                                     stream=None):
    i32, f64 = torch.int32, torch.float64
    a = AccLenArgs()
    a.B, a.V, a.t_max, a.temperature = B, V, t_max, temperature
    if draft_logits.dtype != target_logits.dtype:
        raise ValueError("target and draft logits must share one dtype")
    a.target_logits, a.logits_dtype = _ptr(target_logits), dtype_code(target_logits)
    a.tree_tok, a.tree_parent = _ptr(tree_tok, i32), _ptr(tree_parent, i32)
    a.tree_depth, a.tree_draft_row, a.n_nodes = _ptr(tree_depth, i32), _ptr(tree_draft_row, i32), _ptr(n_nodes, i32)
    a.draft_logits, a.R = _ptr(draft_logits), R
    a.dist, a.p_acc_node = _ptr(dist, f64), _ptr(p_acc_node, f64)
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    _check("radar_accept_length_distribution",
           lib().radar_accept_length_distribution(ctx.handle, ctypes.byref(a), _stream(stream)))


def radar_policy_param_count(k: int) -> int:
    L = lib()
    L.radar_policy_param_count.restype = _sz
    L.radar_policy_param_count.argtypes = [_c_int]
    return int(L.radar_policy_param_count(k))


def radar_train_workspace_bytes(ctx: Context, n: int, k: int, t_max: int) -> int:
    L = lib()
    L.radar_train_workspace_bytes.restype = _sz
    L.radar_train_workspace_bytes.argtypes = [_vp, _c_int, _c_int, _c_int]
    return int(L.radar_train_workspace_bytes(ctx.handle, n, k, t_max))


def radar_policy_train_step(ctx: Context, *, n, k, t_max, log_states, dists, u_action, u_length, alpha, gamma, T_o, T_d,
                            T_p, theta, grad, loss, calls, l_acc, actions, workspace, step=0, lr=1e-4, beta1=0.9,
                            beta2=0.999, eps=1e-8, adam_m=None, adam_v=None, stream=None):
    """One REINFORCE step of the prediction model on n data points {S, D}; see include/radar.h for layouts."""
    f32, f64, i32, u8 = torch.float32, torch.float64, torch.int32, torch.uint8
    L = lib()
    L.radar_policy_train_step.restype = _c_int
    L.radar_policy_train_step.argtypes = [_vp, ctypes.POINTER(TrainArgs), _vp]
    a = TrainArgs()
    a.n, a.k, a.t_max = n, k, t_max
    a.log_states, a.dists = _ptr(log_states, f32), _ptr(dists, f64)
    a.u_action, a.u_length = _ptr(u_action, f32), _ptr(u_length, f32)
    a.alpha, a.gamma, a.T_o, a.T_d, a.T_p = alpha, gamma, T_o, T_d, T_p
    a.lr, a.beta1, a.beta2, a.eps, a.step = lr, beta1, beta2, eps, step
    a.theta, a.grad, a.loss = _ptr(theta, f32), _ptr(grad, f32), _ptr(loss, f32)
    a.adam_m = _ptr(adam_m, f32) if adam_m is not None else None
    a.adam_v = _ptr(adam_v, f32) if adam_v is not None else None
    a.calls, a.l_acc, a.actions = _ptr(calls, i32), _ptr(l_acc, i32), _ptr(actions, u8)
    a.workspace, a.workspace_bytes = _ptr(workspace), workspace.numel() * workspace.element_size()
    _check("radar_policy_train_step", L.radar_policy_train_step(ctx.handle, ctypes.byref(a), _stream(stream)))


def radar_noalloc_scratch_bytes() -> int:
    L = lib()
    L.radar_noalloc_scratch_bytes.restype = _sz
    return int(L.radar_noalloc_scratch_bytes())


def radar_verify_accept_greedy_noalloc(ctx: Context, *, B, V, t_max, N, target_logits, tree_tok, tree_parent,
                                       n_nodes, retrieve, n_leaves, accept_len, path_nodes, path_tokens, next_token,
                                       best_retrieve_row, stream=None):
    """Greedy acceptance without a caller workspace: for hosts that may not allocate device memory at
    this point (all of it already belongs to their own pool, or cudaMalloc's device-wide sync is not
    acceptable).  Scratch is a fixed 1 MiB array inside the library, shared by every call on the
    device - do not overlap calls - and sizes that do not fit raise RadarError(-2).  The first call
    on a device resolves the array's address; make it outside stream capture."""
    i32 = torch.int32
    L = lib()
    L.radar_verify_accept_greedy_noalloc.restype = _c_int
    L.radar_verify_accept_greedy_noalloc.argtypes = [_vp, ctypes.POINTER(AcceptArgs), _vp]
    a = AcceptArgs()
    a.B, a.V, a.t_max, a.N, a.mode, a.temperature = B, V, t_max, N, RADAR_GREEDY, 1.0
    a.target_logits = _ptr(target_logits) if target_logits is not None else None
    a.logits_dtype = dtype_code(target_logits) if target_logits is not None else RADAR_F32
    a.tree_tok, a.tree_parent = _ptr(tree_tok, i32), _ptr(tree_parent, i32)
    a.n_nodes, a.retrieve, a.n_leaves = _ptr(n_nodes, i32), _ptr(retrieve, i32), _ptr(n_leaves, i32)
    a.accept_len, a.path_nodes, a.path_tokens = _ptr(accept_len, i32), _ptr(path_nodes, i32), _ptr(path_tokens, i32)
    a.next_token, a.best_retrieve_row = _ptr(next_token, i32), _ptr(best_retrieve_row, i32)
    _check("radar_verify_accept_greedy_noalloc",
           L.radar_verify_accept_greedy_noalloc(ctx.handle, ctypes.byref(a), _stream(stream)))
