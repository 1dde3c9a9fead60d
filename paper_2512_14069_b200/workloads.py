"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *draws inputs* (numpy, counter-based Philox streams).  It holds
none of the method's arithmetic and is the one module that both the CPU oracle's
tests and the CUDA path's tests / benchmark use, so that both sides see the same
bits.  Every tensor is a function of (config id, tensor id, sequence, ...) only.

The five configurations follow the model shapes of the paper's experiments
(LLaMA-3.1-8B, Vicuna-13B, LLaMA-3.3-70B; k = 10 and t_max = 8 as in its
experimental setup) and stand in for its MT-bench / GSM8K / Alpaca / MBPP runs,
whose prompts and model weights are not available offline.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

M_MAX = 64
GATE_HIDDEN = 128

# tensor ids (second word of every stream key)
T_DRAFT, T_TARGET_NOISE, T_GATE, T_Q, T_KC, T_VC, T_KT, T_VT, T_UACC, T_USAMP, T_PLEN, T_DEPTH, \
    T_NKEEP, T_PEAK, T_TARGET_FRESH, T_ROOT, T_POLICY, T_FEATURES, T_TRAIN = range(19)


@dataclass(frozen=True)
class Config:
    cid: int
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    kv_dtype: str            # "f32" | "bf16"
    P: tuple                 # (lo, hi) inclusive prefix length range; lo == hi for fixed
    V: int
    k: int
    t_max: int
    N: int
    mode: str                # "greedy" | "stochastic"
    temperature: float
    draft_kind: str          # "normal2" | "zipf"
    zipf_a: tuple            # (lo, hi) per-sequence peakedness
    target_sigma: float
    depth_plan: str          # "gate" | "uniform_1_tmax" | "uniform_2_tmax" | "fixed_tmax"
    nkeep_range: tuple | None  # per-sequence rerank size range, None = N everywhere
    # Random-init gate weights give an almost input-independent decision; this constant, added to
    # the "continue" bias, centres the decision inside the trajectory so that depth is input-decided.
    gate_b2_offset: float = 0.0

    @property
    def R(self) -> int:      # draft logits rows one sequence can consume
        return 1 + (self.t_max - 1) * self.k

    @property
    def C(self) -> int:      # pool capacity
        return self.k + (self.t_max - 1) * self.k * self.k


CONFIGS = {
    1: Config(1, "tiny", 1, 4, 4, 64, "f32", (128, 128), 1000, 4, 4, 16, "greedy", 1.0,
              "normal2", (0.0, 0.0), 0.5, "gate", None, -0.1700),
    2: Config(2, "llama31_8b", 1, 32, 8, 128, "bf16", (2048, 2048), 128256, 10, 8, 60, "greedy", 1.0,
              "zipf", (1.0, 1.0), 1.0, "gate", None, 0.1134),
    3: Config(3, "vicuna_13b", 4, 40, 40, 128, "bf16", (4096, 4096), 32000, 8, 6, 48, "stochastic", 1.0,
              "zipf", (0.5, 2.0), 1.0, "gate", None, 0.0300),
    4: Config(4, "llama33_70b", 8, 64, 8, 128, "bf16", (8192, 8192), 128256, 10, 8, 60, "greedy", 1.0,
              "zipf", (1.0, 1.0), 1.0, "uniform_1_tmax", None, 0.0),
    5: Config(5, "stress", 32, 32, 8, 128, "bf16", (4096, 32768), 128256, 10, 8, 60, "stochastic", 0.7,
              "zipf", (1.0, 1.0), 1.0, "uniform_2_tmax", (8, 60), 0.0),
}


def shrink(cfg: Config, **kw) -> Config:
    """A config with some fields replaced (used for reduced-size parity cases)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(kw)
    return Config(**d)


def stream(cfg: Config, tensor_id: int, *idx) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([cfg.cid, tensor_id, *[int(i) for i in idx]])))


# ---- bf16 <-> float32 bit conversions (format only) ------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---- per-sequence scalars ---------------------------------------------------
def prefix_lens(cfg: Config) -> np.ndarray:
    lo, hi = cfg.P
    if lo == hi:
        return np.full(cfg.B, lo, np.int32)
    return stream(cfg, T_PLEN).integers(lo, hi + 1, size=cfg.B).astype(np.int32)


def forced_calls(cfg: Config):
    """Per-sequence number of draft calls when the harness (not the gate) fixes it, else None."""
    if cfg.depth_plan == "gate":
        return None
    if cfg.depth_plan == "fixed_tmax":             # EAGLE-3's fixed schedule: every sequence makes all t_max calls
        return np.full(cfg.B, cfg.t_max, np.int32)
    lo = 1 if cfg.depth_plan == "uniform_1_tmax" else 2
    return stream(cfg, T_DEPTH).integers(lo, cfg.t_max + 1, size=cfg.B).astype(np.int32)


def keep_sizes(cfg: Config) -> np.ndarray:
    if cfg.nkeep_range is None:
        return np.full(cfg.B, cfg.N, np.int32)
    lo, hi = cfg.nkeep_range
    return stream(cfg, T_NKEEP).integers(lo, hi + 1, size=cfg.B).astype(np.int32)


def root_tokens(cfg: Config) -> np.ndarray:
    return stream(cfg, T_ROOT).integers(0, cfg.V, size=cfg.B).astype(np.int32)


def peakedness(cfg: Config) -> np.ndarray:
    lo, hi = cfg.zipf_a
    if lo == hi:
        return np.full(cfg.B, lo, np.float64)
    return stream(cfg, T_PEAK).uniform(lo, hi, size=cfg.B)


# ---- logits -------------------------------------------------------------------
def _draft_row(cfg: Config, g: np.random.Generator, a: float) -> np.ndarray:
    if cfg.draft_kind == "normal2":
        return (2.0 * g.standard_normal(cfg.V)).astype(np.float32)
    perm = g.permutation(cfg.V)
    z = np.empty(cfg.V, np.float64)
    z[perm] = -a * np.log1p(np.arange(cfg.V, dtype=np.float64))
    z += 0.1 * g.standard_normal(cfg.V)
    return z.astype(np.float32)


def draft_logits(cfg: Config, b: int) -> np.ndarray:
    """[R,V] float32: row 0 feeds draft call 1, rows 1+(t-2)k.. feed call t (one per frontier slot)."""
    a = float(peakedness(cfg)[b])
    out = np.empty((cfg.R, cfg.V), np.float32)
    for r in range(cfg.R):
        out[r] = _draft_row(cfg, stream(cfg, T_DRAFT, b, r), a)
    return out


def target_logits(cfg: Config, b: int, draft: np.ndarray, node_draft_row: np.ndarray, n_nodes: int) -> np.ndarray:
    """[64,V] float32 target logits at the tree nodes of sequence b.

    Node i that was expanded (node_draft_row[i] >= 0) gets the draft row that
    produced its children plus N(0, sigma) noise; any other node gets a fresh
    draft-like row plus noise.  Rows >= n_nodes are zero.
    """
    a = float(peakedness(cfg)[b])
    out = np.zeros((M_MAX, cfg.V), np.float32)
    for i in range(n_nodes):
        r = int(node_draft_row[i])
        base = draft[r] if r >= 0 else _draft_row(cfg, stream(cfg, T_TARGET_FRESH, b, i), a)
        noise = stream(cfg, T_TARGET_NOISE, b, i).standard_normal(cfg.V).astype(np.float32)
        out[i] = base + np.float32(cfg.target_sigma) * noise
    return out


# ---- gate weights ------------------------------------------------------------
def gate_weights(cfg: Config) -> dict:
    """Random-init prediction model: every tensor i.i.d. U(-1/sqrt(H), 1/sqrt(H)); float32.

    Shapes follow a single-layer LSTM(input k, hidden H) with gate blocks
    (input, forget, cell, output) and an MLP Linear(H+k, H), ReLU, Linear(H, 2).
    """
    H, k = GATE_HIDDEN, cfg.k
    g = stream(cfg, T_GATE)
    s = 1.0 / np.sqrt(H)
    u = lambda *shape: g.uniform(-s, s, size=shape).astype(np.float32)
    w = {"w_ih": u(4 * H, k), "w_hh": u(4 * H, H), "b_ih": u(4 * H), "b_hh": u(4 * H),
         "w1": u(H, H + k), "b1": u(H), "w2": u(2, H), "b2": u(2)}
    w["b2"][1] += np.float32(cfg.gate_b2_offset)
    return w


def policy_weights(cfg: Config, policy: str, feat_dim: int = 0) -> dict:
    """Random-init weights of the ablation's policy networks (Table 3), same distribution as
    `gate_weights`: "mlp_scores" -> Linear(k, H), ReLU, Linear(H, 2); "lstm_hidden" -> LSTM(input
    feat_dim, hidden H) and Linear(H + feat_dim, H), ReLU, Linear(H, 2).  The "continue" bias is
    left at its draw: the variants are regression workloads, their depth is whatever comes out."""
    H, k = GATE_HIDDEN, cfg.k
    g = stream(cfg, T_POLICY, 0 if policy == "mlp_scores" else 1)
    s = 1.0 / np.sqrt(H)
    u = lambda *shape: g.uniform(-s, s, size=shape).astype(np.float32)
    if policy == "mlp_scores":
        return {"w1": u(H, k), "b1": u(H), "w2": u(2, H), "b2": u(2)}
    assert policy == "lstm_hidden" and feat_dim > 0
    return {"w_ih": u(4 * H, feat_dim), "w_hh": u(4 * H, H), "b_ih": u(4 * H), "b_hh": u(4 * H),
            "w1": u(H, H + feat_dim), "b1": u(H), "w2": u(2, H), "b2": u(2)}


def gate_features(cfg: Config, feat_dim: int) -> np.ndarray:
    """[t_max-1, B, feat_dim] float32 N(0,1): stands in for the draft model's hidden state of each call."""
    return stream(cfg, T_FEATURES).standard_normal((cfg.t_max - 1, cfg.B, feat_dim), dtype=np.float32)


# ---- attention operands -------------------------------------------------------
def _normal(cfg: Config, tid: int, shape, *idx) -> np.ndarray:
    x = stream(cfg, tid, *idx).standard_normal(shape, dtype=np.float32)
    if cfg.kv_dtype == "bf16":
        return f32_to_bf16_bits(x)
    return x


def attn_q(cfg: Config, b: int) -> np.ndarray:
    """[64,Hq,d] (float32, or bf16 bit patterns as uint16)."""
    return _normal(cfg, T_Q, (M_MAX, cfg.Hq, cfg.d), b)


def attn_tree_kv(cfg: Config, b: int):
    return _normal(cfg, T_KT, (M_MAX, cfg.Hkv, cfg.d), b), _normal(cfg, T_VT, (M_MAX, cfg.Hkv, cfg.d), b)


def attn_prefix_kv(cfg: Config, b: int, P: int):
    """Prefix cache of sequence b: K, V [P,Hkv,d]."""
    return _normal(cfg, T_KC, (P, cfg.Hkv, cfg.d), b), _normal(cfg, T_VC, (P, cfg.Hkv, cfg.d), b)


def widen(cfg: Config, x: np.ndarray) -> np.ndarray:
    """The float32 values a stored tensor represents."""
    return bf16_bits_to_f32(x) if x.dtype == np.uint16 else x


# ---- uniforms for stochastic acceptance --------------------------------------
def accept_uniforms(cfg: Config):
    """u_accept [B,64], u_sample [B], float32 in [0,1)."""
    ua = stream(cfg, T_UACC).random((cfg.B, M_MAX), dtype=np.float32)
    us = stream(cfg, T_USAMP).random(cfg.B, dtype=np.float32)
    return ua, us


# ---- synthetic training data for the prediction model (Sec. 4.3: data points {S, D}) -------------
def train_batch(cfg: Config, n: int, seed: int = 0):
    """n synthetic data points.  log_states [t_max][n][k] float32: logs of k descending confidence scores per
    draft call, shrinking with depth like cumulative path probabilities; dists [t_max][n][t_max+1] float64:
    random distributions whose mass moves to longer acceptance lengths as the number of calls grows, with
    p_j = 0 for j > i (a tree of i calls cannot accept more than i tokens); uniforms u_action [n][t_max],
    u_length [n] float32.  Holds no arithmetic of the method: the rows only have the paper's shapes."""
    g = stream(cfg, T_TRAIN, seed)
    k, t_max = cfg.k, cfg.t_max
    base = np.sort(g.uniform(0.02, 1.0, size=(t_max, n, k)), axis=2)[:, :, ::-1]
    decay = np.cumprod(g.uniform(0.5, 1.0, size=(t_max, n, 1)), axis=0)
    log_states = np.log(base * decay).astype(np.float32)
    dists = np.zeros((t_max, n, t_max + 1), np.float64)
    for i in range(1, t_max + 1):
        w = g.gamma(1.0, size=(n, i + 1))
        dists[i - 1, :, : i + 1] = w / w.sum(axis=1, keepdims=True)
    u_action = g.random((n, t_max), dtype=np.float32)
    u_length = g.random(n, dtype=np.float32)
    return log_states, dists, u_action, u_length
