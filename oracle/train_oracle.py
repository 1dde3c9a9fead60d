"""CPU oracle of one REINFORCE step of the prediction model (test infrastructure, not product code).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this module; the CUDA path
shares nothing with it.  Everything is numpy fp64, one data point at a time, in the paper's order:

  Sec. 4.2, Eq. 3-5   the state s_t = confidence scores of the k frontier tokens after draft call t, the
                      actions {0: stop, 1: continue}, the trajectory ends with the first stop;
  Sec. 4.2, Eq. 6-8   reward -alpha for every step before the last, l_acc / T_gen(T) at the last,
                      T_gen(t) = T_o + T_d t + T_pred(t), T_pred(t) = T_p (t + 1) for t < t_max, T_p t at t_max;
  Sec. 4.2, Eq. 9     discount gamma;
  Sec. 4.2, Eq. 10    loss = - sum_t G_t log pi(a_t | s_1..s_t), G_t the discounted return from step t on;
  Sec. 4.3            the data point x = {S, D}: l_acc is drawn from d_T, the acceptance-length distribution
                      for T draft calls;
  App. "Implementation Details"   LSTM(k -> 128) + MLP(128 + k -> 128 -> 2), softmax over the two logits.

Readings the text leaves open (each is a switch of one line here):
  * actions are SAMPLED during training: a_t = 1 iff u_t < pi(1 | .), u_t a uniform passed in;
  * a trajectory that reaches t_max ends there without a decision (the prediction model is not called after the
    last draft call, which is what T_pred says): its decisions are t = 1 .. t_max - 1, all "continue";
  * step indices: rewards r_1 .. r_T belong to draft calls 1 .. T; the decision taken after call t collects
    G_t = sum_{t' = t}^{T} gamma^(t' - t) r_t'.  A stop after call T therefore collects the terminal reward
    undiscounted, a "continue" after call t < T collects -alpha now and the rest discounted;
  * l_acc is drawn by inverse CDF in the order p_0, p_1, ...: the smallest j whose cumulative mass exceeds
    v * total (the last j with mass if rounding leaves none);
  * no baseline is subtracted from the return, dropout is the identity, the batch loss is the mean over data points;
  * the optimiser is not named: Adam (beta 0.9 / 0.999, eps 1e-8, no weight decay, bias-corrected) at the stated
    learning rate.
"""
from __future__ import annotations

import numpy as np

from . import radar_oracle as O

PARAM_ORDER = ("w_ih", "w_hh", "b_ih", "b_hh", "w1", "b1", "w2", "b2")


def t_gen(T: int, t_max: int, T_o: float, T_d: float, T_p: float) -> float:
    """Eq. 7-8."""
    t_pred = T_p * (T + 1) if T < t_max else T_p * T
    return T_o + T_d * T + t_pred


def sample_length(d_row, v: float):
    """Inverse CDF over p_0..p_tmax; returns (l_acc, margin of v * total from the nearest step edge)."""
    w = np.asarray(d_row, np.float64)
    total = float(w.sum())
    target = float(v) * total
    run, last_pos = 0.0, -1
    for j in range(w.shape[0]):
        prev = run
        run += float(w[j])
        if w[j] > 0.0:
            last_pos = j
        if run > target:
            return j, min(run - target, target - prev) / total
    return last_pos, 0.0


def returns(T: int, n_dec: int, reward_T: float, alpha: float, gamma: float) -> np.ndarray:
    """G_t for the decisions after calls t = 1 .. n_dec (Eq. 6, 9, 10): r_t' = -alpha for t' < T, reward_T at T."""
    G = np.zeros(n_dec, np.float64)
    for t in range(1, n_dec + 1):
        g = 0.0
        for tp in range(t, T + 1):
            g += gamma ** (tp - t) * (reward_T if tp == T else -alpha)
        G[t - 1] = g
    return G


def rollout(w, log_states, u_action, t_max: int):
    """The trajectory of one data point: decisions after calls 1 .. (until the first stop, or t_max - 1).
    log_states[t-1] = log of the k confidence scores after call t.  Returns the number of draft calls T, the
    actions, pi(a_t | .), the margins |u_t - pi(1 | .)| and everything backward needs."""
    H = np.asarray(w["w_hh"]).shape[1]
    h, c = np.zeros(H), np.zeros(H)
    steps = []
    T = t_max
    for t in range(1, t_max):
        x = np.exp(np.asarray(log_states[t - 1], np.float64))
        y, h_new, c_new = O.gate_step(x, h, c, w)
        z = y - y.max()
        pi = np.exp(z) / np.exp(z).sum()
        a = 1 if float(u_action[t - 1]) < pi[1] else 0
        steps.append({"x": x, "h_prev": h, "c_prev": c, "h": h_new, "c": c_new, "y": y, "pi": pi, "a": a,
                      "margin": abs(float(u_action[t - 1]) - pi[1])})
        h, c = h_new, c_new
        if a == 0:
            T = t
            break
    return T, steps


def _sig(v):
    return 1.0 / (1.0 + np.exp(-v))


def point_loss_and_grad(w, log_states, dists, u_action, u_length, t_max, alpha, gamma, T_o, T_d, T_p):
    """Loss of one data point and its gradient w.r.t. every parameter (backpropagation through time written
    out; the sampled actions and the sampled length are constants of the gradient, as in REINFORCE)."""
    W = {n: np.asarray(w[n], np.float64) for n in PARAM_ORDER}
    H = W["w_hh"].shape[1]
    T, steps = rollout(W, log_states, u_action, t_max)
    l_acc, len_margin = sample_length(dists[T - 1], u_length)
    reward_T = l_acc / t_gen(T, t_max, T_o, T_d, T_p)
    G = returns(T, len(steps), reward_T, alpha, gamma)
    loss = 0.0
    for s, g in zip(steps, G):
        loss -= g * np.log(s["pi"][s["a"]])
    grad = {n: np.zeros_like(W[n]) for n in PARAM_ORDER}
    dh_next, dc_next = np.zeros(H), np.zeros(H)
    for s, g in reversed(list(zip(steps, G))):
        onehot = np.zeros(2)
        onehot[s["a"]] = 1.0
        dy = -g * (onehot - s["pi"])                       # d(-g log pi_a) / dy
        # head: y = W2 relu(W1 [h; x] + b1) + b2
        cat = np.concatenate([s["h"], s["x"]])
        pre1 = W["w1"] @ cat + W["b1"]
        hid = np.maximum(pre1, 0.0)
        grad["w2"] += np.outer(dy, hid)
        grad["b2"] += dy
        dpre1 = (W["w2"].T @ dy) * (pre1 > 0.0)
        grad["w1"] += np.outer(dpre1, cat)
        grad["b1"] += dpre1
        dh = (W["w1"].T @ dpre1)[:H] + dh_next
        # cell: recompute the gates of this step
        pre = W["w_ih"] @ s["x"] + W["b_ih"] + W["w_hh"] @ s["h_prev"] + W["b_hh"]
        i, f, gg, o = _sig(pre[:H]), _sig(pre[H:2 * H]), np.tanh(pre[2 * H:3 * H]), _sig(pre[3 * H:])
        tc = np.tanh(s["c"])
        dc = dh * o * (1.0 - tc * tc) + dc_next
        dpre = np.concatenate([dc * gg * i * (1.0 - i), dc * s["c_prev"] * f * (1.0 - f),
                               dc * i * (1.0 - gg * gg), dh * tc * o * (1.0 - o)])
        grad["w_ih"] += np.outer(dpre, s["x"])
        grad["w_hh"] += np.outer(dpre, s["h_prev"])
        grad["b_ih"] += dpre
        grad["b_hh"] += dpre
        dh_next = W["w_hh"].T @ dpre
        dc_next = dc * f
    info = {"T": T, "l_acc": l_acc, "reward_T": reward_T, "G": G, "actions": [s["a"] for s in steps],
            "action_margin": min([s["margin"] for s in steps], default=np.inf), "length_margin": len_margin}
    return loss, grad, info


def batch_loss_and_grad(w, log_states, dists, u_action, u_length, t_max, alpha, gamma, T_o, T_d, T_p):
    """Mean over the batch.  log_states [t_max][n][k], dists [t_max][n][t_max+1] (row i-1 = d_i), u_action
    [n][t_max], u_length [n]."""
    n = np.asarray(u_length).shape[0]
    loss = 0.0
    grad = {m: np.zeros(np.asarray(w[m]).shape, np.float64) for m in PARAM_ORDER}
    infos = []
    for j in range(n):
        l, g, info = point_loss_and_grad(w, np.asarray(log_states)[:, j], np.asarray(dists)[:, j], np.asarray(u_action)[j],
                                         float(np.asarray(u_length)[j]), t_max, alpha, gamma, T_o, T_d, T_p)
        loss += l / n
        for m in PARAM_ORDER:
            grad[m] += g[m] / n
        infos.append(info)
    return loss, grad, infos


def adam_step(w, grad, m, v, step: int, lr: float, beta1=0.9, beta2=0.999, eps=1e-8):
    """One Adam update (bias-corrected), step counted from 1.  Returns new (w, m, v) as fp64 dicts."""
    nw, nm, nv = {}, {}, {}
    for name in PARAM_ORDER:
        g = np.asarray(grad[name], np.float64)
        nm[name] = beta1 * np.asarray(m[name], np.float64) + (1.0 - beta1) * g
        nv[name] = beta2 * np.asarray(v[name], np.float64) + (1.0 - beta2) * g * g
        mhat = nm[name] / (1.0 - beta1 ** step)
        vhat = nv[name] / (1.0 - beta2 ** step)
        nw[name] = np.asarray(w[name], np.float64) - lr * mhat / (np.sqrt(vhat) + eps)
    return nw, nm, nv
