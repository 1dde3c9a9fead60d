"""Pins of the training oracle (oracle/train_oracle.py): what the paper and the mathematics fix.

  * T_gen against the latency terms the paper prints (Table 5) and Eq. 7-8 worked by hand;
  * the returns of Eq. 6 / 9 / 10 on two trajectories worked by hand (a stop before t_max, a run to t_max);
  * the inverse-CDF draw of l_acc on small distributions, including the edges;
  * the gradient against torch autograd on torch.nn.LSTM + Linear (an independent implementation of the
    network and of backpropagation) and against central finite differences of the surrogate loss;
  * the policy-gradient identity: for gamma = 1 the expectation of the estimator over every action sequence
    and every acceptance length equals minus the gradient of the exact expected return (by finite
    differences), which fails for a wrong sign, a reward booked to the wrong step or actions that leak into
    the gradient;
  * Adam against torch.optim.Adam.
"""
import itertools

import numpy as np
import pytest

from oracle import radar_oracle as O
from oracle import train_oracle as T


def _weights(rng, k, H):
    s = 1.0 / np.sqrt(H)
    u = lambda *shape: rng.uniform(-s, s, size=shape)
    return {"w_ih": u(4 * H, k), "w_hh": u(4 * H, H), "b_ih": u(4 * H), "b_hh": u(4 * H),
            "w1": u(H, H + k), "b1": u(H), "w2": u(2, H), "b2": u(2)}


def _point(rng, k, t_max):
    logs = np.log(np.sort(rng.uniform(0.01, 1.0, size=(t_max, k)), axis=1)[:, ::-1])
    d = rng.dirichlet(np.ones(t_max + 1), size=t_max)
    return logs, d


def test_t_gen_matches_table_5_terms():
    # LLaMA-3.1-8B row of the latency table: T_o = 68, T_d = 2.7, T_p = 0.4 (ms), t_max = 8
    assert T.t_gen(5, 8, 68.0, 2.7, 0.4) == pytest.approx(68.0 + 2.7 * 5 + 0.4 * 6)
    assert T.t_gen(8, 8, 68.0, 2.7, 0.4) == pytest.approx(68.0 + 2.7 * 8 + 0.4 * 8)      # no call after the last draft
    assert T.t_gen(7, 8, 68.0, 2.7, 0.4) - T.t_gen(6, 8, 68.0, 2.7, 0.4) == pytest.approx(2.7 + 0.4)


def test_returns_worked_by_hand():
    a, g, R = 0.05, 0.99, 0.0421
    G = T.returns(3, 3, R, a, g)                  # stop after call 3: decisions after calls 1, 2, 3
    assert G[2] == pytest.approx(R)
    assert G[1] == pytest.approx(-a + g * R)
    assert G[0] == pytest.approx(-a - g * a + g * g * R)
    G = T.returns(4, 3, R, a, g)                  # t_max = 4 reached: three "continue" decisions, none after call 4
    assert G[2] == pytest.approx(-a + g * R)
    assert G[0] == pytest.approx(-a - g * a - g * g * a + g ** 3 * R)


def test_sample_length_inverse_cdf():
    d = [0.1, 0.2, 0.3, 0.4]
    assert T.sample_length(d, 0.05)[0] == 0
    assert T.sample_length(d, 0.1)[0] == 1        # the step edge itself belongs to the next value (strict >)
    assert T.sample_length(d, 0.59)[0] == 2
    assert T.sample_length(d, 0.95)[0] == 3
    assert T.sample_length([0.3, 0.7, 0.0, 0.0], 1.0)[0] == 1      # nothing exceeds the target: last value with mass
    assert T.sample_length([0.0, 0.0, 2.0, 0.0], 0.5)[0] == 2      # unnormalised rows are normalised by their total
    j, margin = T.sample_length(d, 0.25)
    assert j == 1 and margin == pytest.approx(0.05)


def test_gradient_matches_torch_autograd_and_finite_differences():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    k, H, t_max = 5, 16, 6
    w = _weights(rng, k, H)
    w["b2"][1] += 1.0                             # make long trajectories likely
    logs, d = _point(rng, k, t_max)
    u_act = rng.uniform(0, 0.6, size=t_max)
    hp = dict(t_max=t_max, alpha=0.05, gamma=0.99, T_o=68.0, T_d=2.7, T_p=0.4)
    loss, grad, info = T.point_loss_and_grad(w, logs, d, u_act, 0.7, **hp)
    assert len(info["actions"]) >= 3              # several steps of backpropagation through time

    # torch: the same network from library modules, the same actions and returns
    lstm = torch.nn.LSTM(k, H, batch_first=True).double()
    l1, l2 = torch.nn.Linear(H + k, H).double(), torch.nn.Linear(H, 2).double()
    with torch.no_grad():
        lstm.weight_ih_l0.copy_(torch.from_numpy(w["w_ih"])); lstm.weight_hh_l0.copy_(torch.from_numpy(w["w_hh"]))
        lstm.bias_ih_l0.copy_(torch.from_numpy(w["b_ih"])); lstm.bias_hh_l0.copy_(torch.from_numpy(w["b_hh"]))
        l1.weight.copy_(torch.from_numpy(w["w1"])); l1.bias.copy_(torch.from_numpy(w["b1"]))
        l2.weight.copy_(torch.from_numpy(w["w2"])); l2.bias.copy_(torch.from_numpy(w["b2"]))
    n = len(info["actions"])
    x = torch.from_numpy(np.exp(logs[:n]))[None]
    hs, _ = lstm(x)
    y = l2(torch.relu(l1(torch.cat([hs[0], x[0]], dim=1))))
    logp = torch.log_softmax(y, dim=1)
    tl = -(torch.from_numpy(info["G"]) * logp[torch.arange(n), torch.tensor(info["actions"])]).sum()
    tl.backward()
    assert float(tl.detach()) == pytest.approx(loss, rel=1e-12)
    ref = {"w_ih": lstm.weight_ih_l0.grad, "w_hh": lstm.weight_hh_l0.grad, "b_ih": lstm.bias_ih_l0.grad,
           "b_hh": lstm.bias_hh_l0.grad, "w1": l1.weight.grad, "b1": l1.bias.grad, "w2": l2.weight.grad, "b2": l2.bias.grad}
    for name in T.PARAM_ORDER:
        assert np.max(np.abs(grad[name] - ref[name].numpy())) < 1e-10, name

    # finite differences of the surrogate loss with the actions and returns held fixed
    def surrogate(wv):
        h, c = np.zeros(H), np.zeros(H)
        s = 0.0
        for t in range(n):
            yv, h, c = O.gate_step(np.exp(logs[t]), h, c, wv)
            z = yv - yv.max()
            s -= info["G"][t] * (z[info["actions"][t]] - np.log(np.exp(z).sum()))
        return s
    for name in T.PARAM_ORDER:
        flat = w[name].reshape(-1)
        for idx in rng.choice(flat.shape[0], size=min(4, flat.shape[0]), replace=False):
            old = flat[idx]
            e = 1e-6
            flat[idx] = old + e; up = surrogate(w)
            flat[idx] = old - e; dn = surrogate(w)
            flat[idx] = old
            assert (up - dn) / (2 * e) == pytest.approx(grad[name].reshape(-1)[idx], rel=1e-5, abs=1e-8), (name, idx)


def test_policy_gradient_identity_over_all_trajectories():
    """gamma = 1, t_max = 3: sum over action sequences and lengths of P(tau) P(l) grad-estimate equals
    -d/dtheta of the exact expected return."""
    rng = np.random.default_rng(11)
    k, H, t_max = 3, 6, 3
    w = _weights(rng, k, H)
    logs, d = _point(rng, k, t_max)
    hp = dict(t_max=t_max, alpha=0.05, gamma=1.0, T_o=1.0, T_d=0.3, T_p=0.1)

    def pis(wv):                                   # pi(continue) after calls 1 and 2
        h, c = np.zeros(H), np.zeros(H)
        out = []
        for t in range(t_max - 1):
            y, h, c = O.gate_step(np.exp(logs[t]), h, c, wv)
            z = np.exp(y - y.max())
            out.append(z[1] / z.sum())
        return out

    def expected_return(wv):
        p1, p2 = pis(wv)
        mean_len = [float(np.dot(np.arange(t_max + 1), d[i])) for i in range(t_max)]
        R = lambda Tc: mean_len[Tc - 1] / T.t_gen(Tc, t_max, hp["T_o"], hp["T_d"], hp["T_p"])
        a = hp["alpha"]
        return (1 - p1) * R(1) + p1 * (1 - p2) * (-a + R(2)) + p1 * p2 * (-2 * a + R(3))

    p1, p2 = pis(w)
    est = {n: np.zeros_like(w[n]) for n in T.PARAM_ORDER}
    total_prob = 0.0
    for acts, prob in (((0,), 1 - p1), ((1, 0), p1 * (1 - p2)), ((1, 1), p1 * p2)):
        # uniforms that force this action sequence: u < pi(1) continues
        u = np.array([0.0 if a == 1 else 1.0 for a in acts] + [0.5] * (t_max - len(acts)))
        Tc = len(acts) if acts[-1] == 0 else t_max
        cdf = np.cumsum(d[Tc - 1])
        for j in range(t_max + 1):
            v = (cdf[j] - 0.5 * d[Tc - 1][j]) / cdf[-1]          # the middle of value j's step
            _, g, info = T.point_loss_and_grad(w, logs, d, u, v, **hp)
            assert info["T"] == Tc and info["l_acc"] == j and tuple(info["actions"]) == acts
            for n in T.PARAM_ORDER:
                est[n] += prob * d[Tc - 1][j] * g[n]
            total_prob += prob * d[Tc - 1][j]
    assert total_prob == pytest.approx(1.0)
    for name in T.PARAM_ORDER:
        flat = w[name].reshape(-1)
        for idx in rng.choice(flat.shape[0], size=min(3, flat.shape[0]), replace=False):
            old, e = flat[idx], 1e-6
            flat[idx] = old + e; up = expected_return(w)
            flat[idx] = old - e; dn = expected_return(w)
            flat[idx] = old
            assert -(up - dn) / (2 * e) == pytest.approx(est[name].reshape(-1)[idx], rel=2e-5, abs=1e-9), (name, idx)


def test_adam_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    w = _weights(rng, 3, 4)
    tw = {n: torch.from_numpy(w[n].copy()).requires_grad_(True) for n in T.PARAM_ORDER}
    opt = torch.optim.Adam([tw[n] for n in T.PARAM_ORDER], lr=1e-4)
    m = {n: np.zeros_like(w[n]) for n in T.PARAM_ORDER}
    v = {n: np.zeros_like(w[n]) for n in T.PARAM_ORDER}
    cur = w
    for step in range(1, 4):
        grads = {n: rng.normal(size=w[n].shape) for n in T.PARAM_ORDER}
        for n in T.PARAM_ORDER:
            tw[n].grad = torch.from_numpy(grads[n].copy())
        opt.step()
        cur, m, v = T.adam_step(cur, grads, m, v, step, 1e-4)
        for n in T.PARAM_ORDER:
            assert np.max(np.abs(cur[n] - tw[n].detach().numpy())) < 1e-12, (n, step)
