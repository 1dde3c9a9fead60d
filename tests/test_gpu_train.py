"""REINFORCE step of the prediction model on the GPU against the training oracle (Sec. 4.2 Eq. 3-10,
Sec. 4.3): trajectories, acceptance lengths and actions bit-exact, loss and every parameter gradient within
tolerance, the Adam update over three steps; and one batch whose {S, D} come from the library itself
(expansion + tree + Eq. 11-13 for every number of draft calls)."""
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


HP = dict(alpha=0.05, gamma=0.99, T_o=68.0, T_d=2.7, T_p=0.4)        # latency terms of the paper's Table 5 (ms)
TAU_ACTION = 1e-5         # |u - pi(continue)| below this: the fp32 kernel and the fp64 oracle may decide differently
TAU_LENGTH = 1e-9


def _theta(w):
    from oracle import train_oracle as T
    return np.concatenate([np.asarray(w[n], np.float32).reshape(-1) for n in T.PARAM_ORDER])


def _split(theta, k):
    from oracle import train_oracle as T
    Hh = 128
    shapes = {"w_ih": (4 * Hh, k), "w_hh": (4 * Hh, Hh), "b_ih": (4 * Hh,), "b_hh": (4 * Hh,), "w1": (Hh, Hh + k),
              "b1": (Hh,), "w2": (2, Hh), "b2": (2,)}
    out, o = {}, 0
    for n in T.PARAM_ORDER:
        sz = int(np.prod(shapes[n]))
        out[n] = theta[o:o + sz].reshape(shapes[n])
        o += sz
    assert o == theta.shape[0]
    return out


class Trainer:
    def __init__(self, ctx, n, k, t_max, theta):
        import torch
        from paper_2512_14069_b200 import binding as rb
        self.torch, self.rb, self.ctx, self.n, self.k, self.t_max = torch, rb, ctx, n, k, t_max
        Pn = rb.radar_policy_param_count(k)
        assert Pn == theta.shape[0]
        dev = "cuda:0"
        self.theta = torch.from_numpy(theta.copy()).to(dev)
        self.m, self.v, self.grad = (torch.zeros(Pn, device=dev) for _ in range(3))
        self.loss = torch.zeros(1, device=dev)
        self.calls, self.l_acc = torch.zeros(n, dtype=torch.int32, device=dev), torch.zeros(n, dtype=torch.int32, device=dev)
        self.actions = torch.zeros((n, t_max), dtype=torch.uint8, device=dev)
        self.ws = torch.zeros(rb.radar_train_workspace_bytes(ctx, n, k, t_max), dtype=torch.uint8, device=dev)

    def step(self, log_states, dists, u_action, u_length, step, lr=1e-4):
        self.rb.radar_policy_train_step(
            self.ctx, n=self.n, k=self.k, t_max=self.t_max, log_states=log_states, dists=dists, u_action=u_action,
            u_length=u_length, theta=self.theta, grad=self.grad, loss=self.loss, calls=self.calls, l_acc=self.l_acc,
            actions=self.actions, workspace=self.ws, step=step, lr=lr, adam_m=self.m, adam_v=self.v, **HP)
        self.ctx.check_device_status()


def _compare(tr, w, batch, infos, loss, grad):
    n, t_max = tr.n, tr.t_max
    assert min(i["action_margin"] for i in infos) > TAU_ACTION and min(i["length_margin"] for i in infos) > TAU_LENGTH
    calls, l_acc, actions = tr.calls.cpu().numpy(), tr.l_acc.cpu().numpy(), tr.actions.cpu().numpy()
    for j, info in enumerate(infos):
        assert calls[j] == info["T"] and l_acc[j] == info["l_acc"], j
        nd = len(info["actions"])
        assert list(actions[j, :nd]) == info["actions"] and np.all(actions[j, nd:] == 255), j
    assert float(tr.loss.cpu()) == pytest.approx(loss, rel=2e-5, abs=1e-6)
    g_gpu = _split(tr.grad.cpu().numpy().astype(np.float64), tr.k)
    scale = max(float(np.max(np.abs(grad[m]))) for m in grad)
    for m in grad:
        assert np.max(np.abs(g_gpu[m] - grad[m])) <= 2e-5 * scale + 1e-9, (m, float(np.max(np.abs(g_gpu[m] - grad[m]))), scale)


@pytest.mark.parametrize("n,k,t_max,seed", [(37, 10, 8, 0), (256, 10, 8, 1), (5, 4, 3, 2), (16, 32, 16, 3)])
def test_train_step_matches_oracle(ctx, n, k, t_max, seed):
    from oracle import train_oracle as T
    cfg = W.shrink(W.CONFIGS[2], cid=300 + seed, k=k, t_max=t_max)
    w = W.gate_weights(cfg)
    w["b2"][1] += np.float32(0.8)                     # trajectories of every length
    log_states, dists, u_action, u_length = W.train_batch(cfg, n, seed)
    loss, grad, infos = T.batch_loss_and_grad(w, log_states, dists, u_action, u_length, t_max, **HP)
    assert len({i["T"] for i in infos}) >= min(3, t_max - 1)
    tr = Trainer(ctx, n, k, t_max, _theta(w))
    dev = [H.to_dev(x) for x in (log_states, dists, u_action, u_length)]
    tr.step(*dev, step=0)
    _compare(tr, w, None, infos, loss, grad)
    assert np.array_equal(tr.theta.cpu().numpy(), _theta(w))             # step 0 leaves the parameters alone


def test_three_adam_steps_match_oracle(ctx):
    from oracle import train_oracle as T
    n, k, t_max = 64, 10, 8
    cfg = W.shrink(W.CONFIGS[2], cid=310)
    w = {m: np.asarray(v, np.float64) for m, v in W.gate_weights(cfg).items()}
    w["b2"][1] += 0.8
    tr = Trainer(ctx, n, k, t_max, _theta(w))
    m = {q: np.zeros_like(w[q]) for q in T.PARAM_ORDER}
    v = {q: np.zeros_like(w[q]) for q in T.PARAM_ORDER}
    for step in range(1, 4):
        batch = W.train_batch(cfg, n, 10 + step)
        # the oracle continues from the parameters the GPU holds (fp32), so rounding does not accumulate into decisions
        w = {q: a.astype(np.float64) for q, a in _split(tr.theta.cpu().numpy(), k).items()}
        loss, grad, infos = T.batch_loss_and_grad(w, *batch, t_max, **HP)
        w_new, m, v = T.adam_step(w, grad, m, v, step, 1e-3)
        tr.step(*[H.to_dev(x) for x in batch], step=step, lr=1e-3)
        _compare(tr, w, None, infos, loss, grad)
        got = _split(tr.theta.cpu().numpy().astype(np.float64), k)
        for q in T.PARAM_ORDER:
            # an Adam step moves a parameter by about lr whatever the gradient's size: compare on that scale
            assert np.max(np.abs(got[q] - w_new[q])) <= 0.02 * 1e-3, (q, step)
        m = {q: a.astype(np.float64) for q, a in _split(tr.m.cpu().numpy(), k).items()}
        v = {q: a.astype(np.float64) for q, a in _split(tr.v.cpu().numpy(), k).items()}


def test_train_step_argument_errors(ctx):
    import torch
    from paper_2512_14069_b200 import binding as rb
    tr = Trainer(ctx, 4, 10, 8, np.zeros(rb.radar_policy_param_count(10), np.float32))
    cfg = W.shrink(W.CONFIGS[2], cid=320)
    dev = [H.to_dev(x) for x in W.train_batch(cfg, 4, 0)]
    with pytest.raises(rb.RadarError) as e:
        rb.radar_policy_train_step(ctx, n=4, k=10, t_max=8, log_states=dev[0], dists=dev[1], u_action=dev[2], u_length=dev[3],
                                   theta=tr.theta, grad=tr.grad, loss=tr.loss, calls=tr.calls, l_acc=tr.l_acc,
                                   actions=tr.actions, workspace=tr.ws[:1024], **HP)
    assert e.value.status == -3
    with pytest.raises(rb.RadarError) as e:
        rb.radar_policy_train_step(ctx, n=4, k=10, t_max=40, log_states=dev[0], dists=dev[1], u_action=dev[2], u_length=dev[3],
                                   theta=tr.theta, grad=tr.grad, loss=tr.loss, calls=tr.calls, l_acc=tr.l_acc,
                                   actions=tr.actions, workspace=tr.ws, **HP)
    assert e.value.status == -1
    with pytest.raises(rb.RadarError) as e:                              # an update without optimiser state
        rb.radar_policy_train_step(ctx, n=4, k=10, t_max=8, log_states=dev[0], dists=dev[1], u_action=dev[2], u_length=dev[3],
                                   theta=tr.theta, grad=tr.grad, loss=tr.loss, calls=tr.calls, l_acc=tr.l_acc,
                                   actions=tr.actions, workspace=tr.ws, step=1, **HP)
    assert e.value.status == -1


def test_dataset_from_the_library_then_a_train_step(ctx):
    """The offline data set of Sec. 4.3 built by the library itself, on device buffers end to end: for every number
    of draft calls i the expansion is forced to i calls, the tree is built and Eq. 11-13 gives d_i, written straight
    into slice i - 1 of `dists`; the states are the frontier scores of the t_max-call run.  Both are checked against
    the oracle, then one REINFORCE step runs on them and is compared with the training oracle."""
    import torch
    from oracle import accept_oracle as A
    from oracle import train_oracle as T
    from paper_2512_14069_b200 import binding as rb
    cfg = W.shrink(W.CONFIGS[3], cid=330, B=6, V=3001, P=(64, 64), Hq=4, Hkv=4, t_max=5, N=24)
    k, t_max, n = cfg.k, cfg.t_max, cfg.B
    inp = H.make_inputs(cfg, with_attention=False)
    g = H.CudaRun(cfg, inp, ctx)
    s = g.step
    dists = torch.zeros((t_max, n, t_max + 1), dtype=torch.float64, device="cuda")
    pacc = torch.zeros((n, 64), dtype=torch.float64, device="cuda")
    wb = rb.radar_acclen_workspace_bytes(ctx, n, cfg.V)
    ws = torch.zeros(wb + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    d_ref = np.zeros((t_max, n, t_max + 1))
    for i in range(1, t_max + 1):
        inp["force_calls"] = np.full(n, i, np.int32)
        g.force = H.to_dev(inp["force_calls"])
        _, traces, trees = H.oracle_expand_and_tree(cfg, inp)
        target = H.make_target(cfg, inp, trees)
        g.expand_and_tree()
        rb.radar_accept_length_distribution(
            ctx, B=n, V=cfg.V, t_max=t_max, temperature=1.0, target_logits=H.to_dev(target), tree_tok=s.tree_tok,
            tree_parent=s.tree_parent, tree_depth=s.tree_depth, tree_draft_row=s.tree_draft_row, n_nodes=s.n_nodes,
            draft_logits=g.draft, R=s.R, dist=dists[i - 1], p_acc_node=pacc, workspace=ws[off:off + wb])
        ctx.check_device_status()
        for b in range(n):
            d_ref[i - 1, b], _ = A.accept_length_distribution(target[b], inp["draft"][b], trees[b], 1.0, t_max)
    assert np.max(np.abs(dists.cpu().numpy() - d_ref)) < 1e-9
    assert np.all(d_ref[0, :, 2:] == 0.0)                       # one draft call cannot accept more than one token
    log_states = s.frontier_score                               # [t_max][n][k], left by the run with t_max calls
    ref_states = np.stack([np.stack([traces[b][t]["frontier_score"] for b in range(n)]) for t in range(t_max)])
    assert np.max(np.abs(log_states.cpu().numpy() - ref_states)) <= 1e-5

    w = dict(inp["gate"])
    w["b2"] = w["b2"].copy()
    w["b2"][1] += np.float32(0.5)
    u_action, u_length = W.train_batch(cfg, n, 5)[2:]
    loss, grad, infos = T.batch_loss_and_grad(w, log_states.cpu().numpy(), dists.cpu().numpy(), u_action, u_length, t_max, **HP)
    tr = Trainer(ctx, n, k, t_max, _theta(w))
    tr.step(log_states, dists, H.to_dev(u_action), H.to_dev(u_length), step=0)
    _compare(tr, w, None, infos, loss, grad)
