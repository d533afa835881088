"""Pins of the oracle's value-based variant (n-step Q-learning on the parallel framework: Section 3 allows an
implicit policy; Section 2.2, Eqs. 2-4 give target, loss and gradient).  CPU only."""
import numpy as np
import torch



def test_greedy_is_first_arg_max(orc):
    rng = np.random.RandomState(0)
    for _ in range(300):
        A = rng.randint(2, 33)
        q = rng.randint(-3, 4, A).astype(np.float32) * 0.25          # many ties
        assert orc.q_greedy(q) == int(np.argmax(q))                   # numpy takes the first of equal maxima
        assert orc.q_select(q, 0.999, 0.25) == int(np.argmax(q))      # not exploring: greedy
        assert orc.q_select(q, 0.0, 0.0) == int(np.argmax(q))         # epsilon 0 never explores


def test_exploration_branch_special_cases_and_frequencies(orc):
    q = np.array([0.0, 1.0, 5.0, 2.0], np.float32)
    # u = 0 explores into action 0; u just under epsilon into the last action; u = epsilon is greedy again
    assert orc.q_select(q, 0.0, 0.1) == 0
    assert orc.q_select(q, float(np.nextafter(np.float32(0.1), np.float32(0))), 0.1) == 3
    assert orc.q_select(q, 0.1, 0.1) == 2
    # epsilon = 1, A a power of two, dyadic u: the action is exactly floor(u A)
    q8 = np.zeros(8, np.float32)
    for k in range(8):
        assert orc.q_select(q8, k / 8.0, 1.0) == k
        assert orc.q_select(q8, (k + 0.5) / 8.0, 1.0) == k
    # with the environment's own uniforms: a fraction epsilon of the decisions explores, evenly over the actions
    eps, A, n = 0.2, 6, 20000
    q6 = np.array([0, 0, 0, 9, 0, 0], np.float32)
    us = [orc.action_uniform(11, e, 3) for e in range(n)]
    acts = np.array([orc.q_select(q6, u, eps) for u in us])
    explored = np.array([u < eps for u in us])
    assert abs(explored.mean() - eps) < 4 * np.sqrt(eps * (1 - eps) / n)
    assert np.all(acts[~explored] == 3)
    counts = np.bincount(acts[explored], minlength=A)
    expect = explored.sum() / A
    assert np.all(np.abs(counts - expect) < 5 * np.sqrt(expect))


def test_q_margin(orc):
    assert abs(orc.q_margin(np.array([0.1, 0.5, 0.4], np.float32)) - 0.1) < 1e-7
    assert orc.q_margin(np.array([0.5, 0.5, 0.4], np.float32)) == 0.0


def test_q_head_gradient_hand_case_autograd_and_finite_differences(orc):
    # hand case: B = 2, A = 3, c = 1: L = ((1 - 3)^2 + (0.5 - 0)^2) / 2 = 2.125,
    # dL/dQ_0[2] = 2 (3 - 1) / 2 = 2,  dL/dQ_1[0] = 2 (0 - 0.5) / 2 = -0.5, all else 0
    q = np.array([[1, 2, 3], [0, 0, 0]], np.float32)
    dq, st = orc.q_head_grad(1.0, q, np.array([2, 0]), np.array([1.0, 0.5], np.float32))
    assert np.array_equal(dq, np.array([[0, 0, 2], [-0.5, 0, 0]], np.float32))
    assert abs(st["value_loss"] - 2.125) < 1e-12 and abs(st["mean_max_q"] - 1.5) < 1e-12
    # against autograd of the loss as the equations state it
    rng = np.random.RandomState(2)
    B, A, c = 9, 5, 0.7
    q = rng.randn(B, A).astype(np.float32)
    a = rng.randint(0, A, B)
    R = rng.randn(B).astype(np.float32)
    dq, st = orc.q_head_grad(c, q, a, R)
    qt = torch.tensor(q, dtype=torch.float64, requires_grad=True)
    loss = c * ((torch.tensor(R, dtype=torch.float64) - qt.gather(1, torch.tensor(a)[:, None])[:, 0]) ** 2).mean()
    loss.backward()
    assert np.allclose(dq, qt.grad.numpy(), rtol=1e-6, atol=1e-9)
    assert abs(st["value_loss"] - float(loss.detach())) < 1e-6          # c = 0.7 is a float on the oracle side
    # central differences of the oracle's own loss value
    h = 1e-3
    for i, k in ((0, int(a[0])), (3, int(a[3])), (3, (int(a[3]) + 1) % A)):
        qp, qm = q.astype(np.float64).copy(), q.astype(np.float64).copy()
        qp[i, k] += h
        qm[i, k] -= h
        lp = orc.q_head_grad(c, qp.astype(np.float32), a, R)[1]["value_loss"]
        lm = orc.q_head_grad(c, qm.astype(np.float32), a, R)[1]["value_loss"]
        assert abs((lp - lm) / (2 * h) - dq[i, k]) < 2e-4


def test_nstep_q_iteration_follows_the_equations(orc):
    """On a tiny network: the stored value of a step is Q(s_t, a_t), the bootstrap is max_a Q of the last state,
    the targets are the n-step returns from it (worked case of the returns test: gamma 0.5, rewards (1, 0, -1),
    bootstrap 4 -> (1.25, 0.5, 1)), acting with epsilon = 0 is the arg max, and the parameter gradient is the
    autograd gradient of Eq. 3's loss through the network."""
    R, adv = orc.returns(0.5, np.array([[1], [0], [-1]], np.int8), np.zeros((3, 1), np.uint8),
                         np.array([[0.5], [0.25], [2.0], [max(1.0, 4.0, 2.0)]], np.float32))
    assert np.allclose(R[:, 0], [1.25, 0.5, 1.0]) and np.allclose(adv[:, 0], [0.75, 0.25, -1.0])
    net = orc.make_net((12, 12, 4), [(2, 4, 2)], 4, 3)
    hp = dict(algorithm="nstep_q", epsilon=0.0, gamma=0.9, lr=0.01, term_denom=3)
    o = orc.OraclePAAC("tiny", 4, 3, 3, seed=5, hp=hp, net=net)
    th0 = o.theta.copy()
    ro = o.rollout()
    T, n_e = 3, 4
    for t in range(T):
        _, z, _ = orc.forward(net, th0, ro["frames"][t])
        assert np.array_equal(ro["actions"][t], z.argmax(1))
        assert np.array_equal(ro["values"][t], z[np.arange(n_e), ro["actions"][t]])
    _, zb, _ = orc.forward(net, th0, ro["frames"][T])
    assert np.array_equal(ro["values"][T], zb.max(1))
    up = o.update()
    # autograd of c mean (R - Q(s, a))^2 through the same tiny network in float64
    from test_oracle_pins import rel, torch_forward, torch_params
    ps, _ = torch_params(net, th0)
    leaves = [(W.clone().requires_grad_(True), b.clone().requires_grad_(True)) for W, b in ps]
    frames = ro["frames"][:T].reshape(T * n_e, 12, 12, 4)
    _, logits, _ = torch_forward(net, leaves, frames)
    a = torch.tensor(ro["actions"].reshape(-1).astype(np.int64))
    Rt = torch.tensor(up["R"].reshape(-1), dtype=torch.float64)
    loss = ((Rt - logits.gather(1, a[:, None])[:, 0]) ** 2).mean()
    loss.backward()
    g = torch.cat([torch.cat([W.grad.reshape(-1) if W.grad is not None else torch.zeros(W.numel(), dtype=torch.float64),
                              b.grad.reshape(-1) if b.grad is not None else torch.zeros(b.numel(), dtype=torch.float64)])
                   for W, b in leaves]).numpy()
    assert g.shape == up["grad"].shape
    assert rel(up["grad"], g) < 2e-5
    assert abs(up["value_loss"] - float(loss.detach())) < 1e-6
    # the value head took no part: its gradient is exactly zero
    assert np.all(up["grad"][-(net.fc + 1):] == 0)
