"""Helpers that walk the CUDA library and the CPU oracle through the same iterations."""
import numpy as np

from paper_1705_04862_b200 import binding as pb
from paper_1705_04862_b200.configs import COMMON

TOL = {"fp32": 1e-4, "bf16": 2e-2}      # logits / values / gradients, relative to the tensor's max
TOL_PARAMS_10 = 1e-3                     # parameters after 10 updates


def rel(x, y):
    x = np.asarray(x, np.float64).reshape(-1)
    y = np.asarray(y, np.float64).reshape(-1)
    assert x.shape == y.shape, (x.shape, y.shape)
    return float(np.abs(x - y).max() / (np.abs(y).max() + 1e-12))


def make_pair(orc, cfg, seed=None):
    seed = COMMON["seed"] if seed is None else seed
    bf16 = cfg["precision"] == "bf16"
    hp = dict(gamma=COMMON["gamma"], lr=cfg["lr"], rms_decay=COMMON["rms_decay"], rms_eps=COMMON["rms_eps"],
              clip_norm=COMMON["clip_norm"], entropy_beta=COMMON["entropy_beta"], value_coef=COMMON["value_coef"],
              term_denom=cfg["term_denom"])
    ohp = dict(hp)
    if cfg.get("algorithm", "a2c") == "nstep_q":
        ohp.update(algorithm="nstep_q", epsilon=cfg.get("epsilon", 0.1))
        hp.update(algorithm=pb.ALGO_NSTEP_Q, epsilon=cfg.get("epsilon", 0.1))
    if cfg.get("environment", "hashed") == "pattern":
        ohp.update(environment="pattern")
        hp.update(environment=pb.ENV_PATTERN)
    o = orc.OraclePAAC(cfg["arch"], cfg["n_e"], cfg["t_max"], cfg["n_actions"], seed, bf16=bf16, hp=ohp)
    g = pb.Paac(cfg["arch"], cfg["n_e"], cfg["t_max"], cfg["n_actions"], seed,
                precision=pb.BF16 if bf16 else pb.FP32, **hp)
    return o, g


def layer_slices(orc, net):
    """[(name, slice)] over the canonical parameter vector."""
    out, o, h, w, c = [], 0, net.in_h, net.in_w, net.in_c
    for l in range(net.n_conv):
        n = net.cout[l] * net.k[l] ** 2 * c
        out += [("conv%d.W" % (l + 1), slice(o, o + n)), ("conv%d.b" % (l + 1), slice(o + n, o + n + net.cout[l]))]
        o += n + net.cout[l]
        h, w, c = (h - net.k[l]) // net.stride[l] + 1, (w - net.k[l]) // net.stride[l] + 1, net.cout[l]
    fin = h * w * c
    for name, rows, cols in (("fc", net.fc, fin), ("pi", net.n_actions, net.fc), ("v", 1, net.fc)):
        out += [(name + ".W", slice(o, o + rows * cols)), (name + ".b", slice(o + rows * cols, o + rows * cols + rows))]
        o += rows * cols + rows
    assert o == orc.param_count(net)
    return out


def resync(o, g):
    """Give the library the oracle's parameters and RMSProp state.  With bf16 storage two correct
    implementations drift apart within a few updates (a parameter difference far below one bf16
    unit still flips the rounding of many weights and activations, and the differences grow about
    tenfold per update), so the bf16 cases compare one iteration at a time from a common start."""
    g.set_params(o.theta)
    g.debug_write(pb.DBG_RMS, o.m)


def check_rollout(orc, o, g, tol, lockstep=True):
    """Oracle rolls out with its own sampling; the library is forced onto the oracle's actions so
    that a tolerated near-boundary difference cannot cascade, and its own draw is compared."""
    T, n_e, A = o.t_max, o.n_e, o.A
    ro = o.rollout()
    if lockstep:
        g.force_actions(ro["actions"])
    g.rollout()
    rep = {}
    assert np.array_equal(g.debug_read(pb.DBG_FRAMES).reshape(T, n_e, -1), ro["frames"][:T].reshape(T, n_e, -1))
    assert np.array_equal(g.debug_read(pb.DBG_NEXT_FRAMES).reshape(n_e, -1), ro["frames"][T].reshape(n_e, -1))
    assert np.array_equal(g.debug_read(pb.DBG_REWARDS).reshape(T, n_e), ro["rewards"])
    assert np.array_equal(g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e), ro["terminals"])
    assert np.array_equal(g.debug_read(pb.DBG_ACTIONS).reshape(T, n_e), ro["actions"])
    assert np.array_equal(g.debug_read(pb.DBG_UNIFORMS).reshape(T, n_e), ro["uniforms"])      # bit-exact Philox
    cnt = g.debug_read(pb.DBG_COUNTERS).reshape(3, n_e)
    for j in range(3):
        assert np.array_equal(cnt[j], o.counters[j])
    logits = g.debug_read(pb.DBG_LOGITS).reshape(T, n_e, A)
    values = g.debug_read(pb.DBG_VALUES).reshape(T + 1, n_e)
    rep["logits"] = rel(logits, ro["logits"])
    rep["values"] = rel(values, ro["values"])
    assert rep["logits"] <= tol and rep["values"] <= tol, rep
    # sampled actions: identical unless the uniform sits within rounding of a CDF boundary
    sampled = g.debug_read(pb.DBG_SAMPLED).reshape(T, n_e)
    pg, _, _ = orc.softmax(logits)
    mism = 0
    want = ro["sampled"] if lockstep else ro["actions"]       # what the oracle's own decision rule gave
    for t, e in zip(*np.nonzero(sampled != want)):
        if o.hp["algorithm"] == "nstep_q":
            # the exploring branch is integer-exact; two greedy choices may differ only when the two largest
            # Q-values are closer than the two sides' Q-values are to each other
            assert float(ro["uniforms"][t, e]) >= o.hp["epsilon"], (t, e)
            band = 1e-6 + 2.0 * float(np.abs(logits[t, e] - ro["logits"][t, e]).max())
            assert orc.q_margin(ro["logits"][t, e]) <= band, (t, e)
        else:
            band = 1e-5 + float(np.abs(pg[t, e] - ro["probs"][t, e]).sum())
            assert orc.cdf_margin(ro["probs"][t, e], float(ro["uniforms"][t, e])) <= band, (t, e)
        mism += 1
    rep["action_mismatches"] = mism
    return ro, rep


FLIP_L2 = 5e-2
# how often check_update met ReLU flips (library updating from its own rollout): calls without injection, calls
# that took the flip branch, and the largest number of flipped units seen in one call
FLIP_STATS = {"calls": 0, "with_flips": 0, "max_flips": 0, "units_checked": 0}


def check_update(orc, o, g, tol, check_acts=True, inject=False):
    """One update on both sides, compared tensor by tensor (max norm relative to the tensor's
    largest magnitude, `rel`).

    inject=True: the oracle's stored activations, logits and values are first written into the
    library, so both backward passes start from identical tensors and ReLU masks; every tensor
    must then meet the tolerance.

    inject=False: the library updates from its own rollout.  A unit whose pre-activation is within
    rounding of zero can be switched on on one side and off on the other; both are valid, but such
    a flip moves gradient elements below it by a whole term of their sums.  If no unit flipped,
    every tensor must meet the tolerance; if some did (they must be rare and sit at numerically
    zero activation), the activation gradients are compared where the masks agree and the
    parameter gradients in the L2 sense against FLIP_L2; the parameters must still meet
    TOL_PARAMS_10 after the step, and the step and the RMSProp state agree in the L2 sense.
    FLIP_STATS records how often this branch is taken.
    Returns (oracle update, library stats, report); report["flips"] counts flipped units."""
    L = o.net.n_conv
    theta_before = o.theta.copy()
    up = o.update()
    if inject:
        for l in range(L + 1):
            g.debug_write_act(l, up["acts"][l])
        g.debug_write(pb.DBG_LOGITS, up["logits"])
        g.debug_write(pb.DBG_VALUES, o.ro["values"])
    st = g.update()
    rep, loose = {}, {}
    assert st["status"] == 0 and st["timesteps"] == o.N
    for k, w in (("R", pb.DBG_RETURNS), ("adv", pb.DBG_ADVANTAGES), ("dz", pb.DBG_DLOGITS), ("dV", pb.DBG_DVALUES)):
        rep[k] = rel(g.debug_read(w), up[k])
    acts_g = [g.debug_read(pb.DBG_ACT0 + l) for l in range(L + 1)]
    acts_o = [up["acts"][l].reshape(-1) for l in range(L + 1)]
    agree = [(a > 0) == (b > 0) for a, b in zip(acts_g, acts_o)]
    flips = int(sum((~m).sum() for m in agree))
    rep["flips"] = 0.0
    for l in range(L + 1):
        rep["act%d" % l] = rel(acts_g[l], acts_o[l])
        if inject:
            assert np.array_equal(acts_g[l], acts_o[l])
        bad = ~agree[l]
        assert bad.mean() <= 5e-3, (l, bad.mean())
        if bad.any():
            assert max(acts_g[l][bad].max(), acts_o[l][bad].max()) <= tol * np.abs(acts_o[l]).max(), l
        if check_acts or flips:
            ga_g, ga_o = g.debug_read(pb.DBG_GACT0 + l), up["gacts"][l].reshape(-1)
            if flips == 0:
                rep["gact%d" % l] = rel(ga_g, ga_o)
            else:
                d = (ga_g.astype(np.float64) - ga_o)[agree[l]]
                loose["gact%d" % l] = float(np.linalg.norm(d) / (np.linalg.norm(ga_o[agree[l]]) + 1e-30))
    grad = g.debug_read(pb.DBG_GRAD)
    for name, sl in layer_slices(orc, o.net) + [("all", slice(None))]:
        gg, go = grad[sl].astype(np.float64), up["grad"][sl].astype(np.float64)
        if flips == 0:
            rep["g." + name] = rel(gg, go)
        else:
            loose["g." + name] = float(np.linalg.norm(gg - go) / (np.linalg.norm(go) + 1e-30))
    for k, v in rep.items():
        assert v <= tol, (k, v, rep, loose)
    for k, v in loose.items():
        assert v <= FLIP_L2, (k, v, rep, loose)
    stat_tol = tol if flips == 0 else FLIP_L2
    for k in ("policy_loss", "value_loss", "entropy"):
        assert abs(st[k] - up[k]) <= tol * max(1.0, abs(up[k])), (k, st[k], up[k])
    assert abs(st["grad_norm"] - up["grad_norm"]) <= stat_tol * up["grad_norm"]
    assert abs(st["clip_scale"] - up["clip_scale"]) <= stat_tol
    rep.update(loose)
    rep["flips"] = flips
    theta_g, rms_g = g.params(), g.debug_read(pb.DBG_RMS)
    rep["theta"] = rel(theta_g, o.theta)
    rep["rms"] = rel(rms_g, o.m)
    if not inject:
        FLIP_STATS["calls"] += 1
        FLIP_STATS["units_checked"] += int(sum(a.size for a in acts_o))
        if flips:
            FLIP_STATS["with_flips"] += 1
            FLIP_STATS["max_flips"] = max(FLIP_STATS["max_flips"], flips)
    if flips:
        # the flip branch still pins the optimiser: parameters within TOL_PARAMS_10, step and state in the L2 sense
        assert rep["theta"] <= TOL_PARAMS_10, rep
        ds = (theta_g.astype(np.float64) - theta_before) - (o.theta.astype(np.float64) - theta_before)
        rep["step_l2"] = float(np.linalg.norm(ds) / (np.linalg.norm(o.theta.astype(np.float64) - theta_before) + 1e-30))
        rep["rms_l2"] = float(np.linalg.norm(rms_g.astype(np.float64) - o.m) / (np.linalg.norm(o.m) + 1e-30))
        assert rep["step_l2"] <= FLIP_L2 and rep["rms_l2"] <= 2 * FLIP_L2, rep
    return up, st, rep


def adopt_library_state(o, g, updates):
    """Continue the oracle from where a free-running library stands after `updates` updates: parameters, RMSProp
    state, timestep counter, current states and episode counters are read from the library (integers and stored
    floats, copied bit for bit); nothing the comparison that follows checks is taken from it."""
    o.theta = g.params()
    o.m = g.debug_read(pb.DBG_RMS).copy()
    o.N = updates * o.n_e * o.t_max
    o.state = g.debug_read(pb.DBG_NEXT_FRAMES).reshape(o.n_e, 84, 84, 4).copy()
    for j, c in enumerate(g.debug_read(pb.DBG_COUNTERS).reshape(3, -1)):
        o.counters[j][:] = c
