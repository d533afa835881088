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
    o = orc.OraclePAAC(cfg["arch"], cfg["n_e"], cfg["t_max"], cfg["n_actions"], seed, bf16=bf16, hp=hp)
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
    for t, e in zip(*np.nonzero(sampled != ro["actions"])):
        band = 1e-5 + float(np.abs(pg[t, e] - ro["probs"][t, e]).sum())
        assert orc.cdf_margin(ro["probs"][t, e], float(ro["uniforms"][t, e])) <= band, (t, e)
        mism += 1
    rep["action_mismatches"] = mism
    return ro, rep


def check_update(orc, o, g, tol, check_acts=True):
    L = o.net.n_conv
    B = o.n_e * o.t_max
    up = o.update()
    st = g.update()
    rep = {}
    assert st["status"] == 0 and st["timesteps"] == o.N
    rep["R"] = rel(g.debug_read(pb.DBG_RETURNS), up["R"])
    rep["adv"] = rel(g.debug_read(pb.DBG_ADVANTAGES), up["adv"])
    rep["dz"] = rel(g.debug_read(pb.DBG_DLOGITS), up["dz"])
    rep["dV"] = rel(g.debug_read(pb.DBG_DVALUES), up["dV"])
    if check_acts:
        for l in range(L + 1):
            rep["act%d" % l] = rel(g.debug_read(pb.DBG_ACT0 + l), up["acts"][l])
            rep["gact%d" % l] = rel(g.debug_read(pb.DBG_GACT0 + l), up["gacts"][l])
    grad = g.debug_read(pb.DBG_GRAD)
    for name, sl in layer_slices(orc, o.net):
        rep["g." + name] = rel(grad[sl], up["grad"][sl])
    rep["grad"] = rel(grad, up["grad"])
    for k, v in rep.items():
        assert v <= tol, (k, v, rep)
    for k in ("policy_loss", "value_loss", "entropy"):
        assert abs(st[k] - up[k]) <= tol * max(1.0, abs(up[k])), (k, st[k], up[k])
    assert abs(st["grad_norm"] - up["grad_norm"]) <= tol * up["grad_norm"]
    assert abs(st["clip_scale"] - up["clip_scale"]) <= tol
    rep["theta"] = rel(g.params(), o.theta)
    rep["rms"] = rel(g.debug_read(pb.DBG_RMS), o.m)
    return up, st, rep
