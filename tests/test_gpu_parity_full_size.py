"""The throughput configuration (Nature CNN, bf16, n_e = 1024, t_max = 5: 5120 experiences per update) and
the late-update protocol of the bf16 configurations, against the CPU oracle at full size, through the C-ABI.

The launch shapes here are the ones the bench times: every persistent kernel walks many tiles per CTA, so the
stage rings wrap, both accumulator phases alternate many times and the split-k ranges are the full-size ones.
The oracle's inputs are its own (frames from its integer environment, its own parameters); the library is put
on the oracle's actions so that a tolerated near-boundary draw cannot cascade.
"""
import numpy as np
import pytest

from paper_1705_04862_b200 import binding as pb
from paper_1705_04862_b200.configs import CONFIGS

from parity_util import (FLIP_STATS, TOL, TOL_PARAMS_10, adopt_library_state, check_rollout, check_update, make_pair,
                         rel, resync)

pytestmark = pytest.mark.gpu


def _stored_activations_agree(o, g, ro, tol):
    """The four stored activations of the rollout, all environments and steps, element by element."""
    T, n_e = o.t_max, o.n_e
    rep = {}
    for l in range(o.net.n_conv + 1):
        got = g.debug_read(pb.DBG_ACT0 + l).reshape(T, n_e, -1)
        want = np.stack([ro["acts"][t][l].reshape(n_e, -1) for t in range(T)])
        rep["act%d" % l] = rel(got, want)
        # per environment group too: a tile that went wrong late in a CTA's walk must not hide behind the
        # largest element of the whole tensor
        scale = np.abs(want).max()
        per_env = np.abs(got.astype(np.float64) - want).max(axis=(0, 2)) / scale
        assert per_env.max() <= tol, (l, int(per_env.argmax()), float(per_env.max()))
    return rep


def test_config5_full_size_iteration_against_the_oracle(orc, capsys):
    """One whole iteration at n_e = 1024 in lock step with a 1024-environment oracle: every frame, reward,
    terminal and uniform bit for bit; logits, values and the four stored activations of all 5120 + 1024 states;
    then the 5120-row update from identical forward tensors: every activation gradient, the gradient of every
    layer, the parameter step and the RMSProp state.  A second iteration updates from the library's own
    rollout (its own ReLU masks)."""
    cfg = CONFIGS[4]
    o, g = make_pair(orc, cfg)
    assert np.array_equal(g.params(), o.theta)
    tol = TOL["bf16"]
    ro, r1 = check_rollout(orc, o, g, tol)
    r1.update(_stored_activations_agree(o, g, ro, tol))
    th0 = o.theta.copy()
    up, st, r2 = check_update(orc, o, g, tol, inject=True)
    assert r2["flips"] == 0
    assert r2["theta"] <= TOL_PARAMS_10 and r2["rms"] <= tol
    assert rel(g.params() - th0, o.theta - th0) <= tol                 # the step itself
    for l in range(4):
        assert r2["gact%d" % l] <= tol
    # second iteration: from the oracle's parameters again, the update from the library's own forward pass
    resync(o, g)
    ro, r3 = check_rollout(orc, o, g, tol)
    up, st, r4 = check_update(orc, o, g, tol, inject=False)
    with capsys.disabled():
        print("\n[config 5 full size] rollout %s\n  update (identical masks) %s\n  update (own masks) %s"
              % ({k: float("%.3g" % v) for k, v in r1.items()}, {k: float("%.3g" % v) for k, v in r2.items()},
                 {k: float("%.3g" % v) for k, v in r4.items()}))
    g.close()


def _free_run_then_compare(orc, cfg, updates, capsys):
    """Late-update check for the bf16 configurations: the library runs `updates` iterations by itself on a stream of its
    own (CUDA graphs replay from the third), then the oracle adopts its state and both do one more iteration
    that is compared tensor by tensor, once from the library's own forward pass and once from identical ones."""
    import torch
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        o, g = make_pair(orc, cfg)
        for it in range(updates):
            g.rollout()
            g.update(sync=False)
        assert np.isfinite(g.params()).all()
        adopt_library_state(o, g, updates)
        tol = TOL["bf16"]
        reps = []
        for inject in (False, True):
            resync(o, g)          # parameters and RMSProp state are the oracle's copies of the library's: a no-op in value
            th0 = o.theta.copy()
            ro, r1 = check_rollout(orc, o, g, tol)
            up, st, r2 = check_update(orc, o, g, tol, check_acts=True, inject=inject)
            assert st["timesteps"] == (updates + len(reps) + 1) * cfg["n_e"] * cfg["t_max"]
            if r2["flips"] == 0:
                assert r2["theta"] <= TOL_PARAMS_10 and r2["rms"] <= tol
                assert rel(g.params() - th0, o.theta - th0) <= tol
            reps.append((r1, r2))
        with capsys.disabled():
            print("\n[%s after %d free-running updates] %s" % (cfg["name"], updates,
                  [{k: float("%.3g" % v) for k, v in r2.items() if k in ("flips", "g.all", "theta", "rms", "gact0")}
                   for _, r2 in reps]))
        g.close()


def test_config3_bf16_resync_at_update_100(orc, capsys):
    _free_run_then_compare(orc, CONFIGS[2], 100, capsys)


def test_config4_bf16_resync_at_updates_100_and_199(orc, capsys):
    _free_run_then_compare(orc, CONFIGS[3], 100, capsys)
    _free_run_then_compare(orc, CONFIGS[3], 199, capsys)


def test_config5_bf16_resync_at_update_199(orc, capsys):
    _free_run_then_compare(orc, CONFIGS[4], 199, capsys)


def test_largest_batch_sampled_against_the_oracle(orc):
    """The largest rollout the library accepts (n_e * (t_max + 1) = 131,072 states: n_e = 65,536, t_max = 1, a 15 GB
    workspace) on the tensor-core path: every tensor's element offsets are close to the 32-bit range there.  The
    oracle cannot walk 65,536 environments, so it is asked for sampled ones -- the first 8 in lock step, and
    environments from the middle and the very end of the batch one state at a time (frames re-hashed from their
    integer definition, the network evaluated per state) -- and for the whole batch's returns and head gradients,
    which are cheap."""
    import torch
    n_e, T, A = 65536, 1, 18
    free, _ = torch.cuda.mem_get_info()
    if free < 24 << 30:
        pytest.skip("needs 24 GB of free device memory")
    cfg = dict(CONFIGS[4], n_e=8, t_max=T)
    o, _g = make_pair(orc, cfg)
    _g.close()
    g = pb.Paac("nature", n_e, T, A, 1, precision=pb.BF16, lr=cfg["lr"], term_denom=cfg["term_denom"])
    assert np.array_equal(g.params(), o.theta)
    ro = o.rollout()
    forced = np.full((T, n_e), -1, np.int32)
    forced[:, :8] = ro["actions"]
    g.force_actions(forced)
    g.rollout()
    tol = TOL["bf16"]
    logits = g.debug_read(pb.DBG_LOGITS).reshape(T, n_e, A)
    values = g.debug_read(pb.DBG_VALUES).reshape(T + 1, n_e)
    assert rel(logits[:, :8], ro["logits"]) <= tol and rel(values[:, :8], ro["values"]) <= tol
    acts = g.debug_read(pb.DBG_ACTIONS).reshape(T, n_e)
    terms = g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e)
    rewards = g.debug_read(pb.DBG_REWARDS).reshape(T, n_e)
    unif = g.debug_read(pb.DBG_UNIFORMS).reshape(T, n_e)
    sampled_envs = [8, 127, 128, 32767, 32768, 50001, 65407, 65408, 65534, 65535]
    # start states and the states after the step are hashes of (seed, env, step, tag); the network is per state
    frames0 = np.stack([orc.env_frame(1, e, 0, 0) for e in sampled_envs])
    nxt = g.debug_read(pb.DBG_NEXT_FRAMES).reshape(n_e, 84, 84, 4)
    fr = g.debug_read(pb.DBG_FRAMES).reshape(T, n_e, 84, 84, 4)
    acts_l, z0, v0 = orc.forward(o.net, o.theta, frames0, True)
    scale_z, scale_v = np.abs(ro["logits"]).max(), np.abs(ro["values"]).max()
    for j, e in enumerate(sampled_envs):
        assert np.array_equal(fr[0, e], frames0[j])
        assert np.abs(logits[0, e] - z0[j]).max() <= tol * scale_z and abs(values[0, e] - v0[j]) <= tol * scale_v
        assert unif[0, e] == np.float32(orc.action_uniform(1, e, 0))
        r, t = orc.env_outcome(1, e, 0, int(acts[0, e]), cfg["term_denom"])
        assert (int(rewards[0, e]), int(terms[0, e])) == (r, t)
        tag = 0 if t else int(acts[0, e]) + 1
        f1 = orc.env_frame(1, e, 1, tag)
        assert np.array_equal(nxt[e], f1)
        _, _, vb = orc.forward(o.net, o.theta, f1[None], True)
        assert abs(values[1, e] - vb[0]) <= tol * scale_v
    # the stored hidden units of the sampled states (the convolution maps of 65,536 states would be gigabytes on the host)
    h = g.debug_read(pb.DBG_ACT0 + 3).reshape(n_e, 512)
    for j, e in enumerate(sampled_envs):
        assert np.abs(h[e] - acts_l[3][j]).max() <= tol * np.abs(acts_l[3]).max()
    # the update at B = 65,536: returns, advantages and head gradients of the whole batch from the oracle, the
    # reported norm against the gradient vector, finite parameters
    st = g.update()
    assert st["status"] == 0 and st["timesteps"] == n_e * T
    R, adv = orc.returns(0.99, rewards, terms, values)
    assert rel(g.debug_read(pb.DBG_RETURNS), R) <= 1e-6 and rel(g.debug_read(pb.DBG_ADVANTAGES), adv) <= 1e-5
    dz_o, dV_o, stats_o = orc.head_grad(0.01, 1.0, logits.reshape(-1, A), values[:T].reshape(-1), acts.reshape(-1),
                                        R.reshape(-1), adv.reshape(-1))
    assert rel(g.debug_read(pb.DBG_DLOGITS), dz_o) <= 1e-4 and rel(g.debug_read(pb.DBG_DVALUES), dV_o) <= 1e-4
    assert abs(st["entropy"] - stats_o["entropy"]) <= 1e-4 and abs(st["value_loss"] - stats_o["value_loss"]) <= 1e-4
    grad = g.debug_read(pb.DBG_GRAD)
    assert abs(np.linalg.norm(grad.astype(np.float64)) - st["grad_norm"]) <= 1e-4 * st["grad_norm"]
    assert np.isfinite(g.params()).all()
    g.close()


def test_zz_flip_branch_statistics(capsys):
    """Reports how often the update check met ReLU units switched on on one side only (both valid) in this
    session, i.e. how often gradients were compared in the L2 sense instead of element by element."""
    with capsys.disabled():
        print("\n[ReLU flips] update checks from the library's own forward pass: %d, of which with flipped units: %d "
              "(most in one check: %d of %d units)" % (FLIP_STATS["calls"], FLIP_STATS["with_flips"],
                                                      FLIP_STATS["max_flips"], FLIP_STATS["units_checked"] // max(1, FLIP_STATS["calls"])))
    assert FLIP_STATS["with_flips"] <= FLIP_STATS["calls"]
