"""Parity of the CUDA library with the CPU oracle, element by element, through the C-ABI."""
import numpy as np
import pytest

from paper_1705_04862_b200 import binding as pb
from paper_1705_04862_b200.configs import CONFIGS

from parity_util import TOL, TOL_PARAMS_10, check_rollout, check_update, make_pair, rel, resync

pytestmark = pytest.mark.gpu


def test_init_is_bit_exact(orc):
    for cfg in (CONFIGS[0], CONFIGS[2]):
        o, g = make_pair(orc, cfg)
        assert np.array_equal(g.params(), o.theta)
        g.close()
    o, g = make_pair(orc, CONFIGS[0], seed=(5 << 32) | 9)
    assert np.array_equal(g.params(), o.theta)
    g.close()


def test_config1_nips_fp32_three_updates(orc):
    cfg = CONFIGS[0]
    o, g = make_pair(orc, cfg)
    for it in range(cfg["updates"]):
        ro, r1 = check_rollout(orc, o, g, TOL["fp32"])
        up, st, r2 = check_update(orc, o, g, TOL["fp32"])
        assert r1["action_mismatches"] == 0 and r2["flips"] == 0
        assert r2["theta"] <= TOL_PARAMS_10
    g.close()


def test_config2_nips_fp32_params_after_10_updates(orc):
    """Ten updates with no re-synchronisation: the float trajectories stay together."""
    cfg = CONFIGS[1]
    o, g = make_pair(orc, cfg)
    mism = 0
    for it in range(10):
        ro, r1 = check_rollout(orc, o, g, TOL["fp32"])
        up, st, r2 = check_update(orc, o, g, TOL["fp32"], check_acts=(it < 2))
        mism += r1["action_mismatches"]
    assert rel(g.params(), o.theta) <= TOL_PARAMS_10
    assert rel(g.debug_read(pb.DBG_RMS), o.m) <= TOL_PARAMS_10
    assert mism <= 1
    g.close()


@pytest.mark.parametrize("index,updates", [(0, 3), (1, 10)])
def test_float_configurations_on_the_tensor_cores(orc, index, updates):
    """The float path with every contraction on the tensor cores (operands split into two TF32 pieces, three passes,
    float accumulator): same float tolerances as the CUDA-core path, no re-synchronisation."""
    cfg = CONFIGS[index]
    o, g = make_pair(orc, cfg)
    g.set_option(pb.OPT_FP32_TENSOR_CORES, 1)
    mism = 0
    for it in range(updates):
        ro, r1 = check_rollout(orc, o, g, TOL["fp32"])
        up, st, r2 = check_update(orc, o, g, TOL["fp32"], check_acts=(it < 2))
        mism += r1["action_mismatches"]
    assert rel(g.params(), o.theta) <= TOL_PARAMS_10
    assert rel(g.debug_read(pb.DBG_RMS), o.m) <= TOL_PARAMS_10
    assert mism <= 1
    assert g.error_word() == 0
    g.close()


def test_float_tensor_core_option_on_the_nature_network(orc):
    """The three-pass kernel with bf16 storage and the larger network (CUDA-core-only mode routed through it): ragged
    batch, several tiles in every dimension; compared with the CUDA-core contractions on the same rollout."""
    outs = []
    for three_pass in (0, 1):
        g = pb.Paac("nature", 37, 3, 18, seed=5, precision=pb.BF16, lr=0.0224, term_denom=50)
        g.set_option(pb.OPT_CUDA_CORES_ONLY, 1)
        g.set_option(pb.OPT_FP32_TENSOR_CORES, three_pass)
        if outs:
            g.force_actions(outs[0]["actions"])
        g.rollout()
        acts = g.debug_read(pb.DBG_ACTIONS).copy()
        st = g.update()
        assert g.error_word() == 0
        outs.append(dict(actions=acts, sampled=g.debug_read(pb.DBG_SAMPLED).copy(),
                         logits=g.debug_read(pb.DBG_LOGITS).copy(), grad=g.debug_read(pb.DBG_GRAD).copy(),
                         norm=st["grad_norm"]))
        g.close()
    assert np.mean(outs[0]["sampled"] != outs[1]["sampled"]) <= 0.02
    assert rel(outs[0]["logits"], outs[1]["logits"]) <= TOL["bf16"]
    d = outs[0]["grad"].astype(np.float64) - outs[1]["grad"]
    assert np.linalg.norm(d) / np.linalg.norm(outs[1]["grad"]) <= TOL["bf16"]
    assert abs(outs[0]["norm"] - outs[1]["norm"]) <= TOL["bf16"] * outs[1]["norm"]


@pytest.mark.parametrize("own_stream", [False, True])
def test_config2_free_running_actions_agree(orc, own_stream):
    """Without forcing: both sides sample for themselves; with float parameters the draws agree.  On a stream
    of its own the library replays recorded CUDA graphs from the third iteration on (the legacy default stream
    cannot be captured, so there every iteration is plain launches): both must walk with the oracle."""
    import torch
    cfg = CONFIGS[1]
    stream = torch.cuda.Stream() if own_stream else torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        o, g = make_pair(orc, cfg)
        launches = []
        for it in range(7):
            before = g.launch_count()
            ro, r1 = check_rollout(orc, o, g, TOL["fp32"], lockstep=False)
            check_update(orc, o, g, TOL["fp32"], check_acts=False)
            launches.append(g.launch_count() - before)
        assert len(set(launches)) == 1            # replayed sequences count the same kernels as plain ones
        g.close()


def _bf16_iterations(orc, cfg, iters):
    """Each iteration starts from the oracle's parameters; even ones update from the library's own
    rollout, odd ones from the oracle's injected forward tensors (identical masks)."""
    o, g = make_pair(orc, cfg)
    terms = 0
    for it in range(iters):
        resync(o, g)
        th0 = o.theta.copy()
        ro, r1 = check_rollout(orc, o, g, TOL["bf16"])
        terms += int(ro["terminals"].sum())
        up, st, r2 = check_update(orc, o, g, TOL["bf16"], check_acts=(it < 2), inject=(it % 2 == 1))
        if r2["flips"] == 0:
            assert r2["theta"] <= TOL_PARAMS_10 and r2["rms"] <= TOL["bf16"]
            assert rel(g.params() - th0, o.theta - th0) <= TOL["bf16"]       # the step itself
    g.close()
    return terms


def test_config3_nature_bf16_lockstep(orc):
    _bf16_iterations(orc, CONFIGS[2], 10)


def test_config4_nature_bf16_terminals(orc):
    assert _bf16_iterations(orc, CONFIGS[3], 2) > 0          # return resets were exercised


def test_config5_full_size_first_environments(orc):
    """The throughput configuration in the launch shape the bench times (n_e = 1024): environments are
    independent and the network acts per state, so the first 16 environments of the library must walk
    exactly like a 16-environment oracle with the same seed; then one full-size update is checked
    through quantities the oracle can compute from small inputs and properties that hold at any size."""
    cfg = CONFIGS[4]
    sub = dict(cfg, n_e=16)
    o, _g = make_pair(orc, sub)
    _g.close()
    g = pb.Paac(cfg["arch"], cfg["n_e"], cfg["t_max"], cfg["n_actions"], 1, precision=pb.BF16,
                lr=cfg["lr"], term_denom=cfg["term_denom"])
    T, n_e, A, k = cfg["t_max"], cfg["n_e"], cfg["n_actions"], 16
    ro = o.rollout()
    forced = np.full((T, n_e), -1, np.int32)
    forced[:, :k] = ro["actions"]
    g.force_actions(forced)
    g.rollout()
    fr = g.debug_read(pb.DBG_FRAMES).reshape(T, n_e, -1)
    assert np.array_equal(fr[:, :k], ro["frames"][:T].reshape(T, k, -1))
    assert np.array_equal(g.debug_read(pb.DBG_NEXT_FRAMES).reshape(n_e, -1)[:k], ro["frames"][T].reshape(k, -1))
    assert np.array_equal(g.debug_read(pb.DBG_REWARDS).reshape(T, n_e)[:, :k], ro["rewards"])
    assert np.array_equal(g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e)[:, :k], ro["terminals"])
    assert np.array_equal(g.debug_read(pb.DBG_UNIFORMS).reshape(T, n_e)[:, :k], ro["uniforms"])
    logits = g.debug_read(pb.DBG_LOGITS).reshape(T, n_e, A)
    values = g.debug_read(pb.DBG_VALUES).reshape(T + 1, n_e)
    assert rel(logits[:, :k], ro["logits"]) <= TOL["bf16"] and rel(values[:, :k], ro["values"]) <= TOL["bf16"]
    sampled = g.debug_read(pb.DBG_SAMPLED).reshape(T, n_e)[:, :k]
    pg, _, _ = orc.softmax(np.ascontiguousarray(logits[:, :k]))
    for t, e in zip(*np.nonzero(sampled != ro["actions"])):
        band = 1e-5 + float(np.abs(pg[t, e] - ro["probs"][t, e]).sum())
        assert orc.cdf_margin(ro["probs"][t, e], float(ro["uniforms"][t, e])) <= band
    # every environment's frames are the hash of its own (seed, env, step, action): spot-check far ones
    acts = g.debug_read(pb.DBG_ACTIONS).reshape(T, n_e)
    terms = g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e)
    rewards = g.debug_read(pb.DBG_REWARDS).reshape(T, n_e)
    for e in (17, 500, 1023):
        for t in range(1, T):
            tag = 0 if terms[t - 1, e] else int(acts[t - 1, e]) + 1
            assert np.array_equal(fr[t, e].reshape(84, 84, 4), orc.env_frame(1, e, t, tag))
            assert (int(rewards[t, e]), int(terms[t, e])) == orc.env_outcome(1, e, t, int(acts[t, e]), cfg["term_denom"])
    # full-size update: returns, advantages and head gradients recomputed by the oracle from the small
    # tensors; row sums; the reported norm against the gradient vector
    st = g.update()
    assert st["status"] == 0 and st["timesteps"] == n_e * T and np.isfinite(st["grad_norm"])
    R, adv = orc.returns(0.99, rewards, terms, values)
    assert rel(g.debug_read(pb.DBG_RETURNS), R) <= 1e-6 and rel(g.debug_read(pb.DBG_ADVANTAGES), adv) <= 1e-5
    dz = g.debug_read(pb.DBG_DLOGITS).reshape(-1, A)
    assert np.abs(dz.sum(1)).max() <= 1e-7
    dz_o, dV_o, stats_o = orc.head_grad(0.01, 1.0, logits.reshape(-1, A), values[:T].reshape(-1), acts.reshape(-1),
                                        R.reshape(-1), adv.reshape(-1))
    assert rel(dz, dz_o) <= 1e-4 and rel(g.debug_read(pb.DBG_DVALUES), dV_o) <= 1e-4
    assert abs(st["entropy"] - stats_o["entropy"]) <= 1e-4 and abs(st["value_loss"] - stats_o["value_loss"]) <= 1e-4
    grad = g.debug_read(pb.DBG_GRAD)
    assert abs(np.linalg.norm(grad.astype(np.float64)) - st["grad_norm"]) <= 1e-4 * st["grad_norm"]
    g.close()


def test_tensor_core_path_matches_cuda_core_path(orc):
    """Two implementations of the bf16 network inside the library (tcgen05 tiles vs CUDA-core
    contractions, same rounding points) agree within the bf16 tolerance on a ragged batch."""
    outs = []
    for cores_only in (0, 1):
        g = pb.Paac("nature", 37, 3, 18, seed=5, precision=pb.BF16, lr=0.0224, term_denom=50)
        g.set_option(pb.OPT_CUDA_CORES_ONLY, cores_only)
        if outs:
            g.force_actions(outs[0]["actions"])
        g.rollout()
        acts = g.debug_read(pb.DBG_ACTIONS).copy()
        st = g.update()
        outs.append(dict(actions=acts, sampled=g.debug_read(pb.DBG_SAMPLED).copy(),
                         logits=g.debug_read(pb.DBG_LOGITS).copy(), grad=g.debug_read(pb.DBG_GRAD).copy(),
                         norm=st["grad_norm"]))
        g.close()
    assert np.mean(outs[0]["sampled"] != outs[1]["sampled"]) <= 0.02
    assert rel(outs[0]["logits"], outs[1]["logits"]) <= TOL["bf16"]
    d = outs[0]["grad"].astype(np.float64) - outs[1]["grad"]
    assert np.linalg.norm(d) / np.linalg.norm(outs[1]["grad"]) <= TOL["bf16"]
    assert abs(outs[0]["norm"] - outs[1]["norm"]) <= TOL["bf16"] * outs[1]["norm"]


def test_ragged_sizes_and_action_counts(orc):
    """n_e that is no multiple of any tile (below one tile, and one full 128-row tile plus a ragged tail on the
    tensor-core path), every action-set size of the configs, the largest action set the cluster kernel of the fully
    connected layer takes (31) and the one beyond it (32, which goes through the split-k kernel)."""
    for arch, prec, n_e, t_max, A in (("nips", "fp32", 5, 3, 18), ("nips", "bf16", 3, 2, 4),
                                      ("nature", "fp32", 7, 2, 6), ("nature", "bf16", 13, 1, 2),
                                      ("nips", "fp32", 1, 1, 32), ("nature", "bf16", 133, 2, 31),
                                      ("nature", "bf16", 130, 1, 32)):
        cfg = dict(arch=arch, precision=prec, n_e=n_e, t_max=t_max, n_actions=A, lr=0.01, term_denom=3)
        o, g = make_pair(orc, cfg, seed=77)
        for it in range(2):
            resync(o, g)
            check_rollout(orc, o, g, TOL[prec])
            check_update(orc, o, g, TOL[prec], inject=(it == 1))
        g.close()


def test_resync_after_many_updates(orc):
    """Free-run the library for 60 updates (config 2), copy its parameters and RMSProp state into
    the oracle and compare one more iteration from there."""
    import torch
    cfg = CONFIGS[1]
    torch.cuda.set_stream(torch.cuda.Stream())      # own stream: the 60 free-running updates replay CUDA graphs
    o, g = make_pair(orc, cfg)
    for it in range(60):
        g.rollout()
        st = g.update()
        assert st["status"] == 0 and np.isfinite(st["grad_norm"])
    o.theta = g.params()
    o.m = g.debug_read(pb.DBG_RMS).copy()
    o.N = 60 * cfg["n_e"] * cfg["t_max"]
    o.state = g.debug_read(pb.DBG_NEXT_FRAMES).reshape(cfg["n_e"], 84, 84, 4).copy()
    for j, c in enumerate(g.debug_read(pb.DBG_COUNTERS).reshape(3, -1)):
        o.counters[j][:] = c
    check_rollout(orc, o, g, TOL["fp32"])
    check_update(orc, o, g, TOL["fp32"], check_acts=False)
    g.close()
    torch.cuda.set_stream(torch.cuda.default_stream())


def test_determinism_bitwise(orc):
    """Same seed, same bits -- with plain launches and with replayed graphs (own stream), tensor-core path."""
    import torch
    cfg = CONFIGS[2]
    outs = []
    for rep in range(3):
        stream = torch.cuda.Stream() if rep == 2 else torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            _, g = make_pair(orc, cfg)
            for it in range(5):
                g.rollout()
                g.update()
            outs.append((g.params(), g.debug_read(pb.DBG_GRAD).copy()))
            g.close()
    for k in (1, 2):
        assert np.array_equal(outs[0][0], outs[k][0]) and np.array_equal(outs[0][1], outs[k][1])


def test_error_paths(orc):
    import ctypes as C
    L = pb.lib()
    hp = pb.default_hparams()
    h = C.c_void_p()
    assert L.paac_init(C.byref(h), 7, 4, 5, 4, C.byref(hp), 1) == pb.ERR_ARG
    assert L.paac_init(C.byref(h), 0, 0, 5, 4, C.byref(hp), 1) == pb.ERR_ARG
    assert L.paac_init(C.byref(h), 0, 4, 5, 1, C.byref(hp), 1) == pb.ERR_ARG
    assert L.paac_init(None, 0, 4, 5, 4, C.byref(hp), 1) == pb.ERR_ARG
    assert L.paac_rollout(None, None) == pb.ERR_ARG
    import torch
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    hp2 = pb.default_hparams(workspace=small.data_ptr(), workspace_bytes=1024)
    assert L.paac_init(C.byref(h), 0, 4, 5, 4, C.byref(hp2), 1) == pb.ERR_WORKSPACE
    g = pb.Paac("nips", 4, 2, 4, 3)
    assert L.paac_update(g._h, None) == pb.ERR_STATE          # no rollout yet
    buf = np.zeros(3, np.float32)
    assert L.paac_params(g._h, buf.ctypes.data, 3) == pb.ERR_ARG
    bad = np.full(g.B, 9, np.int32)
    assert L.paac_force_actions(g._h, bad.ctypes.data) == pb.ERR_ARG
    # a NaN parameter makes the gradient norm non-finite: the update is skipped and says so
    th = g.params()
    th_bad = th.copy()
    th_bad[-1] = np.nan          # value-head bias: V, hence the loss gradient, becomes NaN
    g.set_params(th_bad)
    g.rollout()
    rms0 = g.debug_read(pb.DBG_RMS).copy()
    st = g.update()
    assert st["status"] == pb.ERR_NONFINITE
    assert np.array_equal(g.debug_read(pb.DBG_RMS), rms0)
    after = g.params()
    assert np.array_equal(after[np.isfinite(th_bad)], th_bad[np.isfinite(th_bad)])
    g.set_params(th)
    g.rollout()
    assert g.update()["status"] == 0
    g.close()


def test_external_environment_mode_matches_device_environment(orc):
    """Frames, rewards and terminals fed from the host (the oracle's environment) give the same
    actions, values and update as the on-device environment; in the second iteration step 0 is not
    sent again (it is the bootstrap state of the first, already on the device)."""
    cfg = CONFIGS[0]
    o, g = make_pair(orc, cfg)
    _, g2 = make_pair(orc, cfg)
    n_e, T = cfg["n_e"], cfg["t_max"]
    a = np.zeros(n_e, np.int32)
    with pytest.raises(pb.PaacError):
        g2.act_host(0, None, a)                   # nothing on the device yet
    for it in range(2):
        g.rollout()
        g.update()
        # replay the same iteration on g2 through the host entry points
        frames = g.debug_read(pb.DBG_FRAMES).reshape(T, n_e, 84, 84, 4)
        nxt = g.debug_read(pb.DBG_NEXT_FRAMES).reshape(n_e, 84, 84, 4)
        rewards = g.debug_read(pb.DBG_REWARDS).reshape(T, n_e)
        terms = g.debug_read(pb.DBG_TERMINALS).reshape(T, n_e)
        acts_dev = g.debug_read(pb.DBG_ACTIONS).reshape(T, n_e)
        vals_dev = g.debug_read(pb.DBG_VALUES).reshape(T + 1, n_e)
        for t in range(T):
            v = np.zeros(n_e, np.float32)
            g2.act_host(t, None if (it == 1 and t == 0) else np.ascontiguousarray(frames[t]), a, v)
            assert np.array_equal(a, acts_dev[t]) and np.array_equal(v, vals_dev[t])
            if t == 0:
                with pytest.raises(pb.PaacError):
                    g2.act_host(1, None, a)       # only step 0 can be taken from the device
            g2.observe_host(t, np.ascontiguousarray(rewards[t]), np.ascontiguousarray(terms[t]))
        vb = np.zeros(n_e, np.float32)
        g2.act_host(T, np.ascontiguousarray(nxt), None, vb)
        assert np.array_equal(vb, vals_dev[T])
        g2.update()
        assert np.array_equal(g2.params(), g.params())
        assert np.array_equal(g2.debug_read(pb.DBG_FRAMES), g.debug_read(pb.DBG_FRAMES))
    g.close()
    g2.close()


def test_external_environment_mode_with_newest_frames(orc):
    """paac_act_host_newest: the host sends only the frame that joins the four-frame stack (and restart flags); the
    states built on the device are the oracle's stack of the same planes, and the iteration (actions, values,
    update) is the one a context gets that is sent those whole states."""
    cfg = CONFIGS[0]
    n_e, T = cfg["n_e"], cfg["t_max"]
    _, g = make_pair(orc, cfg)
    _, g2 = make_pair(orc, cfg)
    rng = np.random.RandomState(5)
    state = rng.randint(0, 256, (n_e, 84, 84, 4), dtype=np.uint8)
    a, a2 = np.zeros(n_e, np.int32), np.zeros(n_e, np.int32)
    v, v2 = np.zeros(n_e, np.float32), np.zeros(n_e, np.float32)
    with pytest.raises(pb.PaacError):
        g.act_host_newest(0, state[..., 3].copy(), None, a, v)             # step 0 has no new frame
    for it in range(2):
        for t in range(T + 1):
            if t == 0:
                g.act_host(0, state if it == 0 else None, a, v)               # whole state once, then the one on the device
                g2.act_host(0, state, a2, v2)
            else:
                plane = rng.randint(0, 256, (n_e, 84, 84), dtype=np.uint8)
                restart = (rng.randint(0, 3, n_e) == 0).astype(np.uint8) if t % 2 else None
                state = orc.stack_push(state, plane, restart)
                g.act_host_newest(t, plane, restart, a if t < T else None, v)
                g2.act_host(t, state, a2 if t < T else None, v2)
            assert np.array_equal(v, v2)
            if t < T:
                assert np.array_equal(a, a2)
                r = rng.randint(-1, 2, n_e).astype(np.int8)
                term = (rng.randint(0, 5, n_e) == 0).astype(np.uint8)
                g.observe_host(t, r, term)
                g2.observe_host(t, r, term)
        assert np.array_equal(g.debug_read(pb.DBG_FRAMES), g2.debug_read(pb.DBG_FRAMES))
        assert np.array_equal(g.debug_read(pb.DBG_NEXT_FRAMES).reshape(n_e, 84, 84, 4), state)
        g.update()
        g2.update()
        assert np.array_equal(g.params(), g2.params())
    g.close()
    g2.close()


def test_bounded_wait_gives_up_and_the_update_is_skipped(orc):
    """A wait on a barrier nobody signals runs out after its poll limit: the kernel returns, the error word is set,
    the call reports ERR_TIMEOUT, and the context stays usable.  While the word is set an update changes neither
    parameters nor RMSProp state and says why; after it is cleared the learner carries on."""
    g = pb.Paac("nature", 8, 2, 6, seed=3, precision=pb.BF16, lr=0.01, term_denom=50)
    g.rollout()
    assert g.update()["status"] == 0 and g.error_word() == 0
    theta0, rms0 = g.params(), g.debug_read(pb.DBG_RMS).copy()
    assert g.wait_probe(0) == pb.ERR_ARG
    assert g.wait_probe(20000) == pb.ERR_TIMEOUT
    assert g.error_word() == 1
    g.rollout()
    st = g.update()
    assert st["status"] == pb.ERR_TIMEOUT and st["clip_scale"] == 0.0
    g.clear_error_word()
    assert np.array_equal(g.params(), theta0) and np.array_equal(g.debug_read(pb.DBG_RMS), rms0)
    with pytest.raises(pb.PaacError):       # out of order: the skipped update consumed the rollout
        g.update()
    g.rollout()
    assert g.update()["status"] == 0
    assert not np.array_equal(g.params(), theta0)
    g.close()


def test_first_layer_weight_domain(orc):
    """The fp16 image of the first layer holds |bf16(w)| <= 255: the largest such weight gives the oracle's logits,
    anything beyond is refused and nothing changes; tiny weights (below 2^-25) only lose bits far below the tolerance."""
    cfg = dict(arch="nature", precision="bf16", n_e=6, t_max=1, n_actions=4, lr=0.01, term_denom=50)
    o, g = make_pair(orc, cfg, seed=11)
    th = o.theta.copy()
    th[:64] = 0.0
    th[3] = 255.0            # largest magnitude the image holds
    th[7] = -255.0
    th[10] = 1e-9            # far below 2^-25
    th[11] = 2.0 ** -25
    o.theta = th
    g.set_params(th)
    check_rollout(orc, o, g, TOL["bf16"])
    bad = th.copy()
    bad[5] = 256.0
    import ctypes as C
    assert pb.lib().paac_set_params(g._h, bad.ctypes.data, bad.size) == pb.ERR_RANGE
    bad[5] = np.inf
    assert pb.lib().paac_set_params(g._h, bad.ctypes.data, bad.size) == pb.ERR_RANGE
    assert np.array_equal(g.params(), th) and g.error_word() == 0
    # the other layers have no such limit
    ok = th.copy()
    ok[9000] = 300.0
    g.set_params(ok)
    g.close()


def test_partial_tensor_core_weight_gradient_mask(orc):
    """Layers whose weight gradient is taken off the tensor cores (option TC_WGRAD_LAYERS) give the same gradient
    within the bf16 tolerance as the all-tensor-core update."""
    grads = []
    for mask in (0xF, 0b0101):
        g = pb.Paac("nature", 21, 2, 6, seed=9, precision=pb.BF16, lr=0.01, term_denom=50)
        g.set_option(pb.OPT_TC_WGRAD_LAYERS, mask)
        if grads:
            g.force_actions(grads[0][1])
        g.rollout()
        acts = g.debug_read(pb.DBG_ACTIONS).copy()
        st = g.update()
        assert st["status"] == 0
        grads.append((g.debug_read(pb.DBG_GRAD).copy(), acts, st["grad_norm"]))
        g.close()
    assert rel(grads[0][0], grads[1][0]) <= TOL["bf16"]
    assert abs(grads[0][2] - grads[1][2]) <= TOL["bf16"] * grads[0][2]


def test_shape_sweep_two_implementations_agree():
    """Forty ragged shapes (environments 1 .. 1025, steps 1 .. 13, actions 2 .. 32, seeded choice) through the bf16
    network: the tensor-core path and the CUDA-core path of the library finish without a device error and agree on
    the gradient within the bf16 tolerance (L2).  No oracle here: the point is every shape-dependent offset, split
    count and tail."""
    import random
    rnd = random.Random(3)
    combos = [(n, t, a) for n in (1, 2, 3, 5, 16, 37, 64, 100, 129, 255) for t in (1, 2, 3, 5, 7)
              for a in (2, 3, 4, 5, 7, 18, 19, 20, 31, 32)]
    rnd.shuffle(combos)
    combos = combos[:36] + [(1000, 13, 19), (1023, 5, 32), (1025, 1, 3), (511, 5, 18)]
    for n_e, T, A in combos:
        outs = []
        for cores_only in (0, 1):
            g = pb.Paac("nature", n_e, T, A, seed=5, precision=pb.BF16, lr=0.0224, term_denom=50)
            g.set_option(pb.OPT_CUDA_CORES_ONLY, cores_only)
            if outs:
                g.force_actions(outs[0][0])
            g.rollout()
            acts = g.debug_read(pb.DBG_ACTIONS).copy()
            g.update()
            grad = g.debug_read(pb.DBG_GRAD).copy()
            assert g.error_word() == 0 and np.isfinite(grad).all(), (n_e, T, A)
            outs.append((acts, grad))
            g.close()
        d = np.linalg.norm(outs[0][1].astype(np.float64) - outs[1][1]) / max(np.linalg.norm(outs[1][1]), 1e-30)
        assert d <= 5e-2, (n_e, T, A, d)


def test_shape_sweep_float_path_two_implementations_agree():
    """Thirty ragged shapes through the float path, both networks, with the value-based variant and the learnable
    environment mixed in: the CUDA-core contraction (whose tile shape follows the row and column counts) and the
    three-pass tensor-core contraction finish without a device error and agree on the gradient (L2; single ReLU
    flips between two float implementations show up at the 1e-3 level on large batches)."""
    import random
    rnd = random.Random(7)
    combos = [(arch, n, t, a) for arch in ("nips", "nature") for n in (1, 2, 3, 5, 16, 37, 64, 100, 129, 255)
              for t in (1, 2, 5, 7) for a in (2, 3, 5, 18, 19, 32)]
    rnd.shuffle(combos)
    for i, (arch, n_e, T, A) in enumerate(combos[:30]):
        outs = []
        for mode in (0, 1):
            g = pb.Paac(arch, n_e, T, A, seed=5, precision=pb.FP32, lr=0.01, term_denom=50,
                        algorithm=pb.ALGO_NSTEP_Q if i % 3 == 0 else pb.ALGO_A2C,
                        environment=pb.ENV_PATTERN if i % 4 == 0 else pb.ENV_HASHED)
            g.set_option(pb.OPT_FP32_TENSOR_CORES, mode)
            if outs:
                g.force_actions(outs[0][0])
            g.rollout()
            acts = g.debug_read(pb.DBG_ACTIONS).copy()
            g.update()
            grad = g.debug_read(pb.DBG_GRAD).copy()
            assert g.error_word() == 0 and np.isfinite(grad).all(), (arch, n_e, T, A)
            outs.append((acts, grad))
            g.close()
        d = np.linalg.norm(outs[0][1].astype(np.float64) - outs[1][1]) / max(np.linalg.norm(outs[1][1]), 1e-30)
        assert d <= 2e-2, (arch, n_e, T, A, d)


def test_odd_action_counts_on_the_tensor_core_path(orc):
    """Action counts and batch sizes whose product is odd: the heads' partial sums (policy rows, policy biases, value
    row, value bias, one behind the other per split) then start at odd float offsets unless padded; the value row is
    stored in pairs.  (n_e * t_max <= 148 rows gives one split per row.)"""
    for n_e, t_max, A in ((37, 5, 5), (33, 3, 19), (41, 1, 7)):
        cfg = dict(CONFIGS[2], n_e=n_e, t_max=t_max, n_actions=A)
        o, g = make_pair(orc, cfg)
        check_rollout(orc, o, g, TOL["bf16"])
        check_update(orc, o, g, TOL["bf16"])
        assert g.error_word() == 0
        g.close()


def test_update_in_groups_of_states_matches_the_default(orc):
    """PAAC_OPT_UPDATE_CHUNKS: the second layer's data gradient and the first layer's weight gradient alternating over
    2, 3 or 4 groups of states give the default's gradient up to the grouping of the partial sums; against the oracle
    the usual bf16 tolerances hold."""
    cfg = dict(CONFIGS[2], n_e=37, n_actions=5)
    grads = []
    for chunks in (1, 2, 3, 4):
        o, g = make_pair(orc, cfg)
        g.set_option(pb.OPT_UPDATE_CHUNKS, chunks)
        check_rollout(orc, o, g, TOL["bf16"])
        check_update(orc, o, g, TOL["bf16"])
        assert g.error_word() == 0
        grads.append(g.debug_read(pb.DBG_GRAD).copy())
        if chunks == 1:
            for bad in (0, 5):
                with pytest.raises(pb.PaacError):
                    g.set_option(pb.OPT_UPDATE_CHUNKS, bad)
        g.close()
    for gr in grads[1:]:
        assert np.abs(gr - grads[0]).max() <= 1e-5 * np.abs(grads[0]).max()


@pytest.mark.parametrize("base,iters", [(0, 3), (2, 4)])
def test_value_based_variant_matches_the_oracle(orc, base, iters):
    """n-step Q-learning on the same framework (Section 2.2, Eqs. 2-4; Section 3), configurations 1 (float, CUDA
    cores) and 3 (bf16, tensor cores): epsilon-greedy actions from the shared uniforms, Q(s_t, a_t) as the stored
    value, max_a Q as the bootstrap, the Q-loss gradient, and the update, all against the oracle's variant."""
    cfg = dict(CONFIGS[base], algorithm="nstep_q", epsilon=0.25)
    prec = cfg["precision"]
    o, g = make_pair(orc, cfg)
    explored = 0
    for it in range(iters):
        if prec == "bf16":
            resync(o, g)
        ro, r1 = check_rollout(orc, o, g, TOL[prec])
        explored += int((ro["uniforms"] < 0.25).sum())
        # the stored values are the taken actions' Q-values, the last row the greedy value of the final states
        T, n_e = cfg["t_max"], cfg["n_e"]
        vals = g.debug_read(pb.DBG_VALUES).reshape(T + 1, n_e)
        lg = g.debug_read(pb.DBG_LOGITS).reshape(T, n_e, -1)
        acts = g.debug_read(pb.DBG_ACTIONS).reshape(T, n_e)
        assert np.array_equal(vals[:T], np.take_along_axis(lg, acts[..., None], 2)[..., 0])
        up, st, r2 = check_update(orc, o, g, TOL[prec], inject=(prec == "bf16" and it % 2 == 1))
        assert st["policy_loss"] == 0.0 and st["entropy"] == 0.0
        dz = g.debug_read(pb.DBG_DLOGITS).reshape(T * n_e, -1)
        assert np.count_nonzero(dz) <= T * n_e and np.all(g.debug_read(pb.DBG_DVALUES) == 0)
        if r2["flips"] == 0:
            assert r2["theta"] <= TOL_PARAMS_10
    assert explored > 0
    g.close()


def test_value_based_variant_bad_hyperparameters():
    import ctypes as C
    h = C.c_void_p()
    for bad in (dict(algorithm=2), dict(algorithm=pb.ALGO_NSTEP_Q, epsilon=1.5), dict(algorithm=pb.ALGO_NSTEP_Q, epsilon=-0.1)):
        hp = pb.default_hparams(**bad)
        assert pb.lib().paac_init(C.byref(h), 0, 4, 5, 4, C.byref(hp), 1) == pb.ERR_ARG


def test_pattern_environment_matches_the_oracle_and_can_be_learned(orc):
    """The learnable environment (a bright band of rows names the rewarded action): bit-exact frames and rewards in
    lock step with the oracle on both network paths, and a learner on it collects clearly more reward after some
    hundred updates than at the start (chance level is 1 / A)."""
    import torch
    for base in (0, 2):
        cfg = dict(CONFIGS[base], environment="pattern", term_denom=50)
        o, g = make_pair(orc, cfg)
        for it in range(2):
            if cfg["precision"] == "bf16":
                resync(o, g)
            ro, _ = check_rollout(orc, o, g, TOL[cfg["precision"]])
            assert set(np.unique(ro["rewards"])) <= {0, 1}
            check_update(orc, o, g, TOL[cfg["precision"]], inject=(cfg["precision"] == "bf16"))
        g.close()
    with torch.cuda.stream(torch.cuda.Stream()):
        # a contextual bandit: gamma = 0 makes the one-step return the exact target (see bench.py --lr-sweep)
        g = pb.Paac("nature", 16, 5, 6, seed=1, precision=pb.BF16, lr=0.0007 * 16, term_denom=200, gamma=0.0,
                    environment=pb.ENV_PATTERN)
        def mean_reward(iters):
            tot = 0.0
            for _ in range(iters):
                g.rollout()
                tot += float(g.debug_read(pb.DBG_REWARDS).astype(np.float64).mean())
                assert g.update()["status"] == 0
            return tot / iters
        first = mean_reward(20)
        for _ in range(400):
            g.rollout()
            g.update(sync=False)
        last = mean_reward(20)
        assert last > 0.8 and last > first + 0.2, (first, last)
        g.close()
