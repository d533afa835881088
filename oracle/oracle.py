"""Python face of the PAAC oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Loads ``libpaac_oracle.so`` (plain C, built from ``paac_oracle.c`` beside this
file) and strings its steps together in the order of Algorithm 1 of the paper:
roll all environments forward ``t_max`` steps with actions sampled from the
current policy, bootstrap, form n-step returns and advantages, take one batched
gradient step with global-norm clipping and RMSProp.

Only tests, the smoke check and the bench's CPU-baseline leg may import this
module.  It imports nothing from the CUDA package.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "paac_oracle.c")
_LIB = os.path.join(_HERE, "libpaac_oracle.so")
MAX_CONV = 4


def build(force=False):
    """Compile the oracle with gcc (OpenMP over independent states only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class Net(C.Structure):
    _fields_ = [("in_h", C.c_int), ("in_w", C.c_int), ("in_c", C.c_int), ("n_conv", C.c_int),
                ("cout", C.c_int * MAX_CONV), ("k", C.c_int * MAX_CONV), ("stride", C.c_int * MAX_CONV),
                ("fc", C.c_int), ("n_actions", C.c_int)]


def make_net(in_hwc, convs, fc, n_actions):
    """convs: list of (cout, k, stride)."""
    n = Net()
    n.in_h, n.in_w, n.in_c = in_hwc
    n.n_conv = len(convs)
    for i, (co, k, s) in enumerate(convs):
        n.cout[i], n.k[i], n.stride[i] = co, k, s
    n.fc, n.n_actions = fc, n_actions
    return n


def arch_net(arch, n_actions):
    """The two networks of Section 5.1 with the layer sizes of the papers it cites."""
    if arch == "nips":
        return make_net((84, 84, 4), [(16, 8, 4), (32, 4, 2)], 256, n_actions)
    if arch == "nature":
        return make_net((84, 84, 4), [(32, 8, 4), (64, 4, 2), (64, 3, 1)], 512, n_actions)
    raise ValueError(arch)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_param_count.restype = C.c_size_t
        L.orc_param_count.argtypes = [C.POINTER(Net)]
        L.orc_act_size.restype = C.c_size_t
        L.orc_act_size.argtypes = [C.POINTER(Net), C.c_int]
        L.orc_bf16_round.restype = C.c_float
        L.orc_bf16_round.argtypes = [C.c_float]
        L.orc_action_uniform.restype = C.c_float
        L.orc_action_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        L.orc_sample.restype = C.c_int32
        L.orc_cdf_margin.restype = C.c_float
        L.orc_loss_double.restype = C.c_double
        L.orc_clip_rmsprop.restype = C.c_int
        L.orc_q_greedy.restype = C.c_int32
        L.orc_q_select.restype = C.c_int32
        L.orc_q_margin.restype = C.c_float
        _lib = L
    return _lib


def _p(a, t=C.c_void_p):
    return a.ctypes.data_as(t)


def param_count(net):
    return int(lib().orc_param_count(C.byref(net)))


def act_sizes(net):
    return [int(lib().orc_act_size(C.byref(net), l)) for l in range(net.n_conv + 1)]


def act_shapes(net):
    shapes, h, w = [], net.in_h, net.in_w
    for l in range(net.n_conv):
        h = (h - net.k[l]) // net.stride[l] + 1
        w = (w - net.k[l]) // net.stride[l] + 1
        shapes.append((h, w, net.cout[l]))
    shapes.append((net.fc,))
    return shapes


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return list(o)


def bf16_round(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty_like(x)
    f = lib().orc_bf16_round
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def action_uniform(seed, env, step):
    return float(lib().orc_action_uniform(C.c_uint64(seed), C.c_uint32(env), C.c_uint64(step)))


def init_params(net, seed):
    theta = np.zeros(param_count(net), np.float32)
    lib().orc_init_params(C.byref(net), C.c_uint64(seed), _p(theta))
    return theta


def env_frame(seed, env, step, tag, h=84, w=84):
    f = np.zeros((h, w, 4), np.uint8)
    lib().orc_env_frame(C.c_uint64(seed), C.c_uint32(env), C.c_uint32(step), C.c_uint32(tag), h, w, _p(f))
    return f


def env_outcome(seed, env, step, action, term_denom):
    r, t = C.c_int8(), C.c_uint8()
    lib().orc_env_outcome(C.c_uint64(seed), C.c_uint32(env), C.c_uint32(step), C.c_int32(action),
                          C.c_uint32(term_denom), C.byref(r), C.byref(t))
    return r.value, t.value


def env_reset(seed, n_e, h=84, w=84):
    f = np.zeros((n_e, h, w, 4), np.uint8)
    lib().orc_env_reset(C.c_uint64(seed), n_e, h, w, _p(f))
    return f


def env_step(seed, step, actions, term_denom, counters, h=84, w=84):
    """counters = (ep_len, ep_return, episodes) int32 arrays, updated in place."""
    n_e = actions.shape[0]
    actions = np.ascontiguousarray(actions, np.int32)
    f = np.zeros((n_e, h, w, 4), np.uint8)
    r = np.zeros(n_e, np.int8)
    t = np.zeros(n_e, np.uint8)
    lib().orc_env_step(C.c_uint64(seed), n_e, C.c_uint32(step), _p(actions), C.c_uint32(term_denom), h, w,
                       _p(f), _p(r), _p(t), _p(counters[0]), _p(counters[1]), _p(counters[2]))
    return f, r, t


def preprocess(raw_prev, raw_last, state_in=None):
    """Section 5.1 pre-processing: raw uint8 [n, 210, 160, 3] x 2 (+ previous state [n, 84, 84, 4]) -> state."""
    raw_prev = np.ascontiguousarray(raw_prev, np.uint8)
    raw_last = np.ascontiguousarray(raw_last, np.uint8)
    n = raw_prev.shape[0]
    assert raw_prev.shape == (n, 210, 160, 3) and raw_last.shape == raw_prev.shape
    out = np.zeros((n, 84, 84, 4), np.uint8)
    sin = None
    if state_in is not None:
        state_in = np.ascontiguousarray(state_in, np.uint8)
        assert state_in.shape == out.shape
        sin = _p(state_in)
    lib().orc_preprocess(_p(raw_prev), _p(raw_last), sin, _p(out), n)
    return out


def stack_push(state_in, newest, restart=None):
    """Section 5.1 frame stack: state [n, 84, 84, 4] + newest frame [n, 84, 84] (+ restart flags [n]) -> state."""
    state_in = np.ascontiguousarray(state_in, np.uint8)
    newest = np.ascontiguousarray(newest, np.uint8)
    n = state_in.shape[0]
    assert state_in.shape == (n, 84, 84, 4) and newest.shape == (n, 84, 84)
    out = np.zeros_like(state_in)
    rs = None
    if restart is not None:
        restart = np.ascontiguousarray(restart, np.uint8)
        assert restart.shape == (n,)
        rs = _p(restart)
    lib().orc_stack_push(_p(state_in), _p(newest), rs, _p(out), n)
    return out


def pattern_goal(seed, env, step, n_actions):
    lib().orc_pattern_goal.restype = C.c_uint32
    return int(lib().orc_pattern_goal(C.c_uint64(seed), C.c_uint32(env), C.c_uint32(step), n_actions))


def pattern_frame(seed, env, step, tag, n_actions, h=84, w=84):
    f = np.zeros((h, w, 4), np.uint8)
    lib().orc_pattern_frame(C.c_uint64(seed), C.c_uint32(env), C.c_uint32(step), C.c_uint32(tag), n_actions, h, w, _p(f))
    return f


def pattern_reset(seed, n_e, n_actions, h=84, w=84):
    f = np.zeros((n_e, h, w, 4), np.uint8)
    lib().orc_pattern_reset(C.c_uint64(seed), n_e, n_actions, h, w, _p(f))
    return f


def pattern_step(seed, step, actions, term_denom, n_actions, counters, h=84, w=84):
    n_e = actions.shape[0]
    actions = np.ascontiguousarray(actions, np.int32)
    f = np.zeros((n_e, h, w, 4), np.uint8)
    r = np.zeros(n_e, np.int8)
    t = np.zeros(n_e, np.uint8)
    lib().orc_pattern_step(C.c_uint64(seed), n_e, C.c_uint32(step), _p(actions), C.c_uint32(term_denom), n_actions, h, w,
                           _p(f), _p(r), _p(t), _p(counters[0]), _p(counters[1]), _p(counters[2]))
    return f, r, t


def _ptr_array(arrs):
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def forward(net, theta, frames, bf16=False):
    """frames uint8 [n, H, W, C] -> (acts list, logits [n, A], values [n])."""
    frames = np.ascontiguousarray(frames, np.uint8)
    n = frames.shape[0]
    acts = [np.zeros((n,) + s, np.float32) for s in act_shapes(net)]
    logits = np.zeros((n, net.n_actions), np.float32)
    values = np.zeros(n, np.float32)
    lib().orc_forward(C.byref(net), _p(theta), int(bf16), _p(frames), n, _ptr_array(acts), _p(logits), _p(values))
    return acts, logits, values


def softmax(z):
    z = np.ascontiguousarray(z, np.float32)
    A = z.shape[-1]
    zz = z.reshape(-1, A)
    p = np.zeros_like(zz)
    lp = np.zeros_like(zz)
    H = np.zeros(zz.shape[0], np.float32)
    for i in range(zz.shape[0]):
        h = C.c_float()
        lib().orc_softmax(_p(zz[i]), A, _p(p[i]), _p(lp[i]), C.byref(h))
        H[i] = h.value
    return p.reshape(z.shape), lp.reshape(z.shape), H.reshape(z.shape[:-1])


def sample(p, u):
    p = np.ascontiguousarray(p, np.float32)
    return int(lib().orc_sample(_p(p), p.shape[0], C.c_float(u)))


def cdf_margin(p, u):
    p = np.ascontiguousarray(p, np.float32)
    return float(lib().orc_cdf_margin(_p(p), p.shape[0], C.c_float(u)))


def returns(gamma, rewards, terminals, values):
    """rewards int8 [t_max, n_e], terminals uint8 [t_max, n_e], values float [t_max+1, n_e]."""
    t_max, n_e = rewards.shape
    rewards = np.ascontiguousarray(rewards, np.int8)
    terminals = np.ascontiguousarray(terminals, np.uint8)
    values = np.ascontiguousarray(values, np.float32)
    R = np.zeros((t_max, n_e), np.float32)
    adv = np.zeros((t_max, n_e), np.float32)
    lib().orc_returns(n_e, t_max, C.c_float(gamma), _p(rewards), _p(terminals), _p(values), _p(R), _p(adv))
    return R, adv


def head_grad(beta, value_coef, logits, values, actions, R, adv):
    logits = np.ascontiguousarray(logits, np.float32)
    B, A = logits.shape
    values = np.ascontiguousarray(values, np.float32).reshape(B)
    actions = np.ascontiguousarray(actions, np.int32).reshape(B)
    R = np.ascontiguousarray(R, np.float32).reshape(B)
    adv = np.ascontiguousarray(adv, np.float32).reshape(B)
    dz = np.zeros((B, A), np.float32)
    dV = np.zeros(B, np.float32)
    stats = (C.c_double * 3)()
    lib().orc_head_grad(B, A, C.c_float(beta), C.c_float(value_coef), _p(logits), _p(values), _p(actions),
                        _p(R), _p(adv), _p(dz), _p(dV), stats)
    return dz, dV, dict(policy_loss=stats[0], value_loss=stats[1], entropy=stats[2])


def q_greedy(q):
    q = np.ascontiguousarray(q, np.float32)
    return int(lib().orc_q_greedy(_p(q), q.shape[0]))


def q_select(q, u, eps):
    """Epsilon-greedy action from Q-values [A] and one uniform (Section 3: the policy may be implicit)."""
    q = np.ascontiguousarray(q, np.float32)
    return int(lib().orc_q_select(_p(q), q.shape[0], C.c_float(u), C.c_float(eps)))


def q_margin(q):
    q = np.ascontiguousarray(q, np.float32)
    return float(lib().orc_q_margin(_p(q), q.shape[0]))


def q_head_grad(value_coef, q, actions, R):
    """Gradient of the n-step Q loss (Eqs. 3-4) at the Q-values [B, A] -> (dq, stats)."""
    q = np.ascontiguousarray(q, np.float32)
    B, A = q.shape
    actions = np.ascontiguousarray(actions, np.int32).reshape(B)
    R = np.ascontiguousarray(R, np.float32).reshape(B)
    dq = np.zeros((B, A), np.float32)
    stats = (C.c_double * 2)()
    lib().orc_q_head_grad(B, A, C.c_float(value_coef), _p(q), _p(actions), _p(R), _p(dq), stats)
    return dq, dict(value_loss=stats[0], mean_max_q=stats[1])


def loss_double(net, theta64, frames, beta, value_coef, actions, R, adv):
    theta64 = np.ascontiguousarray(theta64, np.float64)
    frames = np.ascontiguousarray(frames, np.uint8)
    n = frames.shape[0]
    actions = np.ascontiguousarray(actions, np.int32)
    R = np.ascontiguousarray(R, np.float32)
    adv = np.ascontiguousarray(adv, np.float32)
    return float(lib().orc_loss_double(C.byref(net), _p(theta64), _p(frames), n, C.c_float(beta),
                                       C.c_float(value_coef), _p(actions), _p(R), _p(adv)))


def backward(net, theta, frames, acts, dz, dV, bf16=False):
    """-> (grad [P], gacts list: gradient w.r.t. each layer's pre-activation)."""
    frames = np.ascontiguousarray(frames, np.uint8)
    n = frames.shape[0]
    grad = np.zeros(param_count(net), np.float32)
    gacts = [np.zeros_like(a) for a in acts]
    dz = np.ascontiguousarray(dz, np.float32)
    dV = np.ascontiguousarray(dV, np.float32)
    lib().orc_backward(C.byref(net), _p(theta), int(bf16), _p(frames), n, _ptr_array(acts), _p(dz), _p(dV),
                       _p(grad), _ptr_array(gacts))
    return grad, gacts


def clip_rmsprop(theta, m, grad, lr, rho, eps, clip):
    """In place on theta and m. -> (status, norm, scale)."""
    norm, scale = C.c_double(), C.c_double()
    st = lib().orc_clip_rmsprop(C.c_size_t(theta.size), _p(theta), _p(m), _p(grad), C.c_float(lr), C.c_float(rho),
                                C.c_float(eps), C.c_float(clip), C.byref(norm), C.byref(scale))
    return int(st), norm.value, scale.value


DEFAULT_HP = dict(gamma=0.99, lr=0.0224, rms_decay=0.99, rms_eps=0.1, clip_norm=40.0,
                  entropy_beta=0.01, value_coef=1.0, term_denom=200, algorithm="a2c", epsilon=0.1,
                  environment="hashed")


class OraclePAAC:
    """State of one PAAC learner on the CPU; rollout() and update() are Algorithm 1's two halves.

    hp["algorithm"] = "a2c" is Algorithm 1 as printed; "nstep_q" keeps the framework (Section 3) and swaps
    what the heads mean (Section 2.2): the A outputs are Q-values, acting is epsilon-greedy, the stored
    value of a step is Q(s_t, a_t), the bootstrap is max_a Q(s_{t_max+1}, a), the loss is Eq. 3 on n-step
    targets.  The value head is carried along unused (its gradient is zero)."""

    def __init__(self, arch, n_e, t_max, n_actions, seed, bf16=False, hp=None, net=None):
        self.net = net if net is not None else arch_net(arch, n_actions)
        self.n_e, self.t_max, self.A, self.seed, self.bf16 = n_e, t_max, n_actions, seed, bf16
        self.hp = dict(DEFAULT_HP)
        self.hp.update(hp or {})
        self.theta = init_params(self.net, seed)
        self.m = np.zeros_like(self.theta)
        self.N = 0
        self.h, self.w = self.net.in_h, self.net.in_w
        self.pattern = self.hp["environment"] == "pattern"
        self.state = pattern_reset(seed, n_e, n_actions, self.h, self.w) if self.pattern else env_reset(seed, n_e, self.h, self.w)
        self.counters = [np.zeros(n_e, np.int32) for _ in range(3)]

    def rollout(self, forced_actions=None):
        """forced_actions: int32 [t_max, n_e] with -1 meaning 'sample'."""
        T, n_e, A = self.t_max, self.n_e, self.A
        step0 = self.N // n_e
        ro = dict(frames=np.zeros((T + 1, n_e, self.h, self.w, 4), np.uint8),
                  actions=np.zeros((T, n_e), np.int32), rewards=np.zeros((T, n_e), np.int8),
                  terminals=np.zeros((T, n_e), np.uint8), values=np.zeros((T + 1, n_e), np.float32),
                  logits=np.zeros((T, n_e, A), np.float32), uniforms=np.zeros((T, n_e), np.float32),
                  probs=np.zeros((T, n_e, A), np.float32), acts=[])
        ro["frames"][0] = self.state
        for t in range(T):
            acts, logits, values = forward(self.net, self.theta, ro["frames"][t], self.bf16)
            p, _, _ = softmax(logits)
            qmode = self.hp["algorithm"] == "nstep_q"
            ro.setdefault("sampled", np.zeros((T, n_e), np.int32))
            for e in range(n_e):
                u = action_uniform(self.seed, e, step0 + t)
                ro["uniforms"][t, e] = u
                a = q_select(logits[e], u, self.hp["epsilon"]) if qmode else sample(p[e], u)
                ro["sampled"][t, e] = a
                if forced_actions is not None and forced_actions[t, e] >= 0:
                    a = int(forced_actions[t, e])
                ro["actions"][t, e] = a
                if qmode:
                    values[e] = logits[e, a]          # what the step is worth to the learner: Q(s_t, a_t)
            ro["logits"][t], ro["values"][t], ro["probs"][t] = logits, values, p
            ro["acts"].append(acts)
            if self.pattern:
                f, r, term = pattern_step(self.seed, step0 + t, ro["actions"][t], self.hp["term_denom"], A, self.counters,
                                          self.h, self.w)
            else:
                f, r, term = env_step(self.seed, step0 + t, ro["actions"][t], self.hp["term_denom"], self.counters,
                                      self.h, self.w)
            ro["frames"][t + 1], ro["rewards"][t], ro["terminals"][t] = f, r, term
        _, zb, vb = forward(self.net, self.theta, ro["frames"][T], self.bf16)
        ro["values"][T] = zb.max(axis=1) if self.hp["algorithm"] == "nstep_q" else vb
        self.state = ro["frames"][T].copy()
        self.ro = ro
        return ro

    def update(self):
        ro, hp, T, n_e = self.ro, self.hp, self.t_max, self.n_e
        B = T * n_e
        R, adv = returns(hp["gamma"], ro["rewards"], ro["terminals"], ro["values"])
        frames = ro["frames"][:T].reshape(B, self.h, self.w, 4)
        acts, logits, values = forward(self.net, self.theta, frames, self.bf16)
        if hp["algorithm"] == "nstep_q":
            dz, qs = q_head_grad(hp["value_coef"], logits, ro["actions"].reshape(B), R.reshape(B))
            dV = np.zeros(B, np.float32)
            stats = dict(policy_loss=0.0, value_loss=qs["value_loss"], entropy=0.0)
        else:
            dz, dV, stats = head_grad(hp["entropy_beta"], hp["value_coef"], logits, values, ro["actions"].reshape(B),
                                      R.reshape(B), adv.reshape(B))
        grad, gacts = backward(self.net, self.theta, frames, acts, dz, dV, self.bf16)
        st, norm, scale = clip_rmsprop(self.theta, self.m, grad, hp["lr"], hp["rms_decay"], hp["rms_eps"],
                                       hp["clip_norm"])
        self.N += B
        out = dict(R=R, adv=adv, dz=dz, dV=dV, grad=grad, gacts=gacts, acts=acts, logits=logits, values=values,
                   grad_norm=norm, clip_scale=scale, status=st, N=self.N)
        out.update(stats)
        self.up = out
        return out
