"""Pins for the CPU oracle: each test compares it with something other than itself --
published vectors, a second implementation, PyTorch float64 autograd, closed forms,
finite differences.  None of these needs a GPU."""
import math
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M32 = 0xFFFFFFFF


# ----------------------------------------------------------------------------- Philox
def py_philox(ctr, key):
    """Second implementation, written from the generator's published definition."""
    c, k = list(ctr), list(key)
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & M32, p1 & M32, ((p0 >> 32) ^ c[3] ^ k[1]) & M32, p0 & M32]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def test_philox_known_answers(orc):
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert orc.philox(w[:4], w[4:6]) == w[6:]
        assert py_philox(w[:4], w[4:6]) == w[6:]
        n += 1
    assert n >= 2


def test_philox_matches_second_implementation(orc):
    rng = np.random.RandomState(0)
    for _ in range(200):
        w = [int(x) for x in rng.randint(0, 2 ** 32, size=6, dtype=np.uint64)]
        assert orc.philox(w[:4], w[4:]) == py_philox(w[:4], w[4:])


def test_action_uniform_mapping_and_uniformity(orc):
    seed = (7 << 32) | 12345
    us = []
    for env in range(40):
        for step in (0, 1, 2, 2 ** 32 + 5):
            out = py_philox([env, step & M32, step >> 32, 2], [seed & M32, seed >> 32])
            u = (out[0] >> 8) / 2.0 ** 24
            assert orc.action_uniform(seed, env, step) == np.float32(u)
            assert 0.0 <= u < 1.0
            us.append(u)
    us = np.array([orc.action_uniform(1, e, s) for e in range(64) for s in range(64)])
    hist, _ = np.histogram(us, bins=16, range=(0, 1))
    expect = us.size / 16
    chi2 = ((hist - expect) ** 2 / expect).sum()
    assert chi2 < 45.0           # 15 degrees of freedom, p ~ 1e-4


# ----------------------------------------------------------------------------- environment
K0, K1, K2 = 0x9E3779B9, 0xBB67AE85, 0x6A09E667


def py_mix(x):
    x ^= x >> 16
    x = (x * K0) & M32
    x ^= x >> 15
    x = (x * K1) & M32
    x ^= x >> 16
    return x


def py_base(seed, env, step, tag):
    h = py_mix((seed & M32) ^ K2)
    h = py_mix(h ^ (seed >> 32))
    h = py_mix(h ^ env)
    h = py_mix(h ^ step)
    return py_mix(h ^ tag)


def py_frame(seed, env, step, tag, h=84, w=84):
    base = py_base(seed, env, step, tag)
    idx = np.arange(1, h * w + 1, dtype=np.uint64)
    x = (base + K0 * idx) & M32
    x ^= x >> np.uint64(16)
    x = (x * K0) & M32
    x ^= x >> np.uint64(15)
    x = (x * K1) & M32
    x ^= x >> np.uint64(16)
    words = x.astype("<u4")
    return words.view(np.uint8).reshape(h, w, 4)


def py_outcome(seed, env, step, action, denom):
    base = py_base(seed, env, step, action + 1)
    hr = py_mix(base ^ 0x52455744) & 15
    r = 1 if hr == 0 else (-1 if hr == 1 else 0)
    ht = py_mix(base ^ 0x5445524D)
    return r, int(((ht * denom) >> 32) == 0)


def test_env_frames_match_second_implementation(orc):
    for seed, env, step, tag in [(1, 0, 0, 0), (1, 3, 17, 5), ((9 << 32) | 77, 1023, 123456, 19), (2 ** 64 - 1, 7, 1, 1)]:
        assert np.array_equal(orc.env_frame(seed, env, step, tag), py_frame(seed, env, step, tag))
    # little-endian channel order of one pixel word
    f = orc.env_frame(1, 2, 3, 4)
    word = py_mix((py_base(1, 2, 3, 4) + K0 * (5 * 84 + 6 + 1)) & M32)
    assert [int(v) for v in f[5, 6]] == [(word >> (8 * c)) & 255 for c in range(4)]


def test_env_outcomes_match_second_implementation_and_frequencies(orc):
    n, rp, rm, term = 0, 0, 0, 0
    for env in range(50):
        for step in range(200):
            a = (env + step) % 6
            r, t = orc.env_outcome(1, env, step, a, 200)
            assert (r, t) == py_outcome(1, env, step, a, 200)
            n += 1
            rp += r == 1
            rm += r == -1
            term += t
    # binomial bounds, 5 sigma
    for cnt, p in ((rp, 1 / 16), (rm, 1 / 16), (term, 1 / 200)):
        assert abs(cnt - n * p) < 5 * math.sqrt(n * p * (1 - p))
    t100 = sum(orc.env_outcome(3, e, s, 0, 100)[1] for e in range(40) for s in range(250))
    assert abs(t100 - 100) < 5 * math.sqrt(100)


def test_env_bytes_are_flat(orc):
    f = np.concatenate([orc.env_frame(5, e, 9, 1).reshape(-1) for e in range(8)])
    hist = np.bincount(f, minlength=256)
    expect = f.size / 256
    assert ((hist - expect) ** 2 / expect).sum() < 400.0     # 255 d.o.f.


def test_env_step_bookkeeping(orc):
    seed, n_e, denom = 11, 64, 8         # frequent terminals
    cnt = [np.zeros(n_e, np.int32) for _ in range(3)]
    ep_len = np.zeros(n_e, int)
    ep_ret = np.zeros(n_e, int)
    eps = np.zeros(n_e, int)
    for step in range(40):
        actions = np.array([(e * 7 + step) % 4 for e in range(n_e)], np.int32)
        f, r, t = orc.env_step(seed, step, actions, denom, cnt)
        for e in range(n_e):
            rr, tt = py_outcome(seed, e, step, int(actions[e]), denom)
            assert (int(r[e]), int(t[e])) == (rr, tt)
            tag = 0 if tt else int(actions[e]) + 1
            if e % 16 == 0:
                assert np.array_equal(f[e], py_frame(seed, e, step + 1, tag))
            ep_len[e] += 1
            ep_ret[e] += rr
            if tt:
                eps[e] += 1
                ep_len[e] = 0
                ep_ret[e] = 0
        assert np.array_equal(cnt[0], ep_len) and np.array_equal(cnt[1], ep_ret) and np.array_equal(cnt[2], eps)
    assert eps.sum() > 0
    assert np.array_equal(orc.env_reset(seed, 3)[2], py_frame(seed, 2, 0, 0))


# ----------------------------------------------------------------------------- bf16, init
def test_bf16_round_matches_torch(orc):
    rng = np.random.RandomState(1)
    x = np.concatenate([rng.randn(2000).astype(np.float32) * 10 ** rng.uniform(-6, 6, 2000).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(orc.bf16_round(x), ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.bf16_round(np.float32([1.00390625]))[0] == 1.0
    assert orc.bf16_round(np.float32([1.01171875]))[0] == np.float32(1.015625)


def test_xavier_init(orc):
    net = orc.arch_net("nips", 4)
    th = orc.init_params(net, 1)
    assert th.size == 677429                       # 4112 + 8224 + 663808 + 257*5
    w1 = th[:4096]
    b = math.sqrt(6.0 / (8 * 8 * 4 + 8 * 8 * 16))
    assert np.all(np.abs(w1) <= np.float32(b)) and np.all(th[4096:4112] == 0)
    wfc = th[4112 + 8224: 4112 + 8224 + 2592 * 256]
    bfc = math.sqrt(6.0 / (2592 + 256))
    assert abs(wfc.var() / (bfc * bfc / 3) - 1) < 0.02 and abs(wfc.mean()) < 3 * bfc / math.sqrt(3 * wfc.size)
    # element i of layer l is philox counter (i, l, 0, 1)
    out = py_philox([5, 1, 0, 1], [1, 0])
    u = np.float32((out[0] >> 8) / 2.0 ** 24)
    b2 = np.float32(math.sqrt(6.0 / (4 * 4 * 16 + 4 * 4 * 32)))
    assert th[4112 + 5] == (np.float32(2) * u - np.float32(1)) * b2
    assert orc.param_count(orc.arch_net("nature", 18)) == 1693875
    assert not np.array_equal(th, orc.init_params(net, 2))
    # the two heads: fan_in = hidden units, fan_out = actions (policy) and 1 (value); layer ids follow the fc layer's.
    # With 18 x 512 and 512 samples the largest magnitude comes within a few per cent of the bound from below, the
    # sample variance is that of a uniform, and one element of each goes through the Python Philox.
    nat = orc.arch_net("nature", 18)
    tn = orc.init_params(nat, 3)
    o_pi = tn.size - (512 + 1) - (18 * 512 + 18)
    wpi, bpi = tn[o_pi:o_pi + 18 * 512], tn[o_pi + 18 * 512:o_pi + 18 * 512 + 18]
    wv, bv = tn[-513:-1], tn[-1]
    b_pi, b_v = math.sqrt(6.0 / (512 + 18)), math.sqrt(6.0 / (512 + 1))
    assert np.all(bpi == 0) and bv == 0
    assert 0.995 * b_pi < np.abs(wpi).max() <= np.float32(b_pi) and 0.97 * b_v < np.abs(wv).max() <= np.float32(b_v)
    assert abs(wpi.var() / (b_pi * b_pi / 3) - 1) < 0.05 and abs(wv.var() / (b_v * b_v / 3) - 1) < 0.2
    for layer, off, bound, i in ((4, o_pi, b_pi, 7), (5, tn.size - 513, b_v, 100)):
        out = py_philox([i, layer, 0, 1], [3, 0])
        u = np.float32((out[0] >> 8) / 2.0 ** 24)
        assert tn[off + i] == (np.float32(2) * u - np.float32(1)) * np.float32(bound)


# ----------------------------------------------------------------------------- network vs PyTorch float64
def torch_params(net, theta, dtype=torch.float64, round_bf16=False):
    """Split the canonical flat vector into torch tensors (conv W as [co][kh][kw][ci] -> OIHW)."""
    ps, o, h, w, c = [], 0, net.in_h, net.in_w, net.in_c
    th = torch.tensor(theta, dtype=dtype)

    def rb(x):
        return x.to(torch.float32).to(torch.bfloat16).to(dtype) if round_bf16 else x
    for l in range(net.n_conv):
        k, co = net.k[l], net.cout[l]
        n = co * k * k * c
        W = th[o:o + n].reshape(co, k, k, c)
        ps.append((W, th[o + n:o + n + co]))
        o += n + co
        h, w, c = (h - k) // net.stride[l] + 1, (w - k) // net.stride[l] + 1, co
    fin = h * w * c
    for out in (net.fc, net.n_actions, 1):
        inn = fin if out == net.fc and len(ps) == net.n_conv else net.fc
        ps.append((th[o:o + out * inn].reshape(out, inn), th[o + out * inn:o + out * inn + out]))
        o += out * inn + out
    assert o == th.numel()
    return ps, rb


def torch_forward(net, leaves, frames, round_bf16=False):
    """leaves: list of (W, b) float64 tensors in canonical layout. Returns acts, logits, values."""
    def rb(x):
        if not round_bf16:
            return x
        return x + (x.detach().to(torch.float32).to(torch.bfloat16).to(x.dtype) - x.detach())
    x = torch.tensor(frames, dtype=torch.float64).permute(0, 3, 1, 2) / 255.0
    acts = []
    for l in range(net.n_conv):
        W, b = leaves[l]
        x = torch.nn.functional.conv2d(x, rb(W).permute(0, 3, 1, 2), b, stride=net.stride[l])
        x = rb(torch.relu(x))
        acts.append(x.permute(0, 2, 3, 1))
    flat = x.permute(0, 2, 3, 1).reshape(x.shape[0], -1)
    W, b = leaves[net.n_conv]
    h = rb(torch.relu(flat @ rb(W).t() + b))
    acts.append(h)
    Wp, bp = leaves[net.n_conv + 1]
    Wv, bv = leaves[net.n_conv + 2]
    return acts, h @ rb(Wp).t() + bp, (h @ rb(Wv).t() + bv).reshape(-1)


def torch_loss(logits, values, actions, R, adv, beta, cv):
    lp = torch.log_softmax(logits, dim=1)
    p = lp.exp()
    H = -(p * lp).sum(1)
    a = torch.tensor(actions, dtype=torch.long)
    pol = -(torch.tensor(adv, dtype=torch.float64) * lp[torch.arange(len(a)), a])
    val = cv * (torch.tensor(R, dtype=torch.float64) - values) ** 2
    return (pol - beta * H + val).mean(), pol.mean(), val.mean(), H.mean()


TINY = [((12, 12, 1), [(2, 4, 2)], 4, 3),
        ((13, 11, 4), [(3, 3, 2), (5, 2, 1)], 6, 4),
        ((20, 20, 4), [(4, 8, 4), (6, 2, 1), (5, 2, 1)], 7, 18)]


def tiny_case(orc, spec, n=5, seed=3):
    hwc, convs, fc, A = spec
    net = orc.make_net(hwc, convs, fc, A)
    rng = np.random.RandomState(seed)
    theta = orc.init_params(net, seed)
    # non-zero biases so that bias gradients and ReLU masks are exercised
    theta = (theta + 0.05 * rng.randn(theta.size)).astype(np.float32)
    frames = rng.randint(0, 256, size=(n,) + hwc, dtype=np.uint8)
    actions = rng.randint(0, A, size=n).astype(np.int32)
    R = rng.randn(n).astype(np.float32)
    adv = rng.randn(n).astype(np.float32)
    return net, theta, frames, actions, R, adv


def rel(x, y):
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    return float(np.abs(x - y).max() / (np.abs(y).max() + 1e-12))


@pytest.mark.parametrize("spec", TINY)
def test_forward_backward_match_torch_float64(orc, spec):
    net, theta, frames, actions, R, adv = tiny_case(orc, spec)
    beta, cv = 0.01, 1.0
    acts, logits, values = orc.forward(net, theta, frames)
    ps, _ = torch_params(net, theta)
    leaves = [(W.clone().requires_grad_(True), b.clone().requires_grad_(True)) for W, b in ps]
    tacts, tlogits, tvalues = torch_forward(net, leaves, frames)
    for a, ta in zip(acts, tacts):
        assert rel(a, ta.detach().numpy()) < 2e-6
    assert rel(logits, tlogits.detach().numpy()) < 2e-6 and rel(values, tvalues.detach().numpy()) < 2e-6
    loss, pol, val, H = torch_loss(tlogits, tvalues, actions, R, adv, beta, cv)
    tlogits.retain_grad()
    tvalues.retain_grad()
    loss.backward()
    dz, dV, stats = orc.head_grad(beta, cv, logits, values, actions, R, adv)
    assert rel(dz, tlogits.grad.numpy()) < 1e-5 and rel(dV, tvalues.grad.numpy()) < 1e-5
    assert abs(stats["policy_loss"] - pol.item()) < 1e-5 and abs(stats["value_loss"] - val.item()) < 1e-5
    assert abs(stats["entropy"] - H.item()) < 1e-6
    grad, gacts = orc.backward(net, theta, frames, acts, dz, dV)
    tgrad = torch.cat([torch.cat([W.grad.reshape(-1), b.grad.reshape(-1)]) for W, b in leaves]).numpy()
    assert grad.shape == tgrad.shape
    # per-layer comparison so a small layer cannot hide behind a large one
    o = 0
    for W, b in leaves:
        for t in (W, b):
            n = t.numel()
            assert rel(grad[o:o + n], tgrad[o:o + n]) < 2e-5, (o, n)
            o += n


@pytest.mark.parametrize("spec", TINY[:2])
def test_gradient_matches_finite_differences(orc, spec):
    net, theta, frames, actions, R, adv = tiny_case(orc, spec, n=4, seed=5)
    beta, cv = 0.02, 0.7
    acts, logits, values = orc.forward(net, theta, frames)
    dz, dV, _ = orc.head_grad(beta, cv, logits, values, actions, R, adv)
    grad, _ = orc.backward(net, theta, frames, acts, dz, dV)
    th64 = theta.astype(np.float64)
    rng = np.random.RandomState(0)
    idx = rng.choice(theta.size, size=min(60, theta.size), replace=False)
    h = 1e-5
    scale = np.abs(grad).max()
    for i in idx:
        tp, tm = th64.copy(), th64.copy()
        tp[i] += h
        tm[i] -= h
        fd = (orc.loss_double(net, tp, frames, beta, cv, actions, R, adv)
              - orc.loss_double(net, tm, frames, beta, cv, actions, R, adv)) / (2 * h)
        assert abs(fd - grad[i]) < 2e-5 * scale + 1e-7, (i, fd, grad[i])


def test_conv_hand_cases(orc):
    # one conv layer whose only non-zero weight picks pixel (r=1, s=2, ci=1) of each window
    net = orc.make_net((6, 7, 2), [(1, 3, 2)], 2, 2)
    theta = np.zeros(orc.param_count(net), np.float32)
    theta[(1 * 3 + 2) * 2 + 1] = 1.0
    rng = np.random.RandomState(0)
    frames = rng.randint(0, 256, size=(2, 6, 7, 2), dtype=np.uint8)
    acts, _, _ = orc.forward(net, theta, frames)
    expect = frames[:, 1::2, 2::2, 1][:, :2, :3].astype(np.float64) / 255.0
    assert np.allclose(acts[0][..., 0], expect, rtol=0, atol=1e-7)
    # negative bias large enough to switch every unit off: ReLU gives zeros, gradients vanish
    theta[18] = -2.0
    acts, logits, values = orc.forward(net, theta, frames)
    assert np.all(acts[0] == 0)
    dz = np.ones((2, 2), np.float32)
    dV = np.ones(2, np.float32)
    grad, _ = orc.backward(net, theta, frames, acts, dz, dV)
    assert np.all(grad[:19] == 0)


def test_bf16_mode_matches_torch_with_explicit_rounding(orc):
    net, theta, frames, actions, R, adv = tiny_case(orc, TINY[2], n=6, seed=9)
    acts, logits, values = orc.forward(net, theta, frames, bf16=True)
    ps, _ = torch_params(net, theta)
    leaves = [(W.clone().requires_grad_(True), b.clone().requires_grad_(True)) for W, b in ps]
    tacts, tlogits, tvalues = torch_forward(net, leaves, frames, round_bf16=True)
    for a, ta in zip(acts, tacts):
        a16 = torch.tensor(a).to(torch.bfloat16).to(torch.float32).numpy()
        assert np.array_equal(a, a16)                      # stored activations are bf16 values
        assert rel(a, ta.detach().numpy()) < 1e-2          # one bf16 ulp where a sum lands on a tie
        assert np.mean(a != ta.detach().numpy().astype(np.float32)) < 0.02
    assert rel(logits, tlogits.detach().numpy()) < 1e-2
    # backward: weight gradients are exact sums of products of the stored bf16 tensors
    dz, dV, _ = orc.head_grad(0.01, 1.0, logits, values, actions, R, adv)
    grad, gacts = orc.backward(net, theta, frames, acts, dz, dV, bf16=True)
    for g in gacts:
        assert np.array_equal(g, torch.tensor(g).to(torch.bfloat16).to(torch.float32).numpy())
    L = net.n_conv
    # fc weight gradient recomputed with numpy from the oracle's own stored tensors (definition of wgrad)
    IN = acts[L - 1].reshape(6, -1).astype(np.float64)
    gW = gacts[L].astype(np.float64).T @ IN
    o = sum(net.cout[l] * net.k[l] ** 2 * c + net.cout[l] for l, c in zip(range(L), [4, 4, 6]))
    assert rel(grad[o:o + gW.size], gW.reshape(-1)) < 1e-6
    # straight-through comparison with torch: gradient of the rounded network, loose (rounding of gacts)
    loss, *_ = torch_loss(tlogits, tvalues, actions, R, adv, 0.01, 1.0)
    loss.backward()
    tgrad = torch.cat([torch.cat([W.grad.reshape(-1), b.grad.reshape(-1)]) for W, b in leaves]).numpy()
    assert rel(grad, tgrad) < 3e-2


# ----------------------------------------------------------------------------- softmax, sampling
def test_softmax_invariants(orc):
    rng = np.random.RandomState(2)
    for A in (2, 4, 6, 18):
        z = (rng.randn(50, A) * 3).astype(np.float32)
        p, lp, H = orc.softmax(z)
        assert np.all(np.abs(p.sum(1) - 1) < 1e-6)
        assert np.all(H >= 0) and np.all(H <= math.log(A) + 1e-6)
        ref = torch.softmax(torch.tensor(z, dtype=torch.float64), 1).numpy()
        assert rel(p, ref) < 1e-6
        p2, lp2, H2 = orc.softmax(z + np.float32(8.0))
        assert rel(p2, p) < 1e-5 and rel(H2, H) < 1e-5
        pe, _, He = orc.softmax(np.full((1, A), 1.25, np.float32))
        assert abs(He[0] - math.log(A)) < 1e-6 and np.allclose(pe, 1 / A)
    # extreme logits do not overflow
    p, lp, H = orc.softmax(np.float32([[1000.0, 0.0, -1000.0]]))
    assert p[0, 0] == 1.0 and H[0] == 0.0 and np.isfinite(lp).all()


def test_sampling_is_inverse_cdf(orc):
    p = np.float32([0.1, 0.2, 0.3, 0.4])
    cdf = np.cumsum(p, dtype=np.float32)
    for u in np.linspace(0, 0.9999, 97):
        k = orc.sample(p, float(u))
        assert k == int(np.searchsorted(cdf, np.float32(u), side="right"))
    assert orc.sample(p, float(cdf[0])) == 1            # strict '<': u equal to a boundary goes up
    assert orc.sample(np.float32([0.5, 0.25]), 0.9) == 1   # nothing reached: last action
    assert abs(orc.cdf_margin(p, 0.35) - 0.05) < 1e-6
    # frequencies follow p
    us = [orc.action_uniform(3, e, s) for e in range(100) for s in range(100)]
    cnt = np.bincount([orc.sample(p, u) for u in us], minlength=4)
    assert np.all(np.abs(cnt / len(us) - p) < 0.02)


def test_head_gradient_rows_sum_to_zero_and_equal_logits(orc):
    rng = np.random.RandomState(4)
    B, A = 12, 6
    z = rng.randn(B, A).astype(np.float32)
    v = rng.randn(B).astype(np.float32)
    a = rng.randint(0, A, B).astype(np.int32)
    R = rng.randn(B).astype(np.float32)
    adv = rng.randn(B).astype(np.float32)
    dz, dV, _ = orc.head_grad(0.05, 1.0, z, v, a, R, adv)
    assert np.all(np.abs(dz.sum(1)) < 1e-7)
    assert np.allclose(dV, 2 * (v - R) / B, rtol=1e-6)
    # equal logits: the entropy term has zero gradient, only the policy term is left
    dz2, _, st = orc.head_grad(0.05, 1.0, np.zeros((B, A), np.float32), v, a, R, adv)
    onehot = np.eye(A)[a]
    assert np.allclose(dz2, -adv[:, None] * (onehot - 1 / A) / B, atol=1e-8)
    assert abs(st["entropy"] - math.log(A)) < 1e-6


# ----------------------------------------------------------------------------- returns
def test_returns_worked_cases(orc):
    r = np.int8([[1], [0], [-1]])
    n = 0
    for line in open(os.path.join(GOLDEN, "returns_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        left, right = line.split("|")
        term = np.uint8([[int(x)] for x in left.split()])
        want = [float(x) for x in right.split()]
        v = np.float32([[0.3], [-0.2], [0.1], [4.0]])
        R, adv = orc.returns(0.5, r, term, v)
        assert [float(x) for x in R[:, 0]] == want
        assert np.allclose(adv[:, 0], np.float32(want) - v[:3, 0])
        n += 1
    assert n == 4


def test_returns_closed_form(orc):
    rng = np.random.RandomState(6)
    T, n_e, g = 5, 40, 0.99
    r = rng.randint(-1, 2, size=(T, n_e)).astype(np.int8)
    term = (rng.rand(T, n_e) < 0.2).astype(np.uint8)
    v = rng.randn(T + 1, n_e).astype(np.float32)
    R, adv = orc.returns(g, r, term, v)
    g32 = float(np.float32(g))
    for e in range(n_e):
        for t in range(T):
            acc, k, done = 0.0, 0, False
            for j in range(t, T):
                acc += g32 ** k * r[j, e]
                k += 1
                if term[j, e]:
                    done = True
                    break
            if not done:
                acc += g32 ** k * float(v[T, e])
            assert abs(R[t, e] - acc) < 1e-5
            assert abs(adv[t, e] - (acc - v[t, e])) < 1e-5
    R0, _ = orc.returns(0.0, r, term, v)
    assert np.array_equal(R0, r.astype(np.float32))
    R1, _ = orc.returns(g, r[:1], np.zeros((1, n_e), np.uint8), v[[0, 1]])
    assert np.allclose(R1[0], r[0] + np.float32(g) * v[1], atol=1e-6)    # one-step TD target


# ----------------------------------------------------------------------------- optimiser
def test_clip_and_rmsprop_closed_forms(orc):
    rng = np.random.RandomState(8)
    P = 1000
    g = rng.randn(P).astype(np.float32) * 3          # norm ~ 95 > 40
    th0 = rng.randn(P).astype(np.float32)
    th, m = th0.copy(), np.zeros(P, np.float32)
    st, norm, sc = orc.clip_rmsprop(th, m, g, 0.0224, 0.99, 0.1, 40.0)
    assert st == 0 and abs(norm - np.linalg.norm(g.astype(np.float64))) < 1e-9 and abs(sc - 40 / norm) < 1e-12
    gs = g.astype(np.float64) * sc
    assert abs(np.linalg.norm(gs) - 40) < 1e-9
    assert np.allclose(m, 0.01 * gs * gs, rtol=1e-5)
    assert np.allclose(th, th0 - 0.0224 * gs / np.sqrt(0.01 * gs * gs + 0.1), rtol=0, atol=1e-6)
    # below the threshold nothing is rescaled; constant gradient: m_n = (1 - rho^n) g^2
    g2 = np.full(P, 0.5, np.float32)
    th, m = th0.copy(), np.zeros(P, np.float32)
    for n in range(1, 6):
        st, norm, sc = orc.clip_rmsprop(th, m, g2, 0.01, 0.9, 0.1, 40.0)
        assert sc == 1.0 and np.allclose(m, (1 - 0.9 ** n) * 0.25, rtol=1e-5)
    # clipping off, non-finite norm leaves everything untouched
    th, m = th0.copy(), np.zeros(P, np.float32)
    st, norm, sc = orc.clip_rmsprop(th, m, g, 0.01, 0.99, 0.1, 0.0)
    assert sc == 1.0
    gbad = g.copy()
    gbad[3] = np.inf
    th, m = th0.copy(), np.ones(P, np.float32)
    st, _, _ = orc.clip_rmsprop(th, m, gbad, 0.01, 0.99, 0.1, 40.0)
    assert st == 1 and np.array_equal(th, th0) and np.all(m == 1)


# ----------------------------------------------------------------------------- whole iteration plumbing
def test_iteration_is_consistent_with_its_steps(orc):
    net = orc.make_net((20, 20, 4), [(4, 8, 4), (6, 2, 1)], 8, 3)
    o = orc.OraclePAAC(None, n_e=3, t_max=4, n_actions=3, seed=5, net=net, hp=dict(term_denom=4, lr=0.003))
    th0 = o.theta.copy()
    ro = o.rollout()
    assert np.array_equal(ro["frames"][0], orc.env_reset(5, 3, 20, 20))
    for t in range(4):
        for e in range(3):
            a = int(ro["actions"][t, e])
            assert a == orc.sample(ro["probs"][t, e], float(ro["uniforms"][t, e]))
            r, term = py_outcome(5, e, t, a, 4)
            assert (int(ro["rewards"][t, e]), int(ro["terminals"][t, e])) == (r, term)
            assert np.array_equal(ro["frames"][t + 1, e], py_frame(5, e, t + 1, 0 if term else a + 1, 20, 20))
    up = o.update()
    assert o.N == 12 and up["status"] == 0
    assert np.array_equal(up["logits"].reshape(4, 3, 3), ro["logits"])      # same theta: recomputed = stored
    assert not np.array_equal(o.theta, th0)
    # second iteration continues from the last state with the global step index
    ro2 = o.rollout(forced_actions=np.full((4, 3), 1, np.int32))
    assert np.array_equal(ro2["frames"][0], ro["frames"][4]) and np.all(ro2["actions"] == 1)
    assert ro2["uniforms"][0, 2] == np.float32(orc.action_uniform(5, 2, 4))


# ----------------------------------------------------------------------------- the learnable environment
def test_pattern_environment(orc):
    """The second synthetic environment: hashed frames with a bright band of rows that names the rewarded action."""
    seed, A = 9, 6
    band = 84 // A
    goals = []
    for e, step, tag in ((0, 0, 0), (3, 7, 2), (11, 123, 0)):
        g = orc.pattern_goal(seed, e, step, A)
        goals.append(g)
        # second implementation of the goal: the Python hash chain of the environment pins
        assert g == py_mix(py_base(seed, e, step, 0) ^ 0x474F414C) % A
        f = orc.pattern_frame(seed, e, step, tag, A)
        ref = py_frame(seed, e, step, tag) & 63               # dim texture
        ref[band * g:band * (g + 1)] = 255
        assert np.array_equal(f, ref)
    # goals are spread over the actions; a matching action pays 1, any other 0; terminals are the hashed ones
    gs = np.array([orc.pattern_goal(seed, e, 5, A) for e in range(3000)])
    assert np.all(np.abs(np.bincount(gs, minlength=A) - 500) < 5 * math.sqrt(500))
    n_e = 64
    counters = [np.zeros(n_e, np.int32) for _ in range(3)]
    acts = np.arange(n_e, dtype=np.int32) % A
    f, r, t = orc.pattern_step(seed, 5, acts, 50, A, counters)
    for e in range(n_e):
        assert r[e] == (1 if acts[e] == orc.pattern_goal(seed, e, 5, A) else 0)
        assert t[e] == orc.env_outcome(seed, e, 5, int(acts[e]), 50)[1]
        tag = 0 if t[e] else int(acts[e]) + 1
        assert np.array_equal(f[e], orc.pattern_frame(seed, e, 6, tag, A))
    assert np.array_equal(orc.pattern_reset(seed, 2, A)[1], orc.pattern_frame(seed, 1, 0, 0, A))
