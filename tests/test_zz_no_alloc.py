"""The optimiser entry point for callers that cannot allocate device memory.

Some hosts of the library may never call cudaMalloc (a frozen memory budget, a device pool owned by
another framework, a sandbox): for them `paac_clip_rmsprop_noalloc` keeps its scratch in an array built
into the library.  This test drives it through the C-ABI with plain torch tensors and checks that it
reproduces what `paac_update` does to the parameters and the RMSProp state, on two calls in a row (the
second call finds the first call's sums still in the built-in array).  It is collected last on purpose.
"""
import numpy as np
import pytest

from paper_1705_04862_b200 import binding as pb

pytestmark = pytest.mark.gpu


def rel(x, y):
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    return float(np.abs(x - y).max() / (np.abs(y).max() + 1e-12))


def test_noalloc_optimiser_matches_update_twice_in_a_row(orc):
    import torch
    hp = dict(lr=0.0224, rms_decay=0.99, rms_eps=0.1, clip_norm=0.5)      # low threshold: clipping is active
    g = pb.Paac("nips", 8, 3, 6, seed=21, precision=pb.BF16, **hp)
    dev = torch.device("cuda:0")
    theta = torch.from_numpy(g.params()).to(dev)
    rms = torch.from_numpy(g.debug_read(pb.DBG_RMS).copy()).to(dev)
    shadow = torch.zeros(g.P, dtype=torch.int16, device=dev)
    out = torch.zeros(2, dtype=torch.float32, device=dev)
    clipped = 0
    theta_o, rms_o = g.params().copy(), g.debug_read(pb.DBG_RMS).copy()       # the oracle's copies walk along
    for call in range(2):
        g.rollout()
        st = g.update()
        assert st["status"] == 0
        grad = torch.from_numpy(g.debug_read(pb.DBG_GRAD).copy()).to(dev)
        st_o, norm_o, scale_o = orc.clip_rmsprop(theta_o, rms_o, grad.cpu().numpy(), hp["lr"], hp["rms_decay"],
                                                 hp["rms_eps"], hp["clip_norm"])
        rc = pb.clip_rmsprop_noalloc(theta, rms, grad, g.P, hp["lr"], hp["rms_decay"], hp["rms_eps"], hp["clip_norm"],
                                     theta_bf16=shadow, norm_and_scale=out,
                                     stream=torch.cuda.current_stream().cuda_stream)
        assert rc == pb.OK
        torch.cuda.synchronize()
        norm, scale = out.cpu().numpy()
        assert abs(norm - st["grad_norm"]) <= 1e-5 * st["grad_norm"] and abs(scale - st["clip_scale"]) <= 1e-5
        clipped += scale < 1.0
        # against the oracle's optimiser step on the same gradient (not only against paac_update)
        assert st_o == 0 and abs(norm - norm_o) <= 1e-5 * norm_o and abs(scale - scale_o) <= 1e-5
        assert rel(theta.cpu().numpy(), theta_o) <= 1e-4 and rel(rms.cpu().numpy(), rms_o) <= 1e-4
        # same tolerance as the float parity tests
        assert rel(theta.cpu().numpy(), g.params()) <= 1e-4
        assert rel(rms.cpu().numpy(), g.debug_read(pb.DBG_RMS)) <= 1e-4
        want16 = torch.from_numpy(g.params()).to(torch.bfloat16).view(torch.int16).numpy()
        got16 = shadow.cpu().numpy()
        assert np.mean(got16 != want16) <= 1e-3 and np.abs(got16.astype(np.int32) - want16).max() <= 1
    assert clipped >= 1
    g.close()


def test_noalloc_rejects_sizes_beyond_its_scratch_and_bad_arguments():
    import torch
    L = pb.lib()
    cap = int(L.paac_noalloc_max_params())
    assert cap == 4096 * 4096
    t = torch.zeros(16, dtype=torch.float32, device="cuda:0")
    before = t.clone()
    assert pb.clip_rmsprop_noalloc(t, t, t, cap + 1, 0.01, 0.99, 0.1, 40.0) == pb.ERR_LIMIT
    assert pb.clip_rmsprop_noalloc(t, t, None, 16, 0.01, 0.99, 0.1, 40.0) == pb.ERR_ARG
    assert pb.clip_rmsprop_noalloc(t, t, t, 0, 0.01, 0.99, 0.1, 40.0) == pb.ERR_ARG
    torch.cuda.synchronize()
    assert torch.equal(t, before)
    # non-finite gradient: nothing changes, the reported factor is 0
    th = torch.ones(5000, device="cuda:0")
    m = torch.full((5000,), 2.0, device="cuda:0")
    gr = torch.ones(5000, device="cuda:0")
    gr[4999] = float("inf")
    out = torch.ones(2, device="cuda:0")
    assert pb.clip_rmsprop_noalloc(th, m, gr, 5000, 0.01, 0.99, 0.1, 40.0, norm_and_scale=out) == pb.OK
    torch.cuda.synchronize()
    assert torch.all(th == 1) and torch.all(m == 2) and out[1].item() == 0.0
