"""The pre-processing kernel (Section 5.1) against the oracle, bit for bit, through the C-ABI."""
import numpy as np
import pytest

from paper_1705_04862_b200 import binding as pb

pytestmark = pytest.mark.gpu


def _run(raw_a, raw_b, state_in, in_place=False):
    import torch
    n = raw_a.shape[0]
    a, b = torch.from_numpy(raw_a).cuda(), torch.from_numpy(raw_b).cuda()
    sin = torch.from_numpy(state_in).cuda() if state_in is not None else None
    out = sin if in_place else torch.zeros((n, 84, 84, 4), dtype=torch.uint8, device="cuda")
    st = pb.preprocess(a, b, sin, out, n, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert st == pb.OK
    return out.cpu().numpy()


def test_small_batches_edge_values_and_in_place(orc):
    rng = np.random.RandomState(3)
    for n in (1, 5):
        a = rng.randint(0, 256, (n, 210, 160, 3), dtype=np.uint8)
        b = rng.randint(0, 256, (n, 210, 160, 3), dtype=np.uint8)
        prev = rng.randint(0, 256, (n, 84, 84, 4), dtype=np.uint8)
        assert np.array_equal(_run(a, b, prev), orc.preprocess(a, b, prev))
        assert np.array_equal(_run(a, b, None), orc.preprocess(a, b, None))
        assert np.array_equal(_run(a, b, prev.copy(), in_place=True), orc.preprocess(a, b, prev))
    # extremes: all white, all black, single bright pixels at the corners
    z = np.zeros((1, 210, 160, 3), np.uint8)
    w = np.full((1, 210, 160, 3), 255, np.uint8)
    assert np.array_equal(_run(z, w, None), orc.preprocess(z, w, None))
    c = z.copy()
    c[0, 0, 0], c[0, 209, 159], c[0, 0, 159], c[0, 209, 0] = 255, 255, 255, 255
    assert np.array_equal(_run(c, z, None), orc.preprocess(c, z, None))


def test_full_size_batch(orc):
    """1024 environments, the size the bench times: every output pixel against the oracle."""
    rng = np.random.RandomState(9)
    n = 1024
    a = rng.randint(0, 256, (n, 210, 160, 3), dtype=np.uint8)
    b = np.roll(a, 7, axis=2)                     # two correlated frames, as consecutive emulator frames are
    prev = rng.randint(0, 256, (n, 84, 84, 4), dtype=np.uint8)
    got = _run(a, b, prev)
    for lo in range(0, n, 128):                   # the oracle in slices: it is a plain loop nest
        assert np.array_equal(got[lo:lo + 128], orc.preprocess(a[lo:lo + 128], b[lo:lo + 128], prev[lo:lo + 128]))


def test_bad_arguments():
    import torch
    x = torch.zeros(16, dtype=torch.uint8, device="cuda")
    L = pb.lib()
    assert L.paac_preprocess(None, x.data_ptr(), None, x.data_ptr(), 1, None) == pb.ERR_ARG
    assert L.paac_preprocess(x.data_ptr(), x.data_ptr(), None, x.data_ptr(), 0, None) == pb.ERR_ARG
    assert L.paac_preprocess(x.data_ptr() + 1, x.data_ptr(), None, x.data_ptr(), 1, None) == pb.ERR_ARG


def test_frame_stack_against_the_oracle(orc):
    """paac_stack_push: the newest plane joins the state (or fills it where an episode restarts), bit for bit, for a
    single environment, a ragged batch, 1024 environments, and in place."""
    import torch
    rng = np.random.RandomState(11)
    for n in (1, 37, 1024):
        prev = rng.randint(0, 256, (n, 84, 84, 4), dtype=np.uint8)
        plane = rng.randint(0, 256, (n, 84, 84), dtype=np.uint8)
        restart = (rng.randint(0, 4, n) == 0).astype(np.uint8)
        for flags in (None, restart):
            sin, pl = torch.from_numpy(prev).cuda(), torch.from_numpy(plane).cuda()
            fl = torch.from_numpy(flags).cuda() if flags is not None else None
            out = torch.zeros_like(sin)
            assert pb.stack_push(sin, pl, fl, out, n, torch.cuda.current_stream().cuda_stream) == pb.OK
            torch.cuda.synchronize()
            want = orc.stack_push(prev, plane, flags)
            assert np.array_equal(out.cpu().numpy(), want)
            assert pb.stack_push(sin, pl, fl, sin, n, torch.cuda.current_stream().cuda_stream) == pb.OK      # in place
            torch.cuda.synchronize()
            assert np.array_equal(sin.cpu().numpy(), want)
    x = torch.zeros(64, dtype=torch.uint8, device="cuda")
    L = pb.lib()
    assert L.paac_stack_push(None, x.data_ptr(), None, x.data_ptr(), 1, None) == pb.ERR_ARG
    assert L.paac_stack_push(x.data_ptr(), x.data_ptr(), None, x.data_ptr(), 0, None) == pb.ERR_ARG
    assert L.paac_stack_push(x.data_ptr() + 4, x.data_ptr(), None, x.data_ptr(), 1, None) == pb.ERR_ARG
