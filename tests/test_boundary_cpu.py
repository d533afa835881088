"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, sizes workspaces, validates arguments, and refuses to run without a device."""
import ctypes as C
import os
import re

from paper_1705_04862_b200 import binding as pb
from paper_1705_04862_b200 import build as pbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_every_declared_symbol():
    pbuild.build()
    L = pb.lib()
    hdr = open(os.path.join(ROOT, "include", "paac.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(paac_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(pb.EXPORTS), declared ^ set(pb.EXPORTS)
    for name in declared:
        assert getattr(L, name) is not None


def test_struct_layouts_match_header():
    assert C.sizeof(pb.HParams) == 80 and pb.HParams.workspace.offset == 40 and pb.HParams.stream.offset == 56
    assert pb.HParams.algorithm.offset == 64 and pb.HParams.epsilon.offset == 68 and pb.HParams.environment.offset == 72
    assert C.sizeof(pb.UpdateStats) == 32 and pb.UpdateStats.timesteps.offset == 24
    assert C.sizeof(pb.RolloutView) == 64


def test_defaults_are_the_papers_hyperparameters():
    hp = pb.default_hparams()
    got = (hp.gamma, hp.lr, hp.rms_decay, hp.rms_eps, hp.clip_norm, hp.entropy_beta, hp.value_coef)
    want = (0.99, 0.0224, 0.99, 0.1, 40.0, 0.01, 1.0)
    assert all(abs(a - b) < 1e-7 for a, b in zip(got, want))
    assert hp.term_denom == 200 and hp.precision == pb.FP32
    assert hp.algorithm == pb.ALGO_A2C and abs(hp.epsilon - 0.1) < 1e-7


def test_workspace_sizing_and_argument_checks():
    hp = pb.default_hparams(precision=pb.BF16)
    big = pb.workspace_bytes(pb.ARCH_NATURE, 1024, 5, 18, hp)
    small = pb.workspace_bytes(pb.ARCH_NATURE, 32, 5, 18, hp)
    assert 0 < small < big < 4 << 30
    frames = 2 * 5 * 1024 * 84 * 84 * 4
    assert big > frames
    assert pb.workspace_bytes(2, 32, 5, 18, hp) == 0
    assert pb.workspace_bytes(pb.ARCH_NIPS, 0, 5, 4, hp) == 0
    assert pb.workspace_bytes(pb.ARCH_NIPS, 4, 0, 4, hp) == 0
    assert pb.workspace_bytes(pb.ARCH_NIPS, 4, 5, 33, hp) == 0
    assert pb.workspace_bytes(pb.ARCH_NIPS, 4, 5, 4, pb.default_hparams(term_denom=0)) == 0
    assert pb.workspace_bytes(pb.ARCH_NIPS, 4, 5, 4, pb.default_hparams(precision=5)) == 0


def test_null_handles_and_strerror():
    L = pb.lib()
    assert L.paac_rollout(None, None) == pb.ERR_ARG
    assert L.paac_update(None, None) == pb.ERR_ARG
    assert L.paac_destroy(None) == pb.ERR_ARG
    assert L.paac_param_count(None) == 0 and L.paac_debug_bytes(None, 0) == 0
    names = {L.paac_strerror(i) for i in range(9)}
    assert len(names) == 9 and L.paac_strerror(99) == b"unknown status"


def test_init_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        return
    L = pb.lib()
    h = C.c_void_p()
    hp = pb.default_hparams()
    assert L.paac_init(C.byref(h), pb.ARCH_NIPS, 4, 5, 4, C.byref(hp), 1) == pb.ERR_CUDA
    assert not h.value
