"""Thin ctypes binding of libpaac_b200.so: argument marshalling only.

Every step of the PAAC iteration runs in the library's CUDA kernels; this module
allocates nothing but host result buffers and (through torch) the device workspace.
If the shared library is missing or cannot be loaded the import of `lib()` raises:
there is no other implementation to fall back to.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpaac_b200.so")

ARCH_NIPS, ARCH_NATURE = 0, 1
FP32, BF16 = 0, 1
ALGO_A2C, ALGO_NSTEP_Q = 0, 1
ENV_HASHED, ENV_PATTERN = 0, 1
OK, ERR_ARG, ERR_WORKSPACE, ERR_CUDA, ERR_NONFINITE, ERR_TIMEOUT, ERR_STATE, ERR_LIMIT, ERR_RANGE = range(9)
(DBG_FRAMES, DBG_NEXT_FRAMES, DBG_ACTIONS, DBG_REWARDS, DBG_TERMINALS, DBG_VALUES, DBG_LOGITS, DBG_UNIFORMS,
 DBG_COUNTERS, DBG_RETURNS, DBG_ADVANTAGES, DBG_DLOGITS, DBG_DVALUES, DBG_GRAD, DBG_RMS, DBG_SAMPLED,
 DBG_ERROR_WORD) = range(17)
DBG_ACT0, DBG_GACT0 = 32, 48
(OPT_CUDA_CORES_ONLY, OPT_TC_WGRAD_LAYERS, OPT_CUDA_GRAPHS, OPT_DEPENDENT_LAUNCH, OPT_FP32_TENSOR_CORES,
 OPT_UPDATE_CHUNKS) = 1, 2, 3, 4, 5, 6

_DBG_DTYPE = {DBG_FRAMES: np.uint8, DBG_NEXT_FRAMES: np.uint8, DBG_ACTIONS: np.int32, DBG_REWARDS: np.int8,
              DBG_TERMINALS: np.uint8, DBG_COUNTERS: np.int32, DBG_SAMPLED: np.int32, DBG_ERROR_WORD: np.uint32}


class HParams(C.Structure):
    _fields_ = [("gamma", C.c_float), ("lr", C.c_float), ("rms_decay", C.c_float), ("rms_eps", C.c_float),
                ("clip_norm", C.c_float), ("entropy_beta", C.c_float), ("value_coef", C.c_float),
                ("term_denom", C.c_uint32), ("precision", C.c_int), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p), ("algorithm", C.c_int),
                ("epsilon", C.c_float), ("environment", C.c_int)]


class RolloutView(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("frames", "next_frames", "actions", "rewards", "terminals", "values",
                                          "logits", "uniforms")]


class UpdateStats(C.Structure):
    _fields_ = [("policy_loss", C.c_float), ("value_loss", C.c_float), ("entropy", C.c_float),
                ("grad_norm", C.c_float), ("clip_scale", C.c_float), ("status", C.c_int32),
                ("timesteps", C.c_uint64)]


EXPORTS = ["paac_default_hparams", "paac_workspace_bytes", "paac_init", "paac_rollout", "paac_update",
           "paac_param_count", "paac_params", "paac_destroy", "paac_strerror", "paac_act_host",
           "paac_observe_host", "paac_set_params", "paac_force_actions", "paac_debug_bytes", "paac_debug_read",
           "paac_debug_write", "paac_debug_wait_probe", "paac_preprocess", "paac_stack_push", "paac_act_host_newest", "paac_launch_count", "paac_profile", "paac_profile_read", "paac_set_option", "paac_clip_rmsprop_noalloc",
           "paac_noalloc_max_params"]

_lib = None


def lib():
    """The loaded library; raises OSError if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError("libpaac_b200.so is not built: run `python -m paper_1705_04862_b200.build` "
                          "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
        L.paac_default_hparams.argtypes = [C.POINTER(HParams)]
        L.paac_default_hparams.restype = None
        L.paac_workspace_bytes.argtypes = [i, i, i, i, C.POINTER(HParams)]
        L.paac_workspace_bytes.restype = sz
        L.paac_init.argtypes = [C.POINTER(vp), i, i, i, i, C.POINTER(HParams), u64]
        L.paac_rollout.argtypes = [vp, C.POINTER(RolloutView)]
        L.paac_update.argtypes = [vp, C.POINTER(UpdateStats)]
        L.paac_param_count.argtypes = [vp]
        L.paac_param_count.restype = sz
        L.paac_params.argtypes = [vp, vp, sz]
        L.paac_destroy.argtypes = [vp]
        L.paac_strerror.argtypes = [i]
        L.paac_strerror.restype = C.c_char_p
        L.paac_act_host.argtypes = [vp, i, vp, vp, vp]
        L.paac_observe_host.argtypes = [vp, i, vp, vp]
        L.paac_set_params.argtypes = [vp, vp, sz]
        L.paac_force_actions.argtypes = [vp, vp]
        L.paac_debug_bytes.argtypes = [vp, i]
        L.paac_debug_bytes.restype = sz
        L.paac_debug_read.argtypes = [vp, i, vp, sz]
        L.paac_debug_write.argtypes = [vp, i, vp, sz]
        L.paac_debug_wait_probe.argtypes = [vp, C.c_uint32]
        L.paac_preprocess.argtypes = [vp, vp, vp, vp, i, vp]
        L.paac_stack_push.argtypes = [vp, vp, vp, vp, i, vp]
        L.paac_act_host_newest.argtypes = [vp, i, vp, vp, vp, vp]
        L.paac_launch_count.argtypes = [vp]
        L.paac_launch_count.restype = u64
        L.paac_profile.argtypes = [vp, i]
        L.paac_set_option.argtypes = [vp, i, i]
        f = C.c_float
        L.paac_clip_rmsprop_noalloc.argtypes = [vp, vp, vp, vp, sz, f, f, f, f, vp, vp]
        L.paac_noalloc_max_params.argtypes = []
        L.paac_noalloc_max_params.restype = sz
        L.paac_profile_read.argtypes = [vp, i, C.POINTER(C.c_char_p), C.POINTER(C.c_double), C.POINTER(u64)]
        _lib = L
    return _lib


class PaacError(RuntimeError):
    def __init__(self, status):
        self.status = status
        super().__init__("paac: %s (status %d)" % (lib().paac_strerror(status).decode(), status))


def _check(status, allow=()):
    if status != OK and status not in allow:
        raise PaacError(status)
    return status


def default_hparams(**over):
    hp = HParams()
    lib().paac_default_hparams(C.byref(hp))
    for k, v in over.items():
        setattr(hp, k, v)
    return hp


def workspace_bytes(arch, n_e, t_max, n_actions, hp):
    return int(lib().paac_workspace_bytes(arch, n_e, t_max, n_actions, C.byref(hp)))


def _host_ptr(a):
    """Address of a numpy array or a (pinned) CPU torch tensor."""
    if isinstance(a, np.ndarray):
        assert a.flags["C_CONTIGUOUS"]
        return a.ctypes.data
    return a.data_ptr()


def clip_rmsprop_noalloc(theta, rms, grad, n, lr, rms_decay, rms_eps, clip_norm, theta_bf16=None,
                         norm_and_scale=None, stream=None):
    """Optimiser step on caller-owned device arrays for hosts that may not allocate device memory (see
    paac_clip_rmsprop_noalloc in include/paac.h).  Arguments are torch CUDA tensors (or raw device
    addresses); returns the library status without raising, so callers can test for ERR_LIMIT."""
    def addr(x):
        return None if x is None else (x if isinstance(x, int) else x.data_ptr())
    return int(lib().paac_clip_rmsprop_noalloc(addr(theta), addr(rms), addr(grad), addr(theta_bf16), n, lr, rms_decay,
                                               rms_eps, clip_norm, addr(norm_and_scale), addr(stream)))


def preprocess(raw_prev, raw_last, state_in, state_out, n, stream=None):
    """Section 5.1 pre-processing on device buffers (torch CUDA uint8 tensors or raw addresses): see paac_preprocess
    in include/paac.h.  Returns the library status."""
    def addr(x):
        return None if x is None else (x if isinstance(x, int) else x.data_ptr())
    return int(lib().paac_preprocess(addr(raw_prev), addr(raw_last), addr(state_in), addr(state_out), n, addr(stream)))


def stack_push(state_in, newest, restart, state_out, n, stream=None):
    """The four-frame stack on device buffers: see paac_stack_push in include/paac.h.  Returns the library status."""
    def addr(x):
        return None if x is None else (x if isinstance(x, int) else x.data_ptr())
    return int(lib().paac_stack_push(addr(state_in), addr(newest), addr(restart), addr(state_out), n, addr(stream)))


class Paac:
    """One learner.  The device workspace is a torch uint8 tensor on `device`; kernels run on
    torch's current stream at construction time."""

    def __init__(self, arch, n_e, t_max, n_actions, seed, precision=FP32, device="cuda:0", **hparams):
        import torch
        L = lib()
        self.arch = {"nips": ARCH_NIPS, "nature": ARCH_NATURE}.get(arch, arch)
        self.n_e, self.t_max, self.A, self.seed, self.precision = n_e, t_max, n_actions, seed, precision
        self.B = n_e * t_max
        self.hp = default_hparams(precision=precision, **hparams)
        need = workspace_bytes(self.arch, n_e, t_max, n_actions, self.hp)
        if need == 0:
            raise PaacError(ERR_ARG)
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self._ws = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
            base = (self._ws.data_ptr() + 255) // 256 * 256
            self.hp.workspace, self.hp.workspace_bytes = base, need
            self._stream = torch.cuda.current_stream(self.device)
            self.hp.stream = self._stream.cuda_stream
            h = C.c_void_p()
            _check(L.paac_init(C.byref(h), self.arch, n_e, t_max, n_actions, C.byref(self.hp), seed))
        self._h = h
        self.P = int(L.paac_param_count(h))

    # -- Algorithm 1 ------------------------------------------------------------------------
    def rollout(self):
        v = RolloutView()
        _check(lib().paac_rollout(self._h, C.byref(v)))
        return v

    def update(self, sync=True):
        if not sync:
            _check(lib().paac_update(self._h, None))
            return None
        s = UpdateStats()
        _check(lib().paac_update(self._h, C.byref(s)), allow=(ERR_NONFINITE, ERR_TIMEOUT, ERR_RANGE))
        return {n: getattr(s, n) for n, _ in UpdateStats._fields_}

    def params(self):
        out = np.empty(self.P, np.float32)
        _check(lib().paac_params(self._h, out.ctypes.data, self.P))
        return out

    # -- external environments -----------------------------------------------------------------
    def act_host(self, t, frames, actions=None, values=None):
        _check(lib().paac_act_host(self._h, t, _host_ptr(frames) if frames is not None else None,
                                   _host_ptr(actions) if actions is not None else None,
                                   _host_ptr(values) if values is not None else None))

    def act_host_newest(self, t, newest, restart=None, actions=None, values=None):
        _check(lib().paac_act_host_newest(self._h, t, _host_ptr(newest), _host_ptr(restart) if restart is not None else None,
                                          _host_ptr(actions) if actions is not None else None,
                                          _host_ptr(values) if values is not None else None))

    def observe_host(self, t, rewards, terminals):
        _check(lib().paac_observe_host(self._h, t, _host_ptr(rewards), _host_ptr(terminals)))

    # -- hooks ---------------------------------------------------------------------------------
    def set_params(self, theta):
        theta = np.ascontiguousarray(theta, np.float32)
        _check(lib().paac_set_params(self._h, theta.ctypes.data, theta.size))

    def force_actions(self, actions):
        if actions is None:
            _check(lib().paac_force_actions(self._h, None))
            return
        a = np.ascontiguousarray(actions, np.int32)
        assert a.size == self.B
        _check(lib().paac_force_actions(self._h, a.ctypes.data))

    def debug_read(self, which):
        """Tensor `which` as a flat numpy array (bf16 tensors are widened to float32)."""
        n = int(lib().paac_debug_bytes(self._h, which))
        if n == 0:
            raise PaacError(ERR_ARG)
        raw = np.empty(n, np.uint8)
        _check(lib().paac_debug_read(self._h, which, raw.ctypes.data, n))
        if which in _DBG_DTYPE:
            return raw.view(_DBG_DTYPE[which])
        if which >= DBG_ACT0 and self.precision == BF16:
            return (raw.view(np.uint16).astype(np.uint32) << 16).view(np.float32)
        return raw.view(np.float32)

    def debug_write(self, which, arr):
        arr = np.ascontiguousarray(arr)
        _check(lib().paac_debug_write(self._h, which, arr.ctypes.data, arr.nbytes))

    def debug_write_act(self, layer, arr):
        """Overwrite stored activation `layer` from float32 values (which, with bf16 storage, must
        already be bf16-representable)."""
        arr = np.ascontiguousarray(arr, np.float32)
        if self.precision == BF16:
            bits = arr.view(np.uint32)
            assert not np.any(bits & 0xFFFF), "not bf16 values"
            arr = (bits >> 16).astype(np.uint16)
        self.debug_write(DBG_ACT0 + layer, arr)

    def error_word(self):
        """The sticky device error bits (0 when every kernel so far ran to the end)."""
        w = np.zeros(1, np.uint32)
        lib().paac_debug_read(self._h, DBG_ERROR_WORD, w.ctypes.data, 4)      # the status only repeats the word
        return int(w[0])

    def clear_error_word(self):
        self.debug_write(DBG_ERROR_WORD, np.zeros(1, np.uint32))

    def wait_probe(self, max_polls):
        """Status of a wait that is made to run out (ERR_TIMEOUT when the device-side bound works)."""
        return int(lib().paac_debug_wait_probe(self._h, max_polls))

    def launch_count(self):
        return int(lib().paac_launch_count(self._h))

    def set_option(self, option, value):
        _check(lib().paac_set_option(self._h, option, value))

    def profile(self, enable):
        _check(lib().paac_profile(self._h, 1 if enable else 0))

    def profile_read(self):
        """{kernel family: (device ms, launches)} since profiling was enabled."""
        n = 64
        names, ms, cnt = (C.c_char_p * n)(), (C.c_double * n)(), (C.c_uint64 * n)()
        k = lib().paac_profile_read(self._h, n, names, ms, cnt)
        if k < 0:
            raise PaacError(ERR_ARG)
        return {names[j].decode(): (ms[j], int(cnt[j])) for j in range(k)}

    def close(self):
        if getattr(self, "_h", None):
            lib().paac_destroy(self._h)
            self._h = None
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
