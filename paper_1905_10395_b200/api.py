"""ctypes binding of include/lsgd.h.  Argument marshalling only: every step of the LSGD path runs in
the CUDA library.  There is no CPU fallback; a missing library is an ImportError-like failure."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblsgd.so")

(OK, ERR_INVALID_ARG, ERR_BAD_GROUPS, ERR_ALIGNMENT, ERR_STATE, ERR_CUDA, ERR_UNSUPPORTED, ERR_DEVICE_FLAG,
 ERR_TOO_LARGE) = range(9)
OBJ_EXTERNAL, OBJ_QUADRATIC, OBJ_MATCOMP, OBJ_MLP, OBJ_PSD_COMPLETION = range(5)
ARITH_FP64, ARITH_FP64_FMA, ARITH_FP32 = range(3)
FLAG_MLP_FUSED_STEP = 1
FLAG_ALGORITHM1 = 2
FLAG_MATCOMP_FUSED_STEP = 4
FLAG_EAGD = 8
# bits of the device status word (lsgd_check_device)
DEVFLAG_BAD_LEADER, DEVFLAG_WAIT_TIMEOUT, DEVFLAG_BAD_INDEX, DEVFLAG_OVERFLOW = 1, 2, 4, 8


class LsgdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (lsgd_status {status})")


class QuadraticDesc(C.Structure):
    _fields_ = [("a", C.c_void_p), ("b", C.c_void_p), ("sigma", C.c_float)]


class MatcompDesc(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("n_cols", C.c_int32), ("rank", C.c_int32), ("n_obs", C.c_int32),
                ("obs_r", C.c_void_p), ("obs_c", C.c_void_p), ("obs_v", C.c_void_p), ("batch", C.c_int32),
                ("n_heldout", C.c_int32), ("heldout_pos", C.c_void_p), ("scratch", C.c_void_p),
                ("scratch_bytes", C.c_uint64)]


class PsdDesc(C.Structure):
    _fields_ = [("n", C.c_int32), ("r", C.c_int32), ("M", C.c_void_p), ("scratch", C.c_void_p),
                ("scratch_bytes", C.c_uint64)]


class MlpDesc(C.Structure):
    _fields_ = [("dims", C.c_int32 * 4), ("batch", C.c_int32), ("pool", C.c_int32), ("pool_x", C.c_void_p),
                ("pool_y", C.c_void_p), ("n_heldout", C.c_int32), ("held_x", C.c_void_p), ("held_y", C.c_void_p),
                ("scratch", C.c_void_p), ("scratch_bytes", C.c_uint64), ("loss_window", C.c_int32)]


class BgemmDesc(C.Structure):
    _fields_ = [("a", C.c_void_p), ("b", C.c_void_p), ("c", C.c_void_p), ("M", C.c_int32), ("N", C.c_int32),
                ("K", C.c_int32), ("batch", C.c_int32), ("a_mn_major", C.c_int32), ("b_mn_major", C.c_int32),
                ("lda", C.c_int64), ("ldb", C.c_int64), ("ldc", C.c_int64), ("stride_a", C.c_int64),
                ("stride_b", C.c_int64), ("stride_c", C.c_int64), ("epilogue", C.c_int32), ("bias", C.c_void_p),
                ("stride_bias", C.c_int64), ("mask", C.c_void_p), ("ld_mask", C.c_int64), ("stride_mask", C.c_int64)]


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("P", C.c_int32), ("G", C.c_int32), ("group_of", C.c_void_p),
                ("d", C.c_int64), ("ld", C.c_int64), ("eta", C.c_float), ("lambda_l", C.c_float),
                ("lambda_g", C.c_float), ("tau", C.c_int32), ("objective", C.c_int32),
                ("objective_desc", C.c_void_p), ("x", C.c_void_p), ("g", C.c_void_p), ("stream", C.c_void_p),
                ("arithmetic", C.c_int32), ("flags", C.c_uint32), ("gamma_l", C.c_float), ("gamma_g", C.c_float),
                ("tau_g", C.c_int32), ("leader_copies", C.c_void_p), ("v", C.c_void_p), ("momentum", C.c_float),
                ("weight_decay", C.c_float)]


_lib = None


def lib() -> C.CDLL:
    """Loads liblsgd.so (built in-tree by paper_1905_10395_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1905_10395_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        H = C.c_void_p
        L.lsgd_create.argtypes = [C.POINTER(Config), C.POINTER(H)]
        L.lsgd_grad.argtypes = [H, C.c_void_p]
        L.lsgd_elect.argtypes = [H, C.c_void_p]
        L.lsgd_step.argtypes = [H]
        L.lsgd_destroy.argtypes = [H]
        L.lsgd_get_leaders.argtypes = [H, C.c_void_p, C.c_void_p]
        L.lsgd_get_loss.argtypes = [H, C.c_void_p]
        L.lsgd_set_leaders.argtypes = [H, C.c_void_p, C.c_int32]
        L.lsgd_set_leaders.restype = C.c_int
        L.lsgd_get_train_loss.argtypes = [H, C.c_void_p]
        L.lsgd_get_train_loss.restype = C.c_int
        L.lsgd_center.argtypes = [H, C.c_void_p]
        L.lsgd_center.restype = C.c_int
        L.lsgd_advance_step.argtypes = [H, C.c_int64]
        L.lsgd_advance_step.restype = C.c_int
        L.lsgd_sync_parameters.argtypes = [H]
        L.lsgd_sync_parameters.restype = C.c_int
        L.lsgd_get_step.argtypes = [H, C.POINTER(C.c_int64)]
        L.lsgd_get_leader_counts.argtypes = [H, C.c_void_p, C.c_void_p]
        L.lsgd_check_device.argtypes = [H, C.POINTER(C.c_uint32)]
        L.lsgd_set_eta.argtypes = [H, C.c_float]
        L.lsgd_shard_best_key.argtypes = [H, C.c_int32, C.c_void_p, C.c_void_p]
        L.lsgd_shard_best_key.restype = C.c_int
        L.lsgd_shard_pick_global.argtypes = [H, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.lsgd_shard_pick_global.restype = C.c_int
        L.lsgd_mlp_get_activations.argtypes = [H, C.c_void_p, C.c_void_p]
        L.lsgd_mlp_get_activations.restype = C.c_int
        L.lsgd_selftest_wait_timeout.argtypes = [H, C.c_int32, C.c_int64, C.POINTER(C.c_int32)]
        L.lsgd_selftest_wait_timeout.restype = C.c_int
        L.lsgd_bgemm_check_device.argtypes = [C.POINTER(C.c_uint32)]
        L.lsgd_bgemm_check_device.restype = C.c_int
        L.lsgd_quadratic_loss_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int64,
                                                  C.c_void_p, C.c_void_p]
        L.lsgd_quadratic_loss_noalloc.restype = C.c_int
        L.lsgd_bgemm_bf16.argtypes = [C.POINTER(BgemmDesc), C.c_void_p]
        L.lsgd_bgemm_bf16.restype = C.c_int
        L.lsgd_status_string.argtypes = [C.c_int]
        L.lsgd_status_string.restype = C.c_char_p
        L.lsgd_mlp_param_offsets.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int64)]
        L.lsgd_mlp_scratch_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32]
        L.lsgd_mlp_scratch_bytes.restype = C.c_uint64
        L.lsgd_matcomp_scratch_bytes.argtypes = [C.c_int32, C.c_int64]
        L.lsgd_matcomp_scratch_bytes.restype = C.c_uint64
        L.lsgd_psd_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int64]
        L.lsgd_psd_scratch_bytes.restype = C.c_uint64
        for name in ("lsgd_create", "lsgd_grad", "lsgd_elect", "lsgd_step", "lsgd_destroy", "lsgd_get_leaders",
                     "lsgd_get_loss", "lsgd_get_step", "lsgd_get_leader_counts", "lsgd_check_device",
                     "lsgd_set_eta", "lsgd_mlp_param_offsets"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(s: int) -> str:
    return lib().lsgd_status_string(int(s)).decode()


def _check(s: int, where: str) -> None:
    if s != OK:
        raise LsgdError(s, where)


def _ptr(t) -> Optional[int]:
    """Device pointer of a torch tensor (or a raw int / None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


# ---- the five entry points, same names as the C ABI -------------------------------------------------
def lsgd_create(cfg: Config) -> C.c_void_p:
    h = C.c_void_p()
    _check(lib().lsgd_create(C.byref(cfg), C.byref(h)), "lsgd_create")
    return h


def lsgd_grad(h, batch=None) -> None:
    _check(lib().lsgd_grad(h, _ptr(batch)), "lsgd_grad")


def lsgd_elect(h, loss=None) -> None:
    _check(lib().lsgd_elect(h, _ptr(loss)), "lsgd_elect")


def lsgd_step(h) -> None:
    _check(lib().lsgd_step(h), "lsgd_step")


def lsgd_destroy(h) -> None:
    _check(lib().lsgd_destroy(h), "lsgd_destroy")


def lsgd_quadratic_loss_noalloc(x, a, b, P: int, d: int, ld: int, loss, stream: int = 0) -> None:
    """Election loss of the quadratic objective without any device allocation (fixed 512 KiB scratch
    inside the library; P * ceil(d / 8192) <= 65536).  For callers that may not allocate."""
    _check(lib().lsgd_quadratic_loss_noalloc(_ptr(x), _ptr(a), _ptr(b), int(P), int(d), int(ld), _ptr(loss),
                                             stream or None), "lsgd_quadratic_loss_noalloc")


def lsgd_bgemm_bf16(desc: BgemmDesc, stream: int = 0) -> None:
    _check(lib().lsgd_bgemm_bf16(C.byref(desc), stream or None), "lsgd_bgemm_bf16")


def lsgd_bgemm_check_device() -> int:
    """Status word of lsgd_bgemm_bf16 on the current device (read and cleared); 0 = no kernel reported anything."""
    f = C.c_uint32()
    s = lib().lsgd_bgemm_check_device(C.byref(f))
    if s not in (OK, ERR_DEVICE_FLAG):
        raise LsgdError(s, "lsgd_bgemm_check_device")
    return f.value


def mlp_param_offsets(dims: Sequence[int]):
    d4 = (C.c_int32 * 4)(*dims)
    w = (C.c_int64 * 3)()
    b = (C.c_int64 * 3)()
    d = C.c_int64()
    _check(lib().lsgd_mlp_param_offsets(d4, w, b, C.byref(d)), "lsgd_mlp_param_offsets")
    return list(w), list(b), d.value


def mlp_scratch_bytes(dims: Sequence[int], P: int, batch: int, n_heldout: int) -> int:
    d4 = (C.c_int32 * 4)(*dims)
    return int(lib().lsgd_mlp_scratch_bytes(d4, P, batch, n_heldout))


def matcomp_scratch_bytes(P: int, ld: int) -> int:
    return int(lib().lsgd_matcomp_scratch_bytes(int(P), int(ld)))


def psd_scratch_bytes(r: int, P: int, ld: int) -> int:
    return int(lib().lsgd_psd_scratch_bytes(int(r), int(P), int(ld)))


def make_config(*, P: int, G: int, group_of: np.ndarray, d: int, ld: int, eta: float, lambda_l: float,
                lambda_g: float, tau: int, objective: int, desc=None, x=None, g=None, stream: int = 0,
                arithmetic: int = ARITH_FP64, flags: int = 0, gamma_l: float = 0.0, gamma_g: float = 0.0,
                tau_g: int = 1, leader_copies=None, v=None, momentum: float = 0.0, weight_decay: float = 0.0):
    """Returns (Config, keepalive) -- keepalive holds the host arrays the struct points to."""
    go = np.ascontiguousarray(group_of, dtype=np.int32)
    cfg = Config()
    cfg.struct_size = C.sizeof(Config)
    cfg.P, cfg.G = int(P), int(G)
    cfg.group_of = go.ctypes.data
    cfg.d, cfg.ld = int(d), int(ld)
    cfg.eta, cfg.lambda_l, cfg.lambda_g = float(eta), float(lambda_l), float(lambda_g)
    cfg.tau = int(tau)
    cfg.objective = int(objective)
    cfg.objective_desc = C.addressof(desc) if desc is not None else None
    cfg.x = _ptr(x)
    cfg.g = _ptr(g)
    cfg.stream = stream or None
    cfg.arithmetic = int(arithmetic)
    cfg.flags = int(flags)
    cfg.gamma_l, cfg.gamma_g, cfg.tau_g = float(gamma_l), float(gamma_g), int(tau_g)
    cfg.leader_copies = _ptr(leader_copies)
    cfg.v = _ptr(v)
    cfg.momentum, cfg.weight_decay = float(momentum), float(weight_decay)
    return cfg, (go, desc)


class Lsgd:
    """Thin owner of one handle.  Tensors passed in must outlive it (the library never copies them)."""

    def __init__(self, cfg: Config, keepalive=()):
        self._keep = keepalive
        self.P, self.G = cfg.P, cfg.G
        self.h = lsgd_create(cfg)

    def grad(self, batch=None):
        lsgd_grad(self.h, batch)

    def elect(self, loss=None):
        lsgd_elect(self.h, loss)

    def step(self):
        lsgd_step(self.h)

    def leaders(self):
        ll = np.empty(self.G, dtype=np.int32)
        gl = np.empty(1, dtype=np.int32)
        _check(lib().lsgd_get_leaders(self.h, ll.ctypes.data, gl.ctypes.data), "lsgd_get_leaders")
        return ll, int(gl[0])

    def set_leaders(self, local_leaders=None, global_leader: int = -1):
        ll = None if local_leaders is None else np.ascontiguousarray(local_leaders, dtype=np.int32)
        _check(lib().lsgd_set_leaders(self.h, None if ll is None else ll.ctypes.data, int(global_leader)),
               "lsgd_set_leaders")

    def shard_best_key(self, n_own: int, global_index, key_out):
        """key_out (device int64[1]) <- this device's best own worker as a cross-device election key."""
        _check(lib().lsgd_shard_best_key(self.h, int(n_own), _ptr(global_index), _ptr(key_out)), "lsgd_shard_best_key")

    def shard_pick_global(self, keys, world: int, my_rank: int, guest_row: int):
        """(winning rank, winner's global worker index, this device's best own worker) from all devices' keys."""
        out = np.empty(3, dtype=np.int32)
        _check(lib().lsgd_shard_pick_global(self.h, _ptr(keys), int(world), int(my_rank), int(guest_row), out.ctypes.data),
               "lsgd_shard_pick_global")
        return int(out[0]), int(out[1]), int(out[2])

    def loss(self):
        out = np.empty(self.P, dtype=np.float32)
        _check(lib().lsgd_get_loss(self.h, out.ctypes.data), "lsgd_get_loss")
        return out

    def train_loss(self):
        out = np.empty(self.P, dtype=np.float32)
        _check(lib().lsgd_get_train_loss(self.h, out.ctypes.data), "lsgd_get_train_loss")
        return out

    def mlp_activations(self, batch: int, d1: int, d2: int):
        """Hidden activations stored by the last grad() of the MLP objective, as float32 [P, batch, d1] / [.., d2]
        (the library holds them as bf16; widening is exact)."""
        h1 = np.empty((self.P, batch, d1), dtype=np.uint16)
        h2 = np.empty((self.P, batch, d2), dtype=np.uint16)
        _check(lib().lsgd_mlp_get_activations(self.h, h1.ctypes.data, h2.ctypes.data), "lsgd_mlp_get_activations")
        widen = lambda a: (a.astype(np.uint32) << 16).view(np.float32)
        return widen(h1), widen(h2)

    def center(self, out):
        """out (device float[ld]) <- average of all workers' parameters (the paper's center variable)."""
        _check(lib().lsgd_center(self.h, _ptr(out)), "lsgd_center")

    def advance_step(self, n: int):
        _check(lib().lsgd_advance_step(self.h, int(n)), "lsgd_advance_step")

    def sync_parameters(self):
        _check(lib().lsgd_sync_parameters(self.h), "lsgd_sync_parameters")

    def t(self) -> int:
        v = C.c_int64()
        _check(lib().lsgd_get_step(self.h, C.byref(v)), "lsgd_get_step")
        return v.value

    def leader_counts(self):
        cg = np.empty(self.P, dtype=np.int32)
        cl = np.empty(self.P, dtype=np.int32)
        _check(lib().lsgd_get_leader_counts(self.h, cg.ctypes.data, cl.ctypes.data), "lsgd_get_leader_counts")
        return cg, cl

    def check_device(self) -> int:
        f = C.c_uint32()
        s = lib().lsgd_check_device(self.h, C.byref(f))
        if s not in (OK, ERR_DEVICE_FLAG):
            raise LsgdError(s, "lsgd_check_device")
        return f.value

    def selftest_wait_timeout(self, budget_cycles: int, which: int = 0) -> int:
        """Runs a pipeline's bounded wait (which = 0: update kernels, 1: product kernels) on a barrier nothing
        completes; 1 if the wait ran out."""
        out = C.c_int32(-1)
        _check(lib().lsgd_selftest_wait_timeout(self.h, int(which), int(budget_cycles), C.byref(out)),
               "lsgd_selftest_wait_timeout")
        return out.value

    def set_eta(self, eta: float):
        _check(lib().lsgd_set_eta(self.h, eta), "lsgd_set_eta")

    def destroy(self):
        if self.h is not None:
            h, self.h = self.h, None
            lsgd_destroy(h)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
