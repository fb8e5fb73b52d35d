"""Thin Python binding of the C ABI in ``include/baoc.h``.

Argument marshalling only: every step of the path runs in the CUDA library.
PyTorch supplies device memory and the stream.  The names follow the C entry
points (``baoc_create`` -> ``Baoc(...)``, ``baoc_sample_stats`` ->
``Baoc.sample_stats`` and so on).  There is no CPU fallback: if the shared
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# BAOC_CHECKED=1 in the environment selects the checked build of the library (in-kernel validation of every tile and
# range, see include/baoc.h); it is a different file, so the choice is made once, at import
CHECKED = os.environ.get("BAOC_CHECKED", "") == "1"
LIB_PATH = os.path.join(_HERE, "libbaoc_checked.so" if CHECKED else "libbaoc.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build the CUDA library first "
        "(python -m paper_2605_04711_b200.build [--checked]); there is no fallback path")

_lib = C.CDLL(LIB_PATH)

OK, E_INVALID, E_ALIGN, E_STATE, E_INFEASIBLE, E_CUDA, E_NONFINITE, E_WORKSPACE = 0, -1, -2, -3, -4, -5, -6, -7
W_NODE_LIMIT = 1


class BaocError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"baoc error {code}: {msg}")
        self.code = code


class Block(C.Structure):
    _fields_ = [("numel", C.c_int64), ("rows", C.c_int32), ("cols", C.c_int32)]


class Config(C.Structure):
    _fields_ = [("adaptive", C.c_uint8), ("momentum", C.c_uint8), ("decoupled_wd", C.c_uint8),
                ("factored", C.c_uint8), ("bits", C.c_uint8), ("quantizer", C.c_uint8), ("af_flags", C.c_uint8),
                ("reserved", C.c_uint8),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float)]


class Opts(C.Structure):
    _fields_ = [("beta_m", C.c_double), ("beta_v", C.c_double), ("beta_rho", C.c_double), ("eps", C.c_double),
                ("a_lo", C.c_double), ("a_hi", C.c_double), ("rho_lo", C.c_double), ("rho_hi", C.c_double),
                ("snr_lo", C.c_double), ("snr_hi", C.c_double), ("w", C.c_double * 5), ("gamma", C.c_double),
                ("eps_adam", C.c_double), ("use_snr", C.c_int32), ("qblock", C.c_int32), ("node_limit", C.c_int64),
                ("quantizer8", C.c_int32), ("debias", C.c_int32)]


class BlockStats(C.Structure):
    _fields_ = [(n, C.c_double) for n in
                ("A", "rho_bar", "snr", "C", "F", "Q32", "Q16", "Q8", "q10", "q90", "rho_mom",
                 "err_m8", "err_v8", "err_m16", "err_v16",
                 "s_A", "s_rho", "s_snr", "s_M", "C_tilde", "s_F", "lQ32", "lQ16", "lQ8", "last_cos")] + \
               [("n_cos", C.c_int64)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class Check(C.Structure):
    _fields_ = [("enabled", C.c_int32), ("code", C.c_uint32), ("kernel", C.c_uint32), ("reserved", C.c_int32),
                ("a", C.c_int64), ("b", C.c_int64), ("c", C.c_int64), ("d", C.c_int64)]


class Sample(C.Structure):
    _fields_ = [("n_rows", C.c_int64), ("n_cols", C.c_int32), ("rows", C.c_void_p), ("cols", C.c_void_p)]


class Info(C.Structure):
    _fields_ = [("n_blocks", C.c_int32), ("n_cfg", C.c_int32), ("numel", C.c_int64), ("n_tiles", C.c_int64),
                ("stats_steps", C.c_int64), ("state_bytes", C.c_int64), ("kernel_launches", C.c_int64),
                ("stats_bytes_per_call", C.c_int64), ("step_bytes_per_call", C.c_int64), ("select_retries", C.c_int64)]


EXPORTS = ["baoc_default_opts", "baoc_create", "baoc_destroy", "baoc_last_error", "baoc_query",
           "baoc_stats_workspace_bytes", "baoc_bind_stats_workspace", "baoc_sample_stats", "baoc_read_stats",
           "baoc_risk", "baoc_risk_from_raw", "baoc_cost_model", "baoc_allocate", "baoc_state_bytes",
           "baoc_configure", "baoc_step", "baoc_step_from_host", "baoc_view", "baoc_nonfinite",
           "baoc_sample_stats_noalloc", "baoc_noalloc_last_error", "baoc_profile", "baoc_profile_last",
           "baoc_export", "baoc_import", "baoc_time_scratch_bytes", "baoc_measure_time_ratios",
           "baoc_set_sampling", "baoc_reconfigure", "baoc_configure_from_window", "baoc_partition",
           "baoc_set_factored_schedule", "baoc_check_status", "baoc_check_selftest"]

_vp = C.c_void_p
_lib.baoc_default_opts.argtypes = [C.POINTER(Opts)]
_lib.baoc_default_opts.restype = None
_lib.baoc_create.argtypes = [C.POINTER(_vp), C.c_int, C.POINTER(Block), C.c_int, C.POINTER(Config), C.POINTER(Opts)]
_lib.baoc_destroy.argtypes = [_vp]
_lib.baoc_destroy.restype = None
_lib.baoc_last_error.argtypes = [_vp]
_lib.baoc_last_error.restype = C.c_char_p
_lib.baoc_query.argtypes = [_vp, C.POINTER(Info)]
_lib.baoc_stats_workspace_bytes.argtypes = [_vp, C.POINTER(C.c_size_t)]
_lib.baoc_bind_stats_workspace.argtypes = [_vp, _vp, C.c_size_t, _vp]
_lib.baoc_sample_stats.argtypes = [_vp, _vp, _vp]
_lib.baoc_read_stats.argtypes = [_vp, C.POINTER(BlockStats), _vp]
_lib.baoc_risk.argtypes = [_vp, _vp, _vp, C.POINTER(BlockStats), _vp]
_lib.baoc_risk_from_raw.argtypes = [_vp, C.POINTER(BlockStats), _vp]
_lib.baoc_cost_model.argtypes = [_vp, _vp, _vp]
_lib.baoc_allocate.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, C.c_double, _vp, _vp, _vp, C.POINTER(C.c_double)]
_lib.baoc_state_bytes.argtypes = [_vp, _vp, C.POINTER(C.c_size_t)]
_lib.baoc_configure.argtypes = [_vp, _vp, _vp, C.c_size_t, _vp]
_lib.baoc_step.argtypes = [_vp, _vp, _vp, C.c_int64, _vp]
_lib.baoc_step_from_host.argtypes = [_vp, _vp, _vp, _vp, C.c_int, C.c_int64, _vp]
_lib.baoc_view.argtypes = [_vp, C.c_int, C.c_int, C.POINTER(_vp), C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
_lib.baoc_nonfinite.argtypes = [_vp, _vp, C.POINTER(C.c_int32), _vp]
_lib.baoc_reconfigure.argtypes = [_vp, _vp, _vp, C.c_size_t, C.c_int64, C.c_int, _vp]
_lib.baoc_configure_from_window.argtypes = [_vp, _vp, _vp, C.c_size_t, _vp]
_lib.baoc_partition.argtypes = [C.c_int, _vp, _vp, C.c_int, _vp, C.c_double, C.c_double, _vp, _vp, _vp]
_lib.baoc_set_sampling.argtypes = [_vp, C.POINTER(Sample)]
_lib.baoc_time_scratch_bytes.argtypes = [_vp, C.POINTER(C.c_size_t)]
_lib.baoc_measure_time_ratios.argtypes = [_vp, _vp, _vp, _vp, C.c_size_t, C.c_int, C.c_int, _vp, _vp, _vp]
_lib.baoc_export.argtypes = [_vp, _vp, C.c_size_t, C.POINTER(C.c_size_t)]
_lib.baoc_import.argtypes = [_vp, _vp, C.c_size_t, _vp, C.c_size_t, _vp, C.c_size_t, _vp]
_lib.baoc_set_factored_schedule.argtypes = [_vp, C.c_int64]
_lib.baoc_check_status.argtypes = [C.POINTER(Check)]
_lib.baoc_check_selftest.argtypes = [_vp]
_lib.baoc_profile.argtypes = [_vp, C.c_int]
_lib.baoc_profile_last.argtypes = [_vp, C.POINTER(C.c_float)]
_lib.baoc_sample_stats_noalloc.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, C.c_double, C.c_double, C.c_double, _vp, _vp]
_lib.baoc_noalloc_last_error.argtypes = []
_lib.baoc_noalloc_last_error.restype = C.c_char_p
NOALLOC_MAX_NUMEL = 67108864


def sample_stats_noalloc(grad: torch.Tensor, gprev: torch.Tensor, m: torch.Tensor, v: torch.Tensor, out4: torch.Tensor,
                         beta_m: float = 0.9, beta_v: float = 0.999, eps: float = 1e-12, numel: Optional[int] = None):
    """``baoc_sample_stats_noalloc``: one gradient observation of one block with no handle, no workspace and no
    allocation (for callers that cannot allocate device memory; see the header).  grad / gprev: bf16 device
    tensors, m / v: fp32 device tensors, out4: float64 device tensor of 4 elements.  Queues two kernels on the
    current stream and returns; calls that overlap on one GPU race on the library's built-in scratch."""
    n = grad.numel() if numel is None else int(numel)
    rc = _lib.baoc_sample_stats_noalloc(grad.data_ptr(), gprev.data_ptr(), m.data_ptr(), v.data_ptr(), n,
                                        float(beta_m), float(beta_v), float(eps), out4.data_ptr(), _stream())
    if rc < 0:
        raise BaocError(rc, _lib.baoc_noalloc_last_error().decode())


def check_status() -> dict:
    """``baoc_check_status``: the first violation the checked build's kernels recorded since the last call (and clears
    it).  {"enabled": 0, "code": 0, ...} from a normal build."""
    c = Check()
    rc = _lib.baoc_check_status(C.byref(c))
    if rc < 0:
        raise BaocError(rc, "baoc_check_status failed")
    return {k: getattr(c, k) for k in ("enabled", "code", "kernel", "a", "b", "c", "d")}


def check_selftest() -> int:
    """``baoc_check_selftest``: queue the kernel that makes the range check fail on purpose-made numbers (no memory is
    touched).  Returns the status code (E_STATE from a normal build)."""
    return _lib.baoc_check_selftest(_stream())


def partition(numel, z, w=None, alpha: float = 0.0, tau: Optional[float] = None):
    """``baoc_partition`` (Algorithm 2): candidate units in forward order -> (block index of every unit, tau used).
    z: [n_units, k] normalised diagnostic vectors; tau None = the upper quartile of the pairwise differences."""
    n = np.ascontiguousarray(numel, np.int64)
    Z = np.ascontiguousarray(z, np.float64)
    if Z.ndim != 2 or Z.shape[0] != n.shape[0]:
        raise ValueError("z must be [n_units, k]")
    ww = None if w is None else np.ascontiguousarray(w, np.float64)
    if ww is not None and ww.shape != (Z.shape[1],):
        raise ValueError("w must have k entries")
    out = np.zeros(n.shape[0], np.int32)
    nb, tu = C.c_int32(), C.c_double()
    rc = _lib.baoc_partition(n.shape[0], n.ctypes.data, Z.ctypes.data, Z.shape[1], _np_ptr(ww), float(alpha),
                             -1.0 if tau is None else float(tau), out.ctypes.data, C.addressof(nb), C.addressof(tu))
    if rc < 0:
        raise BaocError(rc, "baoc_partition: invalid argument")
    return out, tu.value


def unit_diagnostics(stats) -> np.ndarray:
    """[n, 5] normalised diagnostic vectors (s_A, s_M, C~, s_F, l_Q at 8 bits) from ``Baoc.risk``'s per-block records:
    the z_j that ``partition`` takes when the candidate units were run through a window as blocks."""
    return np.asarray([[s.s_A, s.s_M, s.C_tilde, s.s_F, s.lQ8] for s in stats], np.float64)


def default_opts() -> Opts:
    o = Opts()
    _lib.baoc_default_opts(C.byref(o))
    return o


Q_LINEAR, Q_DYNAMIC = 0, 1
AF_SCHEDULE, AF_CLIP, AF_RELATIVE, AF_EPS1 = 1, 2, 4, 8


def make_config(adaptive, momentum, decoupled_wd, factored, bits, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                weight_decay=0.0, quantizer=Q_LINEAR, af_flags=0) -> Config:
    """quantizer: Q_DYNAMIC puts 8-bit Adam on the non-linear codebook; af_flags: Adafactor's options of the factored tuple."""
    return Config(adaptive, momentum, decoupled_wd, factored, bits, quantizer, af_flags, 0, lr, beta1, beta2, eps,
                  weight_decay)


def default_configs() -> List[Config]:
    """fp32 AdamW, 8-bit AdamW, momentum-free RMS scaling, factored second moment, SGD with momentum."""
    return [make_config(1, 1, 1, 0, 32, weight_decay=0.01), make_config(1, 1, 1, 0, 8, weight_decay=0.01),
            make_config(1, 0, 1, 0, 32, weight_decay=0.01), make_config(1, 0, 1, 1, 32, weight_decay=0.01),
            make_config(0, 1, 1, 0, 32, lr=1e-2, weight_decay=0.01)]


def extended_configs() -> List[Config]:
    """The five default tuples plus the plain gradient step, the bf16-state variants of Adam(W), RMS scaling and
    SGD with momentum, the 8-bit variants of RMS scaling and SGD with momentum, and the factored second moment with
    bf16 and 8-bit row / column statistics (indices 11 and 12); then the two alternative readings: Adam on the
    non-linear 8-bit codebook (13) and the factored tuple with all of Adafactor's options (14)."""
    return default_configs() + [make_config(0, 0, 1, 0, 32, lr=1e-2, weight_decay=0.01),
                                make_config(1, 1, 1, 0, 16, weight_decay=0.01),
                                make_config(1, 0, 1, 0, 16, weight_decay=0.01),
                                make_config(0, 1, 1, 0, 16, lr=1e-2, weight_decay=0.01),
                                make_config(1, 0, 1, 0, 8, weight_decay=0.01),
                                make_config(0, 1, 1, 0, 8, lr=1e-2, weight_decay=0.01),
                                make_config(1, 0, 1, 1, 16, weight_decay=0.01),
                                make_config(1, 0, 1, 1, 8, weight_decay=0.01),
                                make_config(1, 1, 1, 0, 8, weight_decay=0.01, quantizer=Q_DYNAMIC),
                                make_config(1, 0, 1, 1, 32, weight_decay=0.01,
                                            af_flags=AF_SCHEDULE | AF_CLIP | AF_RELATIVE | AF_EPS1)]


def pointer_table(tensors: Sequence[torch.Tensor]):
    """Host array of the tensors' data pointers, in the layout the C calls take."""
    return (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


class Baoc:
    """One handle of the library (``baoc_create`` .. ``baoc_destroy``)."""

    def __init__(self, blocks: Sequence, configs: Sequence[Config], opts: Optional[Opts] = None):
        """blocks: objects with ``numel``, ``rows``, ``cols`` (or 3-tuples)."""
        bl = []
        for b in blocks:
            if isinstance(b, (tuple, list)):
                bl.append(Block(*b))
            else:
                bl.append(Block(b.numel, b.rows, b.cols))
        self.n_blocks, self.n_cfg = len(bl), len(configs)
        self._blocks = (Block * len(bl))(*bl)
        self._cfgs = (Config * len(configs))(*configs)
        self._h = _vp()
        self._keep = []            # device buffers the handle points into
        rc = _lib.baoc_create(C.byref(self._h), len(bl), self._blocks, len(configs), self._cfgs,
                              C.byref(opts) if opts is not None else None)
        if rc != 0:
            raise BaocError(rc, "baoc_create rejected its arguments")

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.baoc_destroy(self._h)
            self._h = None

    __del__ = close

    def _check(self, rc: int) -> int:
        if rc < 0:
            raise BaocError(rc, _lib.baoc_last_error(self._h).decode())
        return rc

    def last_error(self) -> str:
        return _lib.baoc_last_error(self._h).decode()

    def query(self) -> Info:
        info = Info()
        self._check(_lib.baoc_query(self._h, C.byref(info)))
        return info

    # ---- sampling window --------------------------------------------------
    def set_sampling(self, samples):
        """``baoc_set_sampling``.  samples: None (dense), or one (rows, cols) pair of integer index arrays per block
        (cols is None for a vector block).  Call before ``bind_stats_workspace``."""
        if samples is None:
            self._check(_lib.baoc_set_sampling(self._h, None))
            return
        keep, arr = [], (Sample * self.n_blocks)()
        for i, (rows, cols) in enumerate(samples):
            r = np.ascontiguousarray(rows, np.int64)
            keep.append(r)
            arr[i].n_rows, arr[i].rows = r.size, r.ctypes.data
            if cols is None:
                arr[i].n_cols, arr[i].cols = 1, None
            else:
                c = np.ascontiguousarray(cols, np.int32)
                keep.append(c)
                arr[i].n_cols, arr[i].cols = c.size, c.ctypes.data
        self._check(_lib.baoc_set_sampling(self._h, arr))

    def stats_workspace_bytes(self) -> int:
        n = C.c_size_t()
        self._check(_lib.baoc_stats_workspace_bytes(self._h, C.byref(n)))
        return n.value

    def bind_stats_workspace(self, ws: torch.Tensor):
        self._check(_lib.baoc_bind_stats_workspace(self._h, ws.data_ptr(), ws.numel() * ws.element_size(), _stream()))
        self._keep.append(ws)

    def sample_stats(self, grads):
        """grads: list of bf16 device tensors, or a table from ``pointer_table``."""
        tab = grads if isinstance(grads, C.Array) else pointer_table(grads)
        self._check(_lib.baoc_sample_stats(self._h, tab, _stream()))

    def read_stats(self) -> List[dict]:
        out = (BlockStats * self.n_blocks)()
        self._check(_lib.baoc_read_stats(self._h, out, _stream()))
        return [s.as_dict() for s in out]

    def risk(self, params, as_dicts: bool = True):
        """Returns (risk [n_blocks, n_cfg] float64, list of per-block stats dicts); with as_dicts=False the second item is
        the array of BlockStats structures as the library filled it (no per-field conversion)."""
        tab = params if isinstance(params, C.Array) else pointer_table(params)
        risk = np.zeros((self.n_blocks, self.n_cfg), np.float64)
        st = (BlockStats * self.n_blocks)()
        self._check(_lib.baoc_risk(self._h, tab, risk.ctypes.data, st, _stream()))
        return risk, ([s.as_dict() for s in st] if as_dicts else st)

    def risk_from_raw(self, raw: Sequence[dict]):
        st = (BlockStats * self.n_blocks)()
        for i, r in enumerate(raw):
            for k in ("A", "rho_bar", "snr", "C", "F", "Q32", "Q16", "Q8"):
                setattr(st[i], k, float(r[k]))
        risk = np.zeros((self.n_blocks, self.n_cfg), np.float64)
        self._check(_lib.baoc_risk_from_raw(self._h, st, risk.ctypes.data))
        return risk, [s.as_dict() for s in st]

    # ---- allocation -------------------------------------------------------
    def cost_model(self):
        mem = np.zeros((self.n_blocks, self.n_cfg), np.int64)
        ratio = np.zeros((self.n_blocks, self.n_cfg), np.float64)
        self._check(_lib.baoc_cost_model(self._h, mem.ctypes.data, ratio.ctypes.data))
        return mem, ratio

    def allocate(self, risk, mem, ratio, b_mem: int, b_time: float, forbid=None, pref=None):
        """Returns (assignment int32[n_blocks], objective, status) with status 0 or W_NODE_LIMIT."""
        risk = np.ascontiguousarray(risk, np.float64)
        mem = np.ascontiguousarray(mem, np.int64)
        ratio = np.ascontiguousarray(ratio, np.float64)
        forbid = None if forbid is None else np.ascontiguousarray(forbid, np.uint8)
        pref = None if pref is None else np.ascontiguousarray(pref, np.float64)
        asg = np.zeros(self.n_blocks, np.int32)
        obj = C.c_double()
        rc = self._check(_lib.baoc_allocate(self._h, risk.ctypes.data, mem.ctypes.data, ratio.ctypes.data, int(b_mem),
                                            float(b_time), _np_ptr(forbid), _np_ptr(pref), asg.ctypes.data, C.byref(obj)))
        return asg, obj.value, rc

    def time_scratch_bytes(self) -> int:
        n = C.c_size_t()
        self._check(_lib.baoc_time_scratch_bytes(self._h, C.byref(n)))
        return n.value

    def measure_time_ratios(self, grads, params, scratch: torch.Tensor, base_cfg: int = 0, reps: int = 3):
        """``baoc_measure_time_ratios``: (ratio [n_blocks, n_cfg], milliseconds [n_blocks, n_cfg])."""
        g = grads if isinstance(grads, C.Array) else pointer_table(grads)
        p = params if isinstance(params, C.Array) else pointer_table(params)
        ratio = np.zeros((self.n_blocks, self.n_cfg), np.float64)
        ms = np.zeros((self.n_blocks, self.n_cfg), np.float64)
        self._check(_lib.baoc_measure_time_ratios(self._h, g, p, scratch.data_ptr(), scratch.numel() * scratch.element_size(),
                                                  int(base_cfg), int(reps), ratio.ctypes.data, ms.ctypes.data, _stream()))
        return ratio, ms

    # ---- training ---------------------------------------------------------
    def state_bytes(self, assign) -> int:
        a = np.ascontiguousarray(assign, np.int32)
        n = C.c_size_t()
        self._check(_lib.baoc_state_bytes(self._h, a.ctypes.data, C.byref(n)))
        return n.value

    def configure(self, assign, state: torch.Tensor):
        a = np.ascontiguousarray(assign, np.int32)
        self._check(_lib.baoc_configure(self._h, a.ctypes.data, state.data_ptr(), state.numel() * state.element_size(),
                                        _stream()))
        self._keep.append(state)

    def reconfigure(self, assign, state: torch.Tensor, steps_done: int, inherit: bool = True):
        """``baoc_reconfigure``: move to a new assignment, migrating compatible states into the new buffer."""
        a = np.ascontiguousarray(assign, np.int32)
        self._check(_lib.baoc_reconfigure(self._h, a.ctypes.data, state.data_ptr(), state.numel() * state.element_size(),
                                          int(steps_done), int(bool(inherit)), _stream()))
        self._keep.append(state)

    def configure_from_window(self, assign, state: torch.Tensor):
        """``baoc_configure_from_window``: instantiate the optimizer with the window's moments as its initial moments."""
        a = np.ascontiguousarray(assign, np.int32)
        self._check(_lib.baoc_configure_from_window(self._h, a.ctypes.data, state.data_ptr(),
                                                    state.numel() * state.element_size(), _stream()))
        self._keep.append(state)

    def step(self, grads, params, step_t: int):
        g = grads if isinstance(grads, C.Array) else pointer_table(grads)
        p = params if isinstance(params, C.Array) else pointer_table(params)
        self._check(_lib.baoc_step(self._h, g, p, int(step_t), _stream()))

    def step_from_host(self, host_grads, dev_grads, params, do_stats: bool, step_t: int):
        hg = host_grads if isinstance(host_grads, C.Array) else pointer_table(host_grads)
        dg = dev_grads if isinstance(dev_grads, C.Array) else pointer_table(dev_grads)
        p = None if params is None else (params if isinstance(params, C.Array) else pointer_table(params))
        self._check(_lib.baoc_step_from_host(self._h, hg, dg, p, int(bool(do_stats)), int(step_t), _stream()))

    def view(self, block: int, which: int):
        """(device pointer, element count, element bytes) of a state tensor (see ``baoc_view``)."""
        p, n, eb = _vp(), C.c_int64(), C.c_int32()
        self._check(_lib.baoc_view(self._h, block, which, C.byref(p), C.byref(n), C.byref(eb)))
        return p.value, n.value, eb.value

    def view_tensor(self, block: int, which: int, dtype: torch.dtype) -> torch.Tensor:
        """A state tensor as a torch view (no copy) into the buffer the caller bound."""
        p, n, eb = self.view(block, which)
        for buf in self._keep:
            base = buf.data_ptr()
            if base <= p < base + buf.numel() * buf.element_size():
                flat = buf.view(torch.uint8).reshape(-1)
                return flat[p - base: p - base + n * eb].view(dtype)
        raise BaocError(E_STATE, "the tensor lies in no buffer bound through this object")

    def export_state(self) -> bytes:
        """The host blob of ``baoc_export`` (window step count and assignment)."""
        n = C.c_size_t()
        self._check(_lib.baoc_export(self._h, None, 0, C.byref(n)))
        buf = C.create_string_buffer(n.value)
        self._check(_lib.baoc_export(self._h, buf, n.value, C.byref(n)))
        return buf.raw[:n.value]

    def import_state(self, blob: bytes, ws: Optional[torch.Tensor] = None, state: Optional[torch.Tensor] = None):
        """``baoc_import``: ws / state are device buffers that already hold the checkpointed bytes."""
        nb = lambda t: t.numel() * t.element_size()
        self._check(_lib.baoc_import(self._h, blob, len(blob), ws.data_ptr() if ws is not None else None,
                                     nb(ws) if ws is not None else 0, state.data_ptr() if state is not None else None,
                                     nb(state) if state is not None else 0, _stream()))
        for t in (ws, state):
            if t is not None:
                self._keep.append(t)

    def set_factored_schedule(self, group_bytes: int):
        """``baoc_set_factored_schedule``: 0 = one reduction and one update launch; > 0 = factored blocks in groups of
        at most that many gradient bytes, each reduced and updated back to back (before ``configure``)."""
        self._check(_lib.baoc_set_factored_schedule(self._h, int(group_bytes)))

    def profile(self, enable: bool):
        self._check(_lib.baoc_profile(self._h, int(bool(enable))))

    def profile_last(self):
        """(ms of the factored row/column kernels, ms of the fused update kernel) of the last step."""
        ms = (C.c_float * 2)()
        self._check(_lib.baoc_profile_last(self._h, ms))
        return float(ms[0]), float(ms[1])

    def nonfinite(self):
        flags = np.zeros(self.n_blocks, np.uint8)
        cnt = C.c_int32()
        self._check(_lib.baoc_nonfinite(self._h, flags.ctypes.data, C.byref(cnt), _stream()))
        return cnt.value, flags
