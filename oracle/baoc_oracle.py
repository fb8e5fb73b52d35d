"""CPU oracle for the BAOC hot path.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

A plain, slow, double-precision numpy restatement of what the paper's method
computes on the path this repository accelerates: the per-block gradient
statistics (Sec. 3.3, Eq. 3-8), their normalisation and the risk matrix
(Appendix A, Eq. 9-21), the aggressiveness penalty (Eq. 1), the budgeted
allocation (Eq. 2, by exhaustive enumeration) and the update rule of each
configuration tuple of Definition 3.1 that the library offers.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares no code with the CUDA library and never calls it.
Every function works on one block at a time, takes plain numpy arrays and
carries floating-point state in float64; the 8-bit codes and their fp32
absmax scales are the state by definition and are kept in their own types.

Where the paper is silent the readings below are used (the same ones the
library documents):
  * coordinates are sampled densely (the sample is the whole block);
  * EMA moments start at zero and are not bias-corrected (Eq. 3 as written);
  * the stability EMA starts at the first available cosine; beta_rho = 0.9;
  * quantiles use linear interpolation at position q*(n-1);
  * the 8-bit quantiser is block-wise absmax with linear codes over 256
    consecutive elements (signed 127 levels for first moments, unsigned 255
    for second moments, round half to even, fp32 absmax); the 16-bit
    quantiser rounds to bfloat16;
  * the update direction of Eq. 8 is m/(sqrt(v)+1e-8) from the window's own
    moments;
  * update rules are the textbook ones for each tuple (see the step_*
    functions).

Parity unpinned: no value printed in the paper distinguishes these readings;
each function below is pinned by closed forms, invariants, library special
cases and brute force in the CPU test-suite instead.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# Options and configuration tuples
# ----------------------------------------------------------------------------

@dataclass
class Opts:
    beta_m: float = 0.9            # Eq. 3, "standard Adam values"
    beta_v: float = 0.999
    beta_rho: float = 0.9          # Eq. 5 smoothing factor (paper gives no value)
    eps: float = 1e-12             # Appendix A.1
    a_lo: float = math.log(2.0)    # Eq. 11
    a_hi: float = math.log(10.0)
    rho_lo: float = 0.2            # Eq. 13
    rho_hi: float = 0.6
    snr_lo: float = 0.0            # Eq. 15
    snr_hi: float = 2.0
    w: Tuple[float, float, float, float, float] = (1.0, 1.0, 1.0, 1.0, 1.0)  # w_A, w_M, w_C, w_F, w_Q
    gamma: float = 0.1             # weight of Agg in the objective
    use_snr: bool = True           # Eq. 17, else s_M = s_rho
    eps_adam: float = 1e-8         # epsilon of the update direction in Eq. 8
    qblock: int = 256              # elements per quantisation block
    quantizer8: str = "linear"     # the 8-bit quantiser of Eq. 8: "linear" absmax codes or the "dynamic" codebook
    debias: bool = False           # alternative reading of the hats in Eq. 3: the diagnostics of Eq. 4-8 are taken from
                                   # the bias-corrected moments m / (1 - beta_m^T), v / (1 - beta_v^T) after T steps


@dataclass
class Config:
    """Definition 3.1: c = (y_a, y_m, y_d, y_f, b) plus the hyper-parameters
    of the update rule it instantiates."""
    adaptive: int
    momentum: int
    decoupled_wd: int
    factored: int
    bits: int
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    quantizer: str = "linear"      # 8-bit states: "linear" absmax codes, or the non-linear "dynamic" codebook
    # Options of the factored tuple that turn its mechanism-pure rule into the published Adafactor algorithm (the
    # paper names Adafactor among its mechanisms without saying which of its parts are meant).  All off by default.
    af_beta2_schedule: bool = False   # beta2_t = 1 - t^-0.8 instead of a constant, and no bias correction
    af_clip: float = 0.0              # d > 0: the update u is divided by max(1, RMS(u) / d)
    af_relative_step: bool = False    # step size max(1e-3, RMS(theta)) * min(1e-2, 1 / sqrt(t)) instead of lr
    af_eps1: float = 0.0              # added to every squared gradient before the row and column means


def default_configs() -> List[Config]:
    """The five tuples of the hot path: fp32 AdamW, 8-bit AdamW, momentum-free
    RMS scaling, factored second moment, SGD with momentum."""
    return [Config(1, 1, 1, 0, 32, weight_decay=0.01),
            Config(1, 1, 1, 0, 8, weight_decay=0.01),
            Config(1, 0, 1, 0, 32, weight_decay=0.01),
            Config(1, 0, 1, 1, 32, weight_decay=0.01),
            Config(0, 1, 1, 0, 32, lr=1e-2, weight_decay=0.01)]


# ----------------------------------------------------------------------------
# Quantisers (the "standard quantizer" of Sec. 3.3, Precision Sensitivity)
# ----------------------------------------------------------------------------

def _blocks_view(x: np.ndarray, qblock: int):
    """Pad x with zeros to a multiple of qblock and view it as [nq, qblock]."""
    d = x.shape[0]
    nq = (d + qblock - 1) // qblock
    pad = np.zeros(nq * qblock, dtype=x.dtype)
    pad[:d] = x
    return pad.reshape(nq, qblock), d


def quantize8(x: np.ndarray, signed: bool, qblock: int = 256):
    """Block-wise absmax linear 8-bit codes.

    Per quantisation block: a = fl32(max |x|); code = clamp(rne(L * x / a)) with
    L = 127 (signed, codes in [-127, 127]) or L = 255 (unsigned, [0, 255]);
    a == 0 gives all-zero codes.  Returns (codes, absmax fp32[nq]).
    """
    x = np.asarray(x, dtype=F64)
    xb, d = _blocks_view(x, qblock)
    a = np.max(np.abs(xb), axis=1).astype(np.float32)
    L = 127.0 if signed else 255.0
    a64 = a.astype(F64)
    safe = np.where(a64 > 0.0, a64, 1.0)
    s = np.rint(L * xb / safe[:, None])             # np.rint rounds half to even
    s = np.clip(s, -L if signed else 0.0, L)
    s = np.where(a64[:, None] > 0.0, s, 0.0)
    codes = s.reshape(-1)[:d].astype(np.int8 if signed else np.uint8)
    return codes, a


def dequantize8(codes: np.ndarray, absmax: np.ndarray, signed: bool, qblock: int = 256) -> np.ndarray:
    """x = code * a / L in double."""
    L = 127.0 if signed else 255.0
    cb, d = _blocks_view(codes.astype(F64), qblock)
    x = cb * absmax.astype(F64)[:, None] / L
    return x.reshape(-1)[:d]


# ----------------------------------------------------------------------------
# Non-linear 8-bit codebook: the alternative reading of "a standard quantizer".
# The block-wise 8-bit optimizers that the paper cites for its AdamW8 baseline
# (Sec. 4.1, Baselines) describe a "dynamic" 8-bit data type: an optional sign
# bit, then a run of zero bits whose length E is a decimal exponent, one
# indicator bit, and the remaining F bits as a linear fraction within a decade.
# The table below is built from that description (it is this repository's own
# construction, no third-party table is reproduced): the magnitudes are
#     10^-E * (0.1 + 0.9 (k + 1) / 2^F),   k = 0 .. 2^F - 1,
# with F = B - 1 - E for E = 0 .. B - 1, where B = 7 value bits for the signed
# type (first moments) and B = 8 for the unsigned one (second moments), plus the
# value 0.  Decade E thus covers (10^-(E+1), 10^-E] with 2^F entries, the largest
# entry is exactly 1 and the smallest positive one 10^-(B-1).  Signed: 127
# magnitudes of either sign and zero, 255 entries; unsigned: 255 and zero, 256.
# A code is the index of its entry in ascending order.  Quantisation is block-
# wise with the fp32 absmax a: the code of x is the entry nearest to x / a (a tie
# goes to the entry of smaller magnitude); x ~ entry * a.
# ----------------------------------------------------------------------------

def dynamic_codebook(signed: bool) -> np.ndarray:
    bits = 7 if signed else 8
    mags = []
    for E in range(bits):
        F = bits - 1 - E
        for k in range(2 ** F):
            mags.append(10.0 ** (-E) * (0.1 + 0.9 * (k + 1) / 2.0 ** F))
    mags = np.sort(np.asarray(mags, F64))
    if signed:
        return np.concatenate([-mags[::-1], [0.0], mags])
    return np.concatenate([[0.0], mags])


def quantize8_dynamic(x: np.ndarray, signed: bool, qblock: int = 256):
    """Codes (uint8 indices into ``dynamic_codebook(signed)``) and the fp32 absmax of every quantisation block."""
    x = np.asarray(x, dtype=F64)
    xb, d = _blocks_view(x, qblock)
    a = np.max(np.abs(xb), axis=1).astype(np.float32)
    a64 = a.astype(F64)
    y = xb / np.where(a64 > 0.0, a64, 1.0)[:, None]
    y = np.where(a64[:, None] > 0.0, y, 0.0)
    t = dynamic_codebook(signed)
    mid = 0.5 * (t[:-1] + t[1:])
    toward_zero_pos = np.searchsorted(mid, y, side="left")      # y on a midpoint: the lower entry, smaller for y > 0
    toward_zero_neg = np.searchsorted(mid, y, side="right")     # the upper entry, smaller in magnitude for y < 0
    idx = np.where(y >= 0.0, toward_zero_pos, toward_zero_neg)
    return idx.reshape(-1)[:d].astype(np.uint8), a


def dequantize8_dynamic(codes: np.ndarray, absmax: np.ndarray, signed: bool, qblock: int = 256) -> np.ndarray:
    """x = entry * a in double."""
    t = dynamic_codebook(signed)
    cb, d = _blocks_view(codes.astype(np.int64), qblock)
    x = t[cb] * absmax.astype(F64)[:, None]
    return x.reshape(-1)[:d]


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64.

    The value is first rounded to fp32, then its low 16 bits are rounded away.
    """
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32)
    out = np.where(np.isfinite(f), out, f)
    return out.astype(F64)


# ----------------------------------------------------------------------------
# O1. Per-step statistics (Eq. 3 and Eq. 5 left)
# ----------------------------------------------------------------------------

@dataclass
class StatsState:
    d: int
    m: np.ndarray
    v: np.ndarray
    g_prev: Optional[np.ndarray] = None
    rho_bar: float = 0.0
    n_cos: int = 0
    t: int = 0
    last_cos: float = 0.0
    # diagnostic only (not used by the risk): EMA of cos(g_t, m_{t-1})
    rho_mom: float = 0.0
    n_cos_mom: int = 0


def stats_init(d: int) -> StatsState:
    return StatsState(d=d, m=np.zeros(d, F64), v=np.zeros(d, F64))


def _cosine(a: np.ndarray, b: np.ndarray, eps: float) -> float:
    """<a,b> / (||a|| ||b|| + eps), with a non-finite result replaced by 0
    (Appendix A.1: a NaN cosine counts as 0)."""
    c = float(np.dot(a, b)) / (math.sqrt(float(np.dot(a, a))) * math.sqrt(float(np.dot(b, b))) + eps)
    return c if math.isfinite(c) else 0.0


def stats_step(st: StatsState, g: np.ndarray, o: Opts) -> None:
    """One gradient observation of one block."""
    g = np.asarray(g, dtype=F64)
    st.t += 1
    if st.g_prev is not None:
        c = _cosine(g, st.g_prev, o.eps)                       # Eq. 5 left
        st.last_cos = c
        st.rho_bar = c if st.n_cos == 0 else o.beta_rho * st.rho_bar + (1.0 - o.beta_rho) * c
        st.n_cos += 1
        cm = _cosine(g, st.m, o.eps)                           # diagnostic
        st.rho_mom = cm if st.n_cos_mom == 0 else o.beta_rho * st.rho_mom + (1.0 - o.beta_rho) * cm
        st.n_cos_mom += 1
    st.m = o.beta_m * st.m + (1.0 - o.beta_m) * g              # Eq. 3
    st.v = o.beta_v * st.v + (1.0 - o.beta_v) * (g * g)
    st.g_prev = g.copy()


# ----------------------------------------------------------------------------
# O2. Finalize (Eq. 4, Eq. 5 right, Eq. 6, Eq. 7, Eq. 8)
# ----------------------------------------------------------------------------

def quantile_linear(x: np.ndarray, q: float) -> float:
    """q-th quantile by linear interpolation between order statistics at
    position q*(n-1)."""
    s = np.sort(np.asarray(x, dtype=F64))
    n = s.shape[0]
    pos = q * (n - 1)
    k = int(math.floor(pos))
    frac = pos - k
    if k + 1 < n:
        return float(s[k] + frac * (s[k + 1] - s[k]))
    return float(s[k])


def anisotropy(v: np.ndarray, eps: float) -> float:
    """Eq. 4."""
    return math.log((quantile_linear(v, 0.9) + eps) / (quantile_linear(v, 0.1) + eps))


def snr(m: np.ndarray, v: np.ndarray, eps: float) -> float:
    """Eq. 5 right: ||m||^2 / (||v||_1 + eps)."""
    return float(np.dot(m, m)) / (float(np.sum(np.abs(v))) + eps)


def distortion(v: np.ndarray, theta: np.ndarray, eps: float) -> float:
    """Eq. 6 with p = 1/(sqrt(v)+eps)."""
    theta = np.asarray(theta, dtype=F64)
    p = 1.0 / (np.sqrt(v) + eps)
    pbar = float(np.mean(p))
    num = np.linalg.norm((p / pbar - 1.0) * theta)
    return float(num / (np.linalg.norm(theta) + eps))


def structure_residual(v: np.ndarray, rows: int, cols: int, eps: float) -> float:
    """Eq. 7: S = v as rows x cols, rank-1 model from row and column means."""
    if cols <= 1:
        return 1.0          # not a matrix block: the factored configuration is not offered
    S = np.asarray(v, dtype=F64).reshape(rows, cols)
    a = S.mean(axis=1)
    b = S.mean(axis=0)
    mu = float(S.mean())
    if mu == 0.0:
        St = np.zeros_like(S)
    else:
        St = np.outer(a, b) / mu
    return float(np.linalg.norm(S - St) / (np.linalg.norm(S) + eps))


def precision_cosine(m: np.ndarray, v: np.ndarray, bits: int, o: Opts) -> float:
    """Eq. 8: cosine between the full-precision direction m/(sqrt(v)+eps_adam)
    and the one computed from quantised moments."""
    u32 = m / (np.sqrt(v) + o.eps_adam)
    if bits == 32:
        mq, vq = m, v
    elif bits == 16:
        mq, vq = round_bf16(m), round_bf16(v)
    elif bits == 8 and o.quantizer8 == "dynamic":
        cm, am = quantize8_dynamic(m, True, o.qblock)
        cv, av = quantize8_dynamic(v, False, o.qblock)
        mq = dequantize8_dynamic(cm, am, True, o.qblock)
        vq = dequantize8_dynamic(cv, av, False, o.qblock)
    elif bits == 8:
        cm, am = quantize8(m, True, o.qblock)
        cv, av = quantize8(v, False, o.qblock)
        mq = dequantize8(cm, am, True, o.qblock)
        vq = dequantize8(cv, av, False, o.qblock)
    else:
        raise ValueError("bits must be 8, 16 or 32")
    ub = mq / (np.sqrt(vq) + o.eps_adam)
    return _cosine(u32, ub, o.eps)


def quant_rel_error(x: np.ndarray, bits: int, signed: bool, o: Opts) -> float:
    """Diagnostic: ||x - Q_b(x)|| / ||x|| (0 for a zero vector)."""
    if bits == 16:
        xq = round_bf16(x)
    elif o.quantizer8 == "dynamic":
        c, a = quantize8_dynamic(x, signed, o.qblock)
        xq = dequantize8_dynamic(c, a, signed, o.qblock)
    else:
        c, a = quantize8(x, signed, o.qblock)
        xq = dequantize8(c, a, signed, o.qblock)
    n = float(np.linalg.norm(x))
    return float(np.linalg.norm(x - xq)) / n if n > 0.0 else 0.0


def window_moments(st: StatsState, o: Opts) -> Tuple[np.ndarray, np.ndarray]:
    """The moments the end-of-window diagnostics are taken from: the recursion of Eq. 3 as it stands, or (o.debias) with
    Adam's bias correction for the st.t steps observed, m / (1 - beta_m^t) and v / (1 - beta_v^t)."""
    if o.debias and st.t > 0:
        return st.m / (1.0 - o.beta_m ** st.t), st.v / (1.0 - o.beta_v ** st.t)
    return st.m, st.v


def stats_finalize(st: StatsState, theta: np.ndarray, rows: int, cols: int, o: Opts) -> Dict[str, float]:
    """Raw diagnostics z_i of one block at the end of the window."""
    m, v = window_moments(st, o)
    return {
        "A": anisotropy(v, o.eps),
        "rho_bar": st.rho_bar,
        "snr": snr(m, v, o.eps),
        "C": distortion(v, theta, o.eps),
        "F": structure_residual(v, rows, cols, o.eps),
        "Q32": precision_cosine(m, v, 32, o),
        "Q16": precision_cosine(m, v, 16, o),
        "Q8": precision_cosine(m, v, 8, o),
        "q10": quantile_linear(v, 0.1),
        "q90": quantile_linear(v, 0.9),
        "rho_mom": st.rho_mom,
        "err_m8": quant_rel_error(m, 8, True, o),
        "err_v8": quant_rel_error(v, 8, False, o),
        "err_m16": quant_rel_error(m, 16, True, o),
        "err_v16": quant_rel_error(v, 16, False, o),
    }


# ----------------------------------------------------------------------------
# O3. Normalisation (Appendix A, Eq. 10-20)
# ----------------------------------------------------------------------------

def _clip(x: float, lo: float, hi: float) -> float:
    return min(max(x, lo), hi)


def normalise(raw: Dict[str, float], o: Opts) -> Dict[str, float]:
    s_A = _clip((raw["A"] - o.a_lo) / (o.a_hi - o.a_lo), 0.0, 1.0)                     # Eq. 12
    s_rho = _clip((raw["rho_bar"] - o.rho_lo) / (o.rho_hi - o.rho_lo), 0.0, 1.0)       # Eq. 14
    s_snr = _clip((math.log(1.0 + raw["snr"]) - o.snr_lo) / (o.snr_hi - o.snr_lo), 0.0, 1.0)  # Eq. 16
    s_M = s_rho * s_snr if o.use_snr else s_rho                                        # Eq. 17
    C_t = math.log(1.0 + raw["C"])                                                     # Eq. 18
    s_F = _clip(raw["F"], 0.0, 1.0)                                                    # Eq. 19
    out = {"s_A": s_A, "s_rho": s_rho, "s_snr": s_snr, "s_M": s_M, "C_tilde": C_t, "s_F": s_F}
    for b in (32, 16, 8):
        Q = _clip(raw[f"Q{b}"], o.eps, 1.0)                                            # Eq. 10
        out[f"lQ{b}"] = -math.log(Q + o.eps)                                           # Eq. 20
    return out


# ----------------------------------------------------------------------------
# O4. Risk, aggressiveness, objective (Eq. 9/21, Eq. 1)
# ----------------------------------------------------------------------------

def risk(z: Dict[str, float], c: Config, o: Opts) -> float:
    wA, wM, wC, wF, wQ = o.w
    return (wA * z["s_A"] * (1 - c.adaptive) + wM * z["s_M"] * (1 - c.momentum)
            + wC * z["C_tilde"] * (1 - c.decoupled_wd) + wF * z["s_F"] * c.factored
            + wQ * z[f"lQ{c.bits}"])


def agg(c: Config) -> float:
    return (1 - c.adaptive) + (1 - c.momentum) + (1 - c.decoupled_wd) + c.factored + 32.0 / c.bits - 1.0


def objective(R: float, c: Config, o: Opts, pref: float = 0.0) -> float:
    """Phi = (R - pref) + gamma * Agg."""
    return (R - pref) + o.gamma * agg(c)


# ----------------------------------------------------------------------------
# Cost model (StateMem definition, Sec. 3.1) and fixed point of the allocator
# ----------------------------------------------------------------------------

def state_bytes(c: Config, numel: int, rows: int, cols: int, qblock: int = 256) -> int:
    """M_{i,c}: bytes of persistent optimizer state of one block."""
    nq = (numel + qblock - 1) // qblock
    def per_tensor():
        if c.bits == 32:
            return 4 * numel
        if c.bits == 16:
            return 2 * numel
        return numel + 4 * nq           # 1-byte codes + one fp32 absmax per quantisation block
    total = 0
    if c.momentum:
        total += per_tensor()
    if c.adaptive:
        if c.factored:
            # row and column statistics in the tuple's precision (8-bit: each vector in its own quantisation blocks)
            if c.bits == 32:
                total += 4 * (rows + cols)
            elif c.bits == 16:
                total += 2 * (rows + cols)
            else:
                total += rows + cols + 4 * ((rows + qblock - 1) // qblock + (cols + qblock - 1) // qblock)
        else:
            total += per_tensor()
    return total


PHI_SCALE = 2.0 ** 30
R_SCALE = 2.0 ** 20


def phi_fixed(phi: float) -> int:
    return int(np.rint(phi * PHI_SCALE))


def ratio_fixed(r: float) -> int:
    return int(np.rint(r * R_SCALE))


def time_cap_fixed(n_blocks: int, b_time: float) -> int:
    return int(math.floor(n_blocks * b_time * R_SCALE))


# ----------------------------------------------------------------------------
# O5. Allocation by exhaustive enumeration (Eq. 2)
# ----------------------------------------------------------------------------

def allocate_bruteforce(phi_fx: Sequence[Sequence[int]], mem: Sequence[Sequence[int]],
                        r_fx: Sequence[Sequence[int]], b_mem: int, r_cap: int,
                        forbid: Optional[Sequence[Sequence[int]]] = None):
    """Enumerate every assignment in lexicographic order (block 0 slowest,
    lower configuration index first) and keep the first one of minimum total
    objective among those within both budgets and free of forbidden pairs.
    Returns (assignment list, objective) or (None, None) when infeasible."""
    n = len(phi_fx)
    k = len(phi_fx[0])
    best, best_val = None, None
    for asg in itertools.product(range(k), repeat=n):
        if forbid is not None and any(forbid[i][c] for i, c in enumerate(asg)):
            continue
        if sum(mem[i][c] for i, c in enumerate(asg)) > b_mem:
            continue
        if sum(r_fx[i][c] for i, c in enumerate(asg)) > r_cap:
            continue
        val = sum(phi_fx[i][c] for i, c in enumerate(asg))
        if best_val is None or val < best_val:
            best, best_val = list(asg), val
    return best, best_val


# ----------------------------------------------------------------------------
# O6. Update rules (Definition 3.1 tuples)
# ----------------------------------------------------------------------------

def _prologue(theta: np.ndarray, g: np.ndarray, c: Config):
    """Weight decay: decoupled (theta shrinks first) or coupled (added to g)."""
    if c.weight_decay != 0.0:
        if c.decoupled_wd:
            theta = theta * (1.0 - c.lr * c.weight_decay)
        else:
            g = g + c.weight_decay * theta
    return theta, g


def _adam_apply(theta, m, v, c: Config, t, use_m: bool):
    """t: the step count, or a pair (t_m, t_v) when the two moments have been accumulating for different numbers of
    steps (after a re-configuration that restarted one of them)."""
    t_m, t_v = t if isinstance(t, tuple) else (t, t)
    bc2 = 1.0 - c.beta2 ** t_v
    denom = np.sqrt(v / bc2) + c.eps
    if use_m:
        bc1 = 1.0 - c.beta1 ** t_m
        return theta - c.lr * (m / bc1) / denom
    return theta - c.lr * m / denom


@dataclass
class StepState:
    """Optimizer state of one block under one configuration."""
    kind: str
    t: int = 0
    t_m0: int = 0      # step counts at which the first / second moment last started from zero
    t_v0: int = 0
    m: Optional[np.ndarray] = None
    v: Optional[np.ndarray] = None
    qm: Optional[np.ndarray] = None
    qv: Optional[np.ndarray] = None
    am: Optional[np.ndarray] = None
    av: Optional[np.ndarray] = None
    r: Optional[np.ndarray] = None
    c: Optional[np.ndarray] = None
    qr: Optional[np.ndarray] = None     # F8: codes and absmax of the row / column statistics
    qc: Optional[np.ndarray] = None
    ar: Optional[np.ndarray] = None
    ac: Optional[np.ndarray] = None


def config_kind(c: Config) -> str:
    """Which update path a tuple selects.  A32 / A16 / A8: Adam with fp32 / bf16 / 8-bit moments; R / R16:
    momentum-free RMS scaling; F: factored second moment; S / S16: SGD with momentum; G: plain gradient step
    (neither mechanism, hence no state, whatever bit-width the tuple names); R8 / S8: the 8-bit forms of R / S;
    F16 / F8: factored with bf16 / 8-bit row and column statistics."""
    if c.factored:
        return {32: "F", 16: "F16", 8: "F8"}[c.bits] if (c.adaptive and not c.momentum) else "unsupported"
    if c.adaptive and c.momentum:
        if c.bits == 8 and c.quantizer == "dynamic":
            return "A8N"                                             # Adam with 8-bit moments in the non-linear codebook
        return {32: "A32", 16: "A16", 8: "A8"}[c.bits]
    if c.adaptive and not c.momentum:
        return {32: "R", 16: "R16", 8: "R8"}[c.bits]
    if not c.adaptive and c.momentum:
        return {32: "S", 16: "S16", 8: "S8"}[c.bits]
    return "G"


def step_init(c: Config, numel: int, rows: int, cols: int, qblock: int = 256) -> StepState:
    kind = config_kind(c)
    nq = (numel + qblock - 1) // qblock
    if kind in ("A32", "A16"):
        return StepState(kind, m=np.zeros(numel, F64), v=np.zeros(numel, F64))
    if kind == "R16":
        return StepState(kind, v=np.zeros(numel, F64))
    if kind == "S16":
        return StepState(kind, m=np.zeros(numel, F64))
    if kind == "G":
        return StepState(kind)
    if kind == "R8":
        return StepState(kind, qv=np.zeros(numel, np.uint8), av=np.zeros(nq, np.float32))
    if kind == "S8":
        return StepState(kind, qm=np.zeros(numel, np.int8), am=np.zeros(nq, np.float32))
    if kind == "A8":
        return StepState(kind, qm=np.zeros(numel, np.int8), qv=np.zeros(numel, np.uint8),
                         am=np.zeros(nq, np.float32), av=np.zeros(nq, np.float32))
    if kind == "A8N":
        return StepState(kind, qm=np.zeros(numel, np.uint8), qv=np.zeros(numel, np.uint8),
                         am=np.zeros(nq, np.float32), av=np.zeros(nq, np.float32))
    if kind == "R":
        return StepState(kind, v=np.zeros(numel, F64))
    if kind in ("F", "F16", "F8"):
        if cols <= 1:
            raise ValueError("the factored configuration needs a matrix block")
        if kind == "F8":
            return StepState(kind, qr=np.zeros(rows, np.uint8), qc=np.zeros(cols, np.uint8),
                             ar=np.zeros((rows + qblock - 1) // qblock, np.float32),
                             ac=np.zeros((cols + qblock - 1) // qblock, np.float32))
        return StepState(kind, r=np.zeros(rows, F64), c=np.zeros(cols, F64))
    if kind == "S":
        return StepState(kind, m=np.zeros(numel, F64))
    raise ValueError("unsupported configuration tuple")


def _factored_stored(st: StepState, qblock: int):
    """Row and column statistics of a factored state as they are stored, in double."""
    if st.kind == "F8":
        return dequantize8(st.qr, st.ar, False, qblock), dequantize8(st.qc, st.ac, False, qblock)
    return np.asarray(st.r, F64), np.asarray(st.c, F64)


def step(theta: np.ndarray, g: np.ndarray, st: StepState, c: Config, rows: int, cols: int,
         qblock: int = 256) -> np.ndarray:
    """One optimizer step of one block; returns the new parameters (float64)
    and updates ``st`` in place.  ``st.t`` counts steps from 1."""
    theta = np.asarray(theta, dtype=F64)
    g = np.asarray(g, dtype=F64)
    st.t += 1
    t = (max(1, st.t - st.t_m0), max(1, st.t - st.t_v0))     # gradients each moment has seen, this one included
    theta_in = theta
    theta, g = _prologue(theta, g, c)
    if st.kind == "A32":
        st.m = c.beta1 * st.m + (1.0 - c.beta1) * g
        st.v = c.beta2 * st.v + (1.0 - c.beta2) * g * g
        return _adam_apply(theta, st.m, st.v, c, t, True)
    # 16-bit states: the stored moments are bf16; the update uses the new moments before they are rounded for
    # storage (the same convention as the 8-bit path)
    if st.kind == "A16":
        m = c.beta1 * st.m + (1.0 - c.beta1) * g
        v = c.beta2 * st.v + (1.0 - c.beta2) * g * g
        st.m, st.v = round_bf16(m), round_bf16(v)
        return _adam_apply(theta, m, v, c, t, True)
    if st.kind == "R16":
        v = c.beta2 * st.v + (1.0 - c.beta2) * g * g
        st.v = round_bf16(v)
        return _adam_apply(theta, g, v, c, t, False)
    if st.kind == "S16":
        m = c.beta1 * st.m + g
        st.m = round_bf16(m)
        return theta - c.lr * m
    if st.kind == "G":
        return theta - c.lr * g
    # 8-bit single-moment rules: dequantise, update, use the un-requantised moment, requantise (as in A8)
    if st.kind == "R8":
        v = dequantize8(st.qv, st.av, False, qblock)
        v = c.beta2 * v + (1.0 - c.beta2) * g * g
        theta = _adam_apply(theta, g, v, c, t, False)
        st.qv, st.av = quantize8(v, False, qblock)
        return theta
    if st.kind == "S8":
        m = dequantize8(st.qm, st.am, True, qblock)
        m = c.beta1 * m + g
        theta = theta - c.lr * m
        st.qm, st.am = quantize8(m, True, qblock)
        return theta
    if st.kind == "A8":
        m = dequantize8(st.qm, st.am, True, qblock)
        v = dequantize8(st.qv, st.av, False, qblock)
        m = c.beta1 * m + (1.0 - c.beta1) * g
        v = c.beta2 * v + (1.0 - c.beta2) * g * g
        theta = _adam_apply(theta, m, v, c, t, True)      # uses the un-requantised moments
        st.qm, st.am = quantize8(m, True, qblock)
        st.qv, st.av = quantize8(v, False, qblock)
        return theta
    if st.kind == "A8N":
        m = dequantize8_dynamic(st.qm, st.am, True, qblock)
        v = dequantize8_dynamic(st.qv, st.av, False, qblock)
        m = c.beta1 * m + (1.0 - c.beta1) * g
        v = c.beta2 * v + (1.0 - c.beta2) * g * g
        theta = _adam_apply(theta, m, v, c, t, True)      # uses the un-requantised moments
        st.qm, st.am = quantize8_dynamic(m, True, qblock)
        st.qv, st.av = quantize8_dynamic(v, False, qblock)
        return theta
    if st.kind == "R":
        st.v = c.beta2 * st.v + (1.0 - c.beta2) * g * g
        return _adam_apply(theta, g, st.v, c, t, False)
    if st.kind in ("F", "F16", "F8"):
        # the row and column statistics are read as stored; the update uses the new ones before they are rounded for
        # storage (the convention of every reduced-precision state here)
        r_old, c_old = _factored_stored(st, qblock)
        t_v = t[1]
        beta2 = 1.0 - float(t_v) ** -0.8 if c.af_beta2_schedule else c.beta2
        G2 = (g * g + c.af_eps1).reshape(rows, cols)
        r = beta2 * r_old + (1.0 - beta2) * G2.mean(axis=1)
        cc = beta2 * c_old + (1.0 - beta2) * G2.mean(axis=0)
        rm = float(r.mean())
        if rm == 0.0:
            v = np.zeros(rows * cols, F64)
        else:
            v = (np.outer(r, cc) / rm).reshape(-1)
        if st.kind == "F":
            st.r, st.c = r, cc
        elif st.kind == "F16":
            st.r, st.c = round_bf16(r), round_bf16(cc)
        else:
            st.qr, st.ar = quantize8(r, False, qblock)
            st.qc, st.ac = quantize8(cc, False, qblock)
        if not (c.af_beta2_schedule or c.af_clip > 0.0 or c.af_relative_step):
            return _adam_apply(theta, g, v, c, t, False)
        # Adafactor's remaining parts.  theta_in: the parameters before this step (the relative step size is taken from
        # them); a decoupled decay then uses that step size in place of lr.
        bc2 = 1.0 if c.af_beta2_schedule else 1.0 - c.beta2 ** t_v
        u = g / (np.sqrt(v / bc2) + c.eps)
        if c.af_clip > 0.0:
            u = u / max(1.0, math.sqrt(float(np.mean(u * u))) / c.af_clip)
        alpha = c.lr
        if c.af_relative_step:
            alpha = max(1e-3, math.sqrt(float(np.mean(theta_in * theta_in)))) * min(1e-2, 1.0 / math.sqrt(float(t_v)))
            if c.weight_decay != 0.0 and c.decoupled_wd:
                theta = theta_in * (1.0 - alpha * c.weight_decay)
        return theta - alpha * u
    if st.kind == "S":
        st.m = c.beta1 * st.m + g
        return theta - c.lr * st.m
    raise ValueError("unsupported configuration tuple")


# ----------------------------------------------------------------------------
# Re-configuration with state inheritance (online variant, Sec. 3.1 remark and
# the appendix study "online reallocation with state inheritance").  The paper
# says only that compatible optimizer states are migrated when possible; the
# reading here:
#   * a first moment is inherited between configurations of the same family
#     (Adam-type averages A32 / A16 / A8, or momentum buffers S / S16 / S8);
#   * an element-wise second moment (A*, R*) is inherited by any configuration
#     with an element-wise second moment; by a factored one as its row and
#     column means; a factored one becomes r_i c_j / mean(r) element-wise;
#   * the value is re-stored in the new precision (fp32, bf16, 8-bit codes);
#   * a moment that cannot be inherited starts from zero, and its bias
#     correction restarts (its start step becomes the current step count).
# ----------------------------------------------------------------------------

_M_FAMILY = {"A32": "avg", "A16": "avg", "A8": "avg", "S": "sum", "S16": "sum", "S8": "sum"}
_V_FAMILY = {"A32": "full", "A16": "full", "A8": "full", "R": "full", "R16": "full", "R8": "full",
             "F": "factored", "F16": "factored", "F8": "factored"}
_BITS = {"A32": 32, "A16": 16, "A8": 8, "R": 32, "R16": 16, "R8": 8, "S": 32, "S16": 16, "S8": 8,
         "F": 32, "F16": 16, "F8": 8, "G": 32}


def _moment_value(st: StepState, which: str, rows: int, cols: int, qblock: int) -> Optional[np.ndarray]:
    """The moment as the old configuration holds it, in double (None if it has none)."""
    if which == "m":
        if st.kind in ("A8", "S8"):
            return dequantize8(st.qm, st.am, True, qblock)
        return None if st.m is None else np.asarray(st.m, F64)
    if st.kind in ("A8", "R8"):
        return dequantize8(st.qv, st.av, False, qblock)
    if _V_FAMILY.get(st.kind) == "factored":
        r, c = _factored_stored(st, qblock)
        rm = float(np.mean(r))
        return np.zeros(rows * cols, F64) if rm == 0.0 else (np.outer(r, c) / rm).reshape(-1)
    return None if st.v is None else np.asarray(st.v, F64)


def reconfigure(st: StepState, c_new: Config, rows: int, cols: int, inherit: bool = True, qblock: int = 256) -> StepState:
    """The state of one block under ``c_new``, given its state ``st`` under the old configuration after ``st.t`` steps."""
    numel = rows * cols
    kind = config_kind(c_new)
    new = step_init(c_new, numel, rows, cols, qblock)
    new.t = st.t
    new.t_m0 = new.t_v0 = st.t                                   # until inherited below
    old_m = _moment_value(st, "m", rows, cols, qblock) if inherit and _M_FAMILY.get(st.kind) == _M_FAMILY.get(kind) else None
    old_v = _moment_value(st, "v", rows, cols, qblock) if inherit and st.kind in _V_FAMILY and kind in _V_FAMILY else None
    bits = _BITS[kind]
    if kind in _M_FAMILY and old_m is not None:
        new.t_m0 = st.t_m0
        if bits == 8:
            new.qm, new.am = quantize8(old_m, True, qblock)
        else:
            new.m = round_bf16(old_m) if bits == 16 else old_m.astype(np.float32).astype(F64)
    if kind in _V_FAMILY and old_v is not None:
        new.t_v0 = st.t_v0
        if _V_FAMILY[kind] == "factored":
            if _V_FAMILY[st.kind] == "factored":
                r, c = _factored_stored(st, qblock)                 # factored -> factored: the statistics themselves
            else:
                V = old_v.reshape(rows, cols)
                r, c = V.mean(axis=1), V.mean(axis=0)
            if bits == 8:
                new.qr, new.ar = quantize8(r, False, qblock)
                new.qc, new.ac = quantize8(c, False, qblock)
            elif bits == 16:
                new.r, new.c = round_bf16(r), round_bf16(c)
            else:
                new.r, new.c = r.astype(np.float32).astype(F64), c.astype(np.float32).astype(F64)
        elif bits == 8:
            new.qv, new.av = quantize8(old_v, False, qblock)
        else:
            new.v = round_bf16(old_v) if bits == 16 else old_v.astype(np.float32).astype(F64)
    return new


# ----------------------------------------------------------------------------
# Hand-over from the sampling window with its moments (Algorithm 1 moves from
# "Warmup and diagnostics" to "Training" without saying what the new optimizer
# starts from).  Reading, per block, with T_w observations in the window:
#   * an Adam-type first moment whose beta1 equals the window's beta_m (as
#     fp32 numbers) starts from m_hat; an SGD momentum buffer with that
#     coefficient starts from m_hat / (1 - beta_m): what m <- beta*m + g would
#     have built from the same gradients;
#   * a second moment whose beta2 equals the window's beta_v starts from v_hat;
#   * such a moment has seen T_w gradients (its start step is -T_w); storage
#     and every other moment as in a re-configuration.
# ----------------------------------------------------------------------------

def warm_start(win: StatsState, c: Config, rows: int, cols: int, o: Opts, qblock: int = 256) -> StepState:
    """The initial state of one block under ``c`` when the window's moments are carried into training."""
    kind = config_kind(c)
    same_m = np.float32(c.beta1) == np.float32(o.beta_m)
    same_v = np.float32(c.beta2) == np.float32(o.beta_v)
    if _M_FAMILY.get(kind) == "sum":
        held = StepState("S", m=win.m / (1.0 - o.beta_m) if same_m else None)
    else:
        held = StepState("A32", m=win.m.copy() if same_m else None, v=win.v.copy() if same_v else None)
    held.t = 0
    held.t_m0 = held.t_v0 = -win.t
    return reconfigure(held, c, rows, cols, True, qblock)


# ----------------------------------------------------------------------------
# O7. Block partitioning (Appendix on block partitioning, Algorithm 2).
#
# Input: candidate units in forward order, with parameter counts n_j and
# normalised diagnostic vectors z_j; weights w_k; n_min = alpha * |Theta|; the
# statistic-difference threshold tau (None: the upper quartile of all pairwise
# Delta among the candidate units, as the paper's implementation sets it).
# Delta(U_a, U_b) = max_k w_k |z_{a,k} - z_{b,k}|.
#
# The algorithm's verbs are loose; the reading taken here, step by step:
#   * every gap between adjacent units is a candidate boundary;
#   * a temporary block made of several units has the size-weighted mean of
#     their z as its diagnostic vector;
#   * minimum-size filtering: while some temporary block is smaller than n_min
#     (and more than one block is left), the first such block is merged into
#     the adjacent block with the smaller Delta to it (ties: the smaller
#     neighbour, then the left one);
#   * block formation: a boundary between adjacent temporary blocks survives
#     iff their Delta exceeds tau (both satisfy the size constraint after the
#     filtering); each decision is taken on the temporary blocks as the
#     filtering left them, so the result does not depend on scan order;
#   * post-processing, split: a block made of several temporary blocks is cut
#     where the Delta between the weighted means of its two sides is largest,
#     provided that Delta exceeds tau and both sides reach n_min; repeated on
#     both halves;
#   * post-processing, re-merge: the minimum-size filtering once more.
# Returns (block index of every unit, tau used).
# ----------------------------------------------------------------------------

def partition_delta(za: np.ndarray, zb: np.ndarray, w: np.ndarray) -> float:
    return float(np.max(w * np.abs(za - zb)))


def _mean_z(sizes: Sequence[int], Z: np.ndarray, members: Sequence[int]) -> np.ndarray:
    """Size-weighted mean of the members' vectors, accumulated in member order as offsets from the first member's
    vector (so that units with identical statistics average to exactly that vector)."""
    first = Z[members[0]]
    acc = np.zeros(Z.shape[1], F64)
    tot = 0.0
    for j in members:
        acc = acc + float(sizes[j]) * (Z[j] - first)
        tot += float(sizes[j])
    return first + acc / tot


def _size_filter(blocks: List[List[int]], sizes: Sequence[int], Z: np.ndarray, w: np.ndarray, n_min: float) -> List[List[int]]:
    blocks = [list(b) for b in blocks]
    while len(blocks) > 1:
        small = next((i for i, b in enumerate(blocks) if sum(sizes[j] for j in b) < n_min), None)
        if small is None:
            break
        zs = _mean_z(sizes, Z, blocks[small])
        cands = []
        for nb in (small - 1, small + 1):
            if 0 <= nb < len(blocks):
                cands.append((partition_delta(zs, _mean_z(sizes, Z, blocks[nb]), w), sum(sizes[j] for j in blocks[nb]), nb))
        cands.sort()                                   # smaller Delta, then smaller neighbour, then the left one
        nb = cands[0][2]
        lo, hi = min(small, nb), max(small, nb)
        blocks[lo:hi + 1] = [blocks[lo] + blocks[hi]]
    return blocks


def partition_blocks(sizes: Sequence[int], Z: np.ndarray, w: Optional[Sequence[float]] = None, alpha: float = 0.0,
                     tau: Optional[float] = None):
    Z = np.asarray(Z, F64)
    m, K = Z.shape
    w = np.ones(K, F64) if w is None else np.asarray(w, F64)
    n_min = alpha * float(sum(sizes))
    if tau is None:
        pair = [partition_delta(Z[a], Z[b], w) for a in range(m) for b in range(a + 1, m)]
        tau = quantile_linear(np.asarray(pair, F64), 0.75) if pair else 0.0
    # minimum-size filtering on the candidate units
    temp = _size_filter([[j] for j in range(m)], sizes, Z, w, n_min)
    # block formation
    formed: List[List[List[int]]] = [[temp[0]]]
    for a in range(len(temp) - 1):
        if partition_delta(_mean_z(sizes, Z, temp[a]), _mean_z(sizes, Z, temp[a + 1]), w) > tau:
            formed.append([temp[a + 1]])
        else:
            formed[-1].append(temp[a + 1])
    # post-processing: split where the two sides are clearly separated
    def split(parts: List[List[int]]) -> List[List[List[int]]]:
        best, best_cut = -1.0, -1
        for cut in range(1, len(parts)):
            left = [j for p in parts[:cut] for j in p]
            right = [j for p in parts[cut:] for j in p]
            if sum(sizes[j] for j in left) < n_min or sum(sizes[j] for j in right) < n_min:
                continue
            d = partition_delta(_mean_z(sizes, Z, left), _mean_z(sizes, Z, right), w)
            if d > best:
                best, best_cut = d, cut
        if best_cut < 0 or not best > tau:
            return [parts]
        return split(parts[:best_cut]) + split(parts[best_cut:])
    final = [[j for p in blk for j in p] for f in formed for blk in split(f)]
    # post-processing: re-merge what is still too small
    final = _size_filter(final, sizes, Z, w, n_min)
    ids = np.zeros(m, np.int32)
    for b, members in enumerate(final):
        ids[members] = b
    return ids, float(tau)
