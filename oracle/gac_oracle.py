"""ctypes front end of the CPU oracle in ``gac_oracle.c``.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
CPU-baseline leg of the benchmark may import this module.  The CUDA library
and its Python binding never do, and the two share no code.

The functions here only marshal arguments and walk the tensor list in list
order (the "flattened concatenation of all trainable parameter gradients",
App. A.1); all arithmetic is in the C file.

Tensors are CPU ``torch`` tensors (float32 or bfloat16) or ``numpy`` arrays
(float32, or uint16 holding bfloat16 bit patterns); they must be contiguous.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gac_oracle.c")
_LIB = os.path.join(_HERE, "libgac_oracle.so")

F32, BF16 = 0, 1
SAFE, PROJECT, VIOLATION = 0, 1, 2
MODE_ADAPTIVE, MODE_FIXED = 0, 1
STATE_RAW, STATE_PROJECTED, STATE_HOLD = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no optimisation flags that change fp
    semantics: no -ffast-math, and -ffp-contract=off so a*b+c is two roundings
    exactly as written)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Acc(ctypes.Structure):
    _fields_ = [("sum", ctypes.c_double * 3), ("comp", ctypes.c_double * 3)]


class _HParams(ctypes.Structure):
    _fields_ = [("c_low", ctypes.c_double), ("c_high", ctypes.c_double),
                ("eps", ctypes.c_double), ("beta", ctypes.c_double),
                ("mode", ctypes.c_int32), ("state_mode", ctypes.c_int32),
                ("alpha_fixed", ctypes.c_double),
                ("zero_on_violation", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("clip_max_norm", ctypes.c_double), ("clip_eps", ctypes.c_double)]


class _AdamW(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double)]


class _Decision(ctypes.Structure):
    _fields_ = [("dot", ctypes.c_double), ("gg", ctypes.c_double), ("dd", ctypes.c_double),
                ("cosine", ctypes.c_double), ("alpha", ctypes.c_double),
                ("coef64", ctypes.c_double), ("coef", ctypes.c_float),
                ("regime", ctypes.c_int32), ("nonfinite", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, u64, i32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int
        L.orc_acc_init.argtypes = [ctypes.POINTER(_Acc)]
        L.orc_stats_accumulate.argtypes = [ctypes.POINTER(_Acc), vp, i32, vp, i32, u64, i32]
        L.orc_acc_value.argtypes = [ctypes.POINTER(_Acc), ctypes.c_double * 3]
        L.orc_acc_merge.argtypes = [ctypes.POINTER(_Acc), ctypes.POINTER(_Acc)]
        L.orc_stats_pairwise.argtypes = [vp, i32, vp, i32, u64, ctypes.c_double * 3]
        L.orc_decide.argtypes = [ctypes.c_double * 3, ctypes.POINTER(_HParams), i32,
                                 ctypes.POINTER(_Decision)]
        L.orc_project.argtypes = [vp, i32, vp, i32, u64, ctypes.POINTER(_HParams), i32, i32,
                                  ctypes.c_float, i32, ctypes.c_double]
        L.orc_outgoing_sqnorm.argtypes = [ctypes.POINTER(_Acc), vp, i32, vp, i32, u64,
                                          ctypes.POINTER(_HParams), i32, ctypes.c_float, i32]
        L.orc_outgoing_sqnorm.restype = None
        L.orc_clip_scale.argtypes = [ctypes.c_double, ctypes.POINTER(_HParams)]
        L.orc_clip_scale.restype = ctypes.c_double
        L.orc_project_adamw.argtypes = [vp, i32, vp, i32, vp, vp, vp, u64, ctypes.POINTER(_HParams), i32,
                                        i32, ctypes.c_float, i32, ctypes.c_double,
                                        ctypes.POINTER(_AdamW), u64]
        L.orc_project_adamw.restype = None
        L.orc_round_to_bf16.argtypes = [vp, vp, u64]
        for f in (L.orc_acc_init, L.orc_stats_accumulate, L.orc_acc_value, L.orc_acc_merge,
                  L.orc_stats_pairwise, L.orc_decide, L.orc_project, L.orc_round_to_bf16):
            f.restype = None
        _lib = L
    return _lib


@dataclass
class HParams:
    """Algorithm 1 inputs and the gains of Eq. 3 / Eq. 5 (paper defaults)."""
    c_low: float = 0.05
    c_high: float = 0.3
    eps: float = 1e-8
    beta: float = 1.0
    mode: int = MODE_ADAPTIVE
    alpha_fixed: float = 0.0
    state_mode: int = STATE_RAW
    zero_on_violation: int = 0
    clip_max_norm: float = 0.0      # 0 = no clipping
    clip_eps: float = 1e-6

    def c(self) -> _HParams:
        return _HParams(self.c_low, self.c_high, self.eps, self.beta, self.mode, self.state_mode,
                        self.alpha_fixed, self.zero_on_violation, 0, self.clip_max_norm,
                        self.clip_eps)


@dataclass
class Decision:
    dot: float
    gg: float
    dd: float
    cos: float
    alpha: float
    coef64: float
    coef: float          # binary32 value, held exactly in a Python float
    regime: int
    nonfinite: int
    out_norm: float = float("nan")   # norm of the outgoing gradient before clipping (set by project)
    clip_scale: float = 1.0          # factor applied by global-norm clipping (set by project)


def _ptr_dt_n(t):
    """(address, element type code, element count) of a contiguous CPU tensor/array."""
    if isinstance(t, np.ndarray):
        if not t.flags["C_CONTIGUOUS"]:
            raise ValueError("oracle needs contiguous arrays")
        if t.dtype == np.float32:
            return t.ctypes.data, F32, t.size
        if t.dtype == np.uint16:
            return t.ctypes.data, BF16, t.size
        raise TypeError(f"unsupported numpy dtype {t.dtype}")
    import torch
    if not isinstance(t, torch.Tensor) or t.device.type != "cpu" or not t.is_contiguous():
        raise TypeError("oracle needs contiguous CPU tensors")
    if t.dtype == torch.float32:
        return t.data_ptr(), F32, t.numel()
    if t.dtype == torch.bfloat16:
        return t.data_ptr(), BF16, t.numel()
    raise TypeError(f"unsupported torch dtype {t.dtype}")


def _ranges(n: int, parts: int, quantum: int = 1 << 16):
    """Fixed split of [0,n) into at most `parts` contiguous ranges."""
    if parts <= 1 or n <= quantum:
        return [(0, n)]
    per = -(-n // parts)
    per = -(-per // quantum) * quantum
    return [(lo, min(lo + per, n)) for lo in range(0, n, per)]


_ELEM_BYTES = {F32: 4, BF16: 2}


def stats(g_list: Sequence, d_list: Sequence, first_step: bool = False, threads: int = 1):
    """(dot, gg, dd) over the concatenation of the list, Neumaier-compensated fp64
    (App. A.1).  threads > 1 accumulates fixed contiguous ranges separately and
    merges them in range order, so the result does not depend on scheduling."""
    L = lib()
    jobs = []
    for g, d in zip(g_list, d_list):
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, nd = _ptr_dt_n(d)
        if n != nd:
            raise ValueError("g and d differ in length")
        for lo, hi in _ranges(n, threads):
            jobs.append((gp + lo * _ELEM_BYTES[gdt], gdt, dp + lo * _ELEM_BYTES[ddt], ddt, hi - lo))

    def run(job):
        a = _Acc()
        L.orc_acc_init(ctypes.byref(a))
        L.orc_stats_accumulate(ctypes.byref(a), job[0], job[1], job[2], job[3], job[4],
                               1 if first_step else 0)
        return a

    total = _Acc()
    L.orc_acc_init(ctypes.byref(total))
    if threads <= 1:
        for job in jobs:   # one running sum over the whole concatenation
            L.orc_stats_accumulate(ctypes.byref(total), job[0], job[1], job[2], job[3], job[4],
                                   1 if first_step else 0)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            for a in ex.map(run, jobs):
                L.orc_acc_merge(ctypes.byref(total), ctypes.byref(a))
    out = (ctypes.c_double * 3)()
    L.orc_acc_value(ctypes.byref(total), out)
    return float(out[0]), float(out[1]), float(out[2])


def stats_pairwise(g_list: Sequence, d_list: Sequence):
    """Same three sums with recursive pairwise summation per tensor (the second,
    independent summation order)."""
    L = lib()
    tot = [0.0, 0.0, 0.0]
    for g, d in zip(g_list, d_list):
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, _ = _ptr_dt_n(d)
        out = (ctypes.c_double * 3)()
        L.orc_stats_pairwise(gp, gdt, dp, ddt, n, out)
        for k in range(3):
            tot[k] += float(out[k])
    return tuple(tot)


def decide(sums, hp: HParams, first_step: bool = False) -> Decision:
    """Cosine (App. A.1), regime (Algorithm 1) and gains (Eq. 5 / Eq. 3)."""
    L = lib()
    s = (ctypes.c_double * 3)(*sums)
    o = _Decision()
    chp = hp.c()
    L.orc_decide(s, ctypes.byref(chp), 1 if first_step else 0, ctypes.byref(o))
    return Decision(o.dot, o.gg, o.dd, o.cosine, o.alpha, o.coef64, float(o.coef), o.regime,
                    o.nonfinite)


def outgoing_norm(g_list: Sequence, d_list: Sequence, hp: HParams, dec: Decision,
                  first_step: bool = False, coef: Optional[float] = None) -> float:
    """Euclidean norm of the (unrounded) gradient that a safe or projection step
    sends on, by brute force over every element."""
    L = lib()
    chp = hp.c()
    k = dec.coef if coef is None else float(np.float32(coef))
    acc = _Acc()
    L.orc_acc_init(ctypes.byref(acc))
    for g, d in zip(g_list, d_list):
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, _ = _ptr_dt_n(d)
        L.orc_outgoing_sqnorm(ctypes.byref(acc), gp, gdt, dp, ddt, n, ctypes.byref(chp), dec.regime,
                              ctypes.c_float(k), 1 if first_step else 0)
    out = (ctypes.c_double * 3)()
    L.orc_acc_value(ctypes.byref(acc), out)
    return float(out[0]) ** 0.5


def project(g_list: Sequence, d_list: Sequence, hp: HParams, dec: Decision,
            first_step: bool = False, coef: Optional[float] = None, threads: int = 1) -> None:
    """In-place rank-one update of g and refresh of the stored direction d
    (App. A.2), followed -- when hp.clip_max_norm > 0 -- by global-norm clipping
    of what a safe or projection step sends on.  `coef` overrides the decision's
    binary32 coefficient.  Records out_norm and clip_scale in `dec`."""
    L = lib()
    chp = hp.c()
    k = dec.coef if coef is None else float(np.float32(coef))
    scale = 1.0
    if hp.clip_max_norm > 0 and not dec.nonfinite and dec.regime != VIOLATION:
        dec.out_norm = outgoing_norm(g_list, d_list, hp, dec, first_step, coef)
        scale = float(L.orc_clip_scale(dec.out_norm ** 2, ctypes.byref(chp)))
    dec.clip_scale = scale
    jobs = []
    for g, d in zip(g_list, d_list):
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, nd = _ptr_dt_n(d)
        if nd != n or (ddt == BF16 and gdt != BF16):
            raise TypeError("stored direction must be float32 (or bfloat16 with a bfloat16 gradient) "
                            "of the gradient's length")
        for lo, hi in _ranges(n, threads):
            jobs.append((gp + lo * _ELEM_BYTES[gdt], gdt, dp + lo * _ELEM_BYTES[ddt], ddt, hi - lo))

    def run(job):
        L.orc_project(job[0], job[1], job[2], job[3], job[4], ctypes.byref(chp), dec.regime,
                      dec.nonfinite, ctypes.c_float(k), 1 if first_step else 0,
                      ctypes.c_double(scale))

    if threads <= 1:
        for job in jobs:
            run(job)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, jobs))


def step(g_list, d_list, hp: HParams, first_step: bool = False, threads: int = 1) -> Decision:
    """One whole GAC step of Algorithm 1 on the list: stats, decision, in-place update."""
    dec = decide(stats(g_list, d_list, first_step, threads), hp, first_step)
    project(g_list, d_list, hp, dec, first_step, threads=threads)
    return dec


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 values to bfloat16 bit patterns (uint16)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().orc_round_to_bf16(x.ctypes.data, out.ctypes.data, x.size)
    return out


class RunningStats:
    """The same three sums, fed one tensor pair at a time so that a list larger
    than host memory can be streamed through in list order."""

    def __init__(self, first_step: bool = False, threads: int = 1):
        self.first_step, self.threads = first_step, threads
        self._tot = _Acc()
        lib().orc_acc_init(ctypes.byref(self._tot))

    def add(self, g, d) -> None:
        L = lib()
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, nd = _ptr_dt_n(d)
        if n != nd:
            raise ValueError("g and d differ in length")
        fs = 1 if self.first_step else 0
        jobs = [(gp + lo * _ELEM_BYTES[gdt], gdt, dp + lo * _ELEM_BYTES[ddt], ddt, hi - lo)
                for lo, hi in _ranges(n, self.threads)]
        if len(jobs) == 1:
            j = jobs[0]
            L.orc_stats_accumulate(ctypes.byref(self._tot), j[0], j[1], j[2], j[3], j[4], fs)
            return

        def run(j):
            a = _Acc()
            L.orc_acc_init(ctypes.byref(a))
            L.orc_stats_accumulate(ctypes.byref(a), j[0], j[1], j[2], j[3], j[4], fs)
            return a

        with ThreadPoolExecutor(max_workers=self.threads) as ex:
            for a in ex.map(run, jobs):
                L.orc_acc_merge(ctypes.byref(self._tot), ctypes.byref(a))

    def value(self):
        out = (ctypes.c_double * 3)()
        lib().orc_acc_value(ctypes.byref(self._tot), out)
        return float(out[0]), float(out[1]), float(out[2])


@dataclass
class AdamW:
    """AdamW hyper-parameters; defaults are the paper's (Table 2)."""
    lr: float = 1e-6
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 1e-2

    def c(self) -> _AdamW:
        return _AdamW(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay)


def project_adamw(g_list, d_list, p_list, m_list, v_list, hp: HParams, dec: Decision, opt: AdamW,
                  t: int, first_step: bool = False, coef: Optional[float] = None) -> bool:
    """The GAC update consumed directly by AdamW (Algorithm 1's parameter update with
    the optimizer of Table 2): p, m, v and the stored direction d change in place, g is
    only read.  `t` is the number of updates applied so far including this one.
    Returns True when the update was applied (False on a skipped step)."""
    L = lib()
    chp, copt = hp.c(), opt.c()
    k = dec.coef if coef is None else float(np.float32(coef))
    scale = 1.0
    if hp.clip_max_norm > 0 and not dec.nonfinite and dec.regime != VIOLATION:
        dec.out_norm = outgoing_norm(g_list, d_list, hp, dec, first_step, coef)
        scale = float(L.orc_clip_scale(dec.out_norm ** 2, ctypes.byref(chp)))
    dec.clip_scale = scale
    for g, d, p, m, v in zip(g_list, d_list, p_list, m_list, v_list):
        gp, gdt, n = _ptr_dt_n(g)
        dp, ddt, dn = _ptr_dt_n(d)
        ptrs = [dp]
        for x in (p, m, v):
            xp, xdt, xn = _ptr_dt_n(x)
            if xdt != F32 or xn != n:
                raise TypeError("p, m, v must be float32 of the gradient's length")
            ptrs.append(xp)
        L.orc_project_adamw(gp, gdt, ptrs[0], ddt, ptrs[1], ptrs[2], ptrs[3], n, ctypes.byref(chp),
                            dec.regime, dec.nonfinite, ctypes.c_float(k), 1 if first_step else 0,
                            ctypes.c_double(scale), ctypes.byref(copt), t)
    return (not dec.nonfinite) and dec.regime != VIOLATION
