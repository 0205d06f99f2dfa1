"""Thin ctypes binding of the C ABI in ``include/gac.h``: argument marshalling
only.  Every step of the path runs in the CUDA library; if the library is
missing this module raises -- there is no CPU fallback.

PyTorch appears here only as the owner of device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# GAC_B200_LIBRARY selects another build of the same library (a debug build, or one compiled with
# another launch-geometry table through -DGAC_GEOMETRY_HEADER); the default is the in-tree build.
LIB_PATH = os.environ.get("GAC_B200_LIBRARY") or os.path.join(_HERE, "libgac_b200.so")

GAC_OK, GAC_ERR_INVALID_ARG, GAC_ERR_DTYPE, GAC_ERR_CUDA, GAC_ERR_STATE, GAC_ERR_NONFINITE, \
    GAC_ERR_TIMEOUT = range(7)
GAC_F32, GAC_BF16 = 0, 1
GAC_REGIME_SAFE, GAC_REGIME_PROJECT, GAC_REGIME_VIOLATION = 0, 1, 2
GAC_MODE_ADAPTIVE, GAC_MODE_FIXED = 0, 1
GAC_STATE_RAW, GAC_STATE_PROJECTED, GAC_STATE_HOLD, GAC_STATE_EXCHANGE = 0, 1, 2, 3
GAC_SET_G, GAC_SET_D = 0, 1
REGIME_NAMES = {0: "safe", 1: "project", 2: "violation"}


class gac_tensor(ctypes.Structure):
    _fields_ = [("g", ctypes.c_void_p), ("d", ctypes.c_void_p), ("numel", ctypes.c_uint64)]


class gac_hparams(ctypes.Structure):
    _fields_ = [("c_low", ctypes.c_double), ("c_high", ctypes.c_double), ("eps", ctypes.c_double),
                ("beta", ctypes.c_double), ("mode", ctypes.c_int32), ("state_mode", ctypes.c_int32),
                ("alpha_fixed", ctypes.c_double), ("zero_on_violation", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("clip_max_norm", ctypes.c_double),
                ("clip_eps", ctypes.c_double)]


class gac_result(ctypes.Structure):
    _fields_ = [("dot", ctypes.c_double), ("gg", ctypes.c_double), ("dd", ctypes.c_double),
                ("cos", ctypes.c_double), ("alpha", ctypes.c_double), ("coef64", ctypes.c_double),
                ("coef", ctypes.c_float), ("regime", ctypes.c_int32), ("nonfinite", ctypes.c_int32),
                ("staleness", ctypes.c_uint32), ("step", ctypes.c_uint64),
                ("out_norm", ctypes.c_double), ("clip_scale", ctypes.c_double),
                ("applied_steps", ctypes.c_uint64), ("g_set", ctypes.c_uint32),
                ("out_set", ctypes.c_uint32), ("ref_lost", ctypes.c_uint32),
                ("timed_out", ctypes.c_uint32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class gac_opt_tensor(ctypes.Structure):
    _fields_ = [("p", ctypes.c_void_p), ("m", ctypes.c_void_p), ("v", ctypes.c_void_p)]


class gac_adamw(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double)]


class gac_info(ctypes.Structure):
    _fields_ = [("total_elems", ctypes.c_uint64), ("n_chunks", ctypes.c_uint64),
                ("n_tensors", ctypes.c_uint32), ("grid", ctypes.c_uint32),
                ("threads", ctypes.c_uint32), ("chunk_elems", ctypes.c_uint32),
                ("launches", ctypes.c_uint64), ("misaligned_tensors", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32)]


EXPORTS = ["gac_default_hparams", "gac_init", "gac_stats", "gac_stats_partial", "gac_decide",
           "gac_project", "gac_free", "gac_last_error", "gac_set_launch", "gac_get_info",
           "gac_stats_static", "gac_default_adamw", "gac_attach_adamw", "gac_project_adamw",
           "gac_rebind", "gac_next_gradient_set", "gac_exchange_bytes", "gac_exchange_attach",
           "gac_stats_exchange", "gac_decide_exchange"]

_lib = None


class GacError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gac status {status}: {message}")
        self.status = status


def load_library() -> ctypes.CDLL:
    """Loads the in-tree CUDA library; raises if it was not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2603_01501_b200.build` (needs nvcc); "
                          "this package has no CPU fallback")
    L = ctypes.CDLL(LIB_PATH)
    vp, u32, u64, i32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int
    L.gac_default_hparams.argtypes = [ctypes.POINTER(gac_hparams)]
    L.gac_default_hparams.restype = None
    L.gac_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(gac_tensor), u32, i32, i32,
                           ctypes.POINTER(gac_hparams), i32]
    L.gac_stats.argtypes = [vp, u64, u32, vp, ctypes.POINTER(gac_result)]
    L.gac_stats_partial.argtypes = [vp, u64, u32, vp, vp]
    L.gac_decide.argtypes = [vp, vp, vp, ctypes.POINTER(gac_result)]
    L.gac_project.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(gac_result)]
    L.gac_free.argtypes = [vp]
    L.gac_last_error.argtypes = [vp]
    L.gac_last_error.restype = ctypes.c_char_p
    L.gac_set_launch.argtypes = [vp, i32, i32]
    L.gac_get_info.argtypes = [vp, ctypes.POINTER(gac_info)]
    L.gac_stats_static.argtypes = [ctypes.POINTER(gac_tensor), u32, i32, i32,
                                   ctypes.POINTER(gac_hparams), u64, u32, i32, vp, vp]
    L.gac_stats_static.restype = i32
    L.gac_rebind.argtypes = [vp, ctypes.POINTER(gac_tensor), u32]
    L.gac_rebind.restype = i32
    L.gac_next_gradient_set.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    L.gac_next_gradient_set.restype = i32
    L.gac_default_adamw.argtypes = [ctypes.POINTER(gac_adamw)]
    L.gac_default_adamw.restype = None
    L.gac_attach_adamw.argtypes = [vp, ctypes.POINTER(gac_opt_tensor), u32, u64]
    L.gac_attach_adamw.restype = i32
    L.gac_project_adamw.argtypes = [vp, vp, ctypes.POINTER(gac_adamw), ctypes.POINTER(ctypes.c_float),
                                    ctypes.POINTER(gac_result)]
    L.gac_project_adamw.restype = i32
    L.gac_exchange_bytes.argtypes = [u32]
    L.gac_exchange_bytes.restype = ctypes.c_size_t
    L.gac_exchange_attach.argtypes = [vp, u32, u32, ctypes.POINTER(vp), u32]
    L.gac_exchange_attach.restype = i32
    L.gac_stats_exchange.argtypes = [vp, u64, u32, vp]
    L.gac_stats_exchange.restype = i32
    L.gac_decide_exchange.argtypes = [vp, vp, ctypes.POINTER(gac_result)]
    L.gac_decide_exchange.restype = i32
    for name in ("gac_init", "gac_stats", "gac_stats_partial", "gac_decide", "gac_project",
                 "gac_free", "gac_set_launch", "gac_get_info"):
        getattr(L, name).restype = i32
    _lib = L
    return L


@dataclass
class HParams:
    """Algorithm 1 inputs (c_low, c_high), the cosine's eps (App. A.1) and the
    gains of Eq. 3 / Eq. 5; defaults are the paper's."""
    c_low: float = 0.05
    c_high: float = 0.3
    eps: float = 1e-8
    beta: float = 1.0
    mode: int = GAC_MODE_ADAPTIVE
    alpha_fixed: float = 0.0
    state_mode: int = GAC_STATE_RAW
    zero_on_violation: int = 0
    clip_max_norm: float = 0.0     # > 0 folds global-norm clipping into the projection pass
    clip_eps: float = 1e-6

    def c(self) -> gac_hparams:
        return gac_hparams(self.c_low, self.c_high, self.eps, self.beta, self.mode,
                           self.state_mode, self.alpha_fixed, self.zero_on_violation, 0,
                           self.clip_max_norm, self.clip_eps)


_DT = {torch.float32: GAC_F32, torch.bfloat16: GAC_BF16}


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class GacContext:
    """Owner of one ``gac_ctx``.  Keeps references to the tensors so that the
    device pointers in the chunk table stay valid."""

    def __init__(self, handle: int, g_list, d_list):
        self.handle = ctypes.c_void_p(handle)
        self._keep = (list(g_list), list(d_list))

    def _check(self, rc: int, allow_nonfinite: bool = False):
        if rc != GAC_OK and not (allow_nonfinite and rc == GAC_ERR_NONFINITE):
            raise GacError(rc, load_library().gac_last_error(self.handle).decode())

    def __del__(self):
        try:
            gac_free(self)
        except Exception:
            pass


def gac_init(g_list: Sequence[torch.Tensor], d_list: Sequence[torch.Tensor],
             hp: Optional[HParams] = None, device: Optional[int] = None) -> GacContext:
    """gac_init of the C ABI on lists of CUDA tensors (g_i, d_i)."""
    L = load_library()
    hp = hp or HParams()
    if len(g_list) != len(d_list):
        raise ValueError("g and d lists differ in length")
    n = len(g_list)
    arr = (gac_tensor * max(n, 1))()
    g_dt = d_dt = None
    for i, (g, d) in enumerate(zip(g_list, d_list)):
        if not (g.is_cuda and d.is_cuda and g.is_contiguous() and d.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
        if g.numel() != d.numel():
            raise ValueError(f"tensor {i}: g and d differ in numel")
        if g.dtype not in _DT or d.dtype not in _DT:
            raise GacError(GAC_ERR_DTYPE, f"unsupported dtype {g.dtype}/{d.dtype}")
        if g_dt is None:
            g_dt, d_dt = g.dtype, d.dtype
        elif (g.dtype, d.dtype) != (g_dt, d_dt):
            raise GacError(GAC_ERR_DTYPE, "all tensors of a list must share one (g,d) dtype pair")
        arr[i] = gac_tensor(g.data_ptr(), d.data_ptr(), g.numel())
    if device is None:
        device = g_list[0].device.index if n else torch.cuda.current_device()
    out = ctypes.c_void_p()
    chp = hp.c()
    rc = L.gac_init(ctypes.byref(out), arr, n, _DT.get(g_dt, 0), _DT.get(d_dt, 0),
                    ctypes.byref(chp), device)
    if rc != GAC_OK:
        raise GacError(rc, L.gac_last_error(None).decode())
    return GacContext(out.value, g_list, d_list)


def gac_stats(ctx: GacContext, step: int, staleness: int = 0, stream=None,
              fetch: bool = True) -> Optional[gac_result]:
    """gac_stats; with fetch=False nothing leaves the device and None is returned."""
    L = load_library()
    res = gac_result() if fetch else None
    rc = L.gac_stats(ctx.handle, step, staleness, _stream_ptr(stream),
                     ctypes.byref(res) if fetch else None)
    ctx._check(rc, allow_nonfinite=True)
    return res


def gac_stats_partial(ctx: GacContext, step: int, sums_out: torch.Tensor, staleness: int = 0,
                      stream=None) -> None:
    if not (sums_out.is_cuda and sums_out.dtype == torch.float64 and sums_out.numel() >= 3):
        raise ValueError("sums_out must be a CUDA float64 tensor of 3 elements")
    ctx._check(load_library().gac_stats_partial(ctx.handle, step, staleness, _stream_ptr(stream),
                                                sums_out.data_ptr()))


def gac_decide(ctx: GacContext, sums_in: torch.Tensor, stream=None,
               fetch: bool = True) -> Optional[gac_result]:
    if not (sums_in.is_cuda and sums_in.dtype == torch.float64 and sums_in.numel() >= 3):
        raise ValueError("sums_in must be a CUDA float64 tensor of 3 elements")
    res = gac_result() if fetch else None
    rc = load_library().gac_decide(ctx.handle, _stream_ptr(stream), sums_in.data_ptr(),
                                   ctypes.byref(res) if fetch else None)
    ctx._check(rc, allow_nonfinite=True)
    return res


def gac_exchange_bytes(world: int) -> int:
    """Size of one rank's slot array for the peer exchange of the three sums."""
    return int(load_library().gac_exchange_bytes(world))


def gac_exchange_attach(ctx: GacContext, rank: int, world: int, slots: Sequence[torch.Tensor],
                        timeout_ms: int = 0) -> None:
    """gac_exchange_attach: `slots[r]` is rank r's slot array (a zero-filled CUDA uint8 tensor of
    gac_exchange_bytes(world) bytes, or an integer device address of one mapped from a peer)."""
    arr = (ctypes.c_void_p * max(world, 1))()
    for r, t in enumerate(slots):
        if isinstance(t, torch.Tensor):
            if not (t.is_cuda and t.is_contiguous() and t.numel() * t.element_size() >= gac_exchange_bytes(world)):
                raise ValueError("a slot array must be a contiguous CUDA tensor of gac_exchange_bytes(world) bytes")
            arr[r] = t.data_ptr()
        else:
            arr[r] = int(t)
    if len(slots) != world:
        raise ValueError("one slot array per rank")
    ctx._check(load_library().gac_exchange_attach(ctx.handle, rank, world, arr, timeout_ms))
    ctx._keep_slots = list(slots)


def gac_stats_exchange(ctx: GacContext, step: int, staleness: int = 0, stream=None) -> None:
    ctx._check(load_library().gac_stats_exchange(ctx.handle, step, staleness, _stream_ptr(stream)))


def gac_decide_exchange(ctx: GacContext, stream=None, fetch: bool = True) -> Optional[gac_result]:
    """gac_decide_exchange; raises GacError(GAC_ERR_TIMEOUT) when fetching a record whose wait ran out."""
    res = gac_result() if fetch else None
    rc = load_library().gac_decide_exchange(ctx.handle, _stream_ptr(stream), ctypes.byref(res) if fetch else None)
    ctx._check(rc, allow_nonfinite=True)
    return res


def gac_project(ctx: GacContext, stream=None, coef_override: Optional[float] = None,
                fetch: bool = False) -> Optional[gac_result]:
    L = load_library()
    res = gac_result() if fetch else None
    k = ctypes.c_float(coef_override) if coef_override is not None else None
    rc = L.gac_project(ctx.handle, _stream_ptr(stream),
                       ctypes.byref(k) if k is not None else None,
                       ctypes.byref(res) if fetch else None)
    ctx._check(rc, allow_nonfinite=True)
    return res


def gac_next_gradient_set(ctx: GacContext) -> int:
    """Exchange mode: GAC_SET_G or GAC_SET_D, the buffer set the next gradient belongs in."""
    out = ctypes.c_int(0)
    ctx._check(load_library().gac_next_gradient_set(ctx.handle, ctypes.byref(out)))
    return out.value


def gac_free(ctx: GacContext) -> None:
    if ctx.handle:
        load_library().gac_free(ctx.handle)
        ctx.handle = ctypes.c_void_p(None)
    # the library no longer touches the buffers: let go of them, so that their owner can free them
    ctx._keep = ([], [])
    for extra in ("_keep_opt", "_keep_slots", "_keep_symm"):
        if hasattr(ctx, extra):
            setattr(ctx, extra, None)


def gac_set_launch(ctx: GacContext, chunk_elems: int = 0, ctas_per_sm: int = 0) -> None:
    ctx._check(load_library().gac_set_launch(ctx.handle, chunk_elems, ctas_per_sm))


def gac_get_info(ctx: GacContext) -> gac_info:
    info = gac_info()
    ctx._check(load_library().gac_get_info(ctx.handle, ctypes.byref(info)))
    return info


def gac_stats_static(g_list: Sequence[torch.Tensor], d_list: Sequence[torch.Tensor], hp: HParams,
                     step: int, result_dev: torch.Tensor, staleness: int = 0, stream=None) -> None:
    """gac_stats_static of the C ABI: the statistics and the decision of one step
    without any allocation by the library (work memory is built into it).
    `result_dev` is a caller-owned CUDA uint8 tensor of at least
    ``ctypes.sizeof(gac_result)`` bytes that receives the record on the stream;
    read it with ``result_from_tensor`` after synchronising."""
    L = load_library()
    if not (result_dev.is_cuda and result_dev.dtype == torch.uint8 and result_dev.is_contiguous()
            and result_dev.numel() >= ctypes.sizeof(gac_result) and result_dev.data_ptr() % 8 == 0):
        raise ValueError("result_dev must be an 8-byte aligned CUDA uint8 tensor of >= sizeof(gac_result) bytes")
    n = len(g_list)
    arr = (gac_tensor * max(n, 1))()
    for i, (g, d) in enumerate(zip(g_list, d_list)):
        arr[i] = gac_tensor(g.data_ptr(), d.data_ptr(), g.numel())
    chp = hp.c()
    g_dt = _DT[g_list[0].dtype] if n else 0
    d_dt = _DT[d_list[0].dtype] if n else 0
    dev = result_dev.device.index
    rc = L.gac_stats_static(arr, n, g_dt, d_dt, ctypes.byref(chp), step, staleness, dev,
                            _stream_ptr(stream), result_dev.data_ptr())
    if rc != GAC_OK:
        raise GacError(rc, L.gac_last_error(None).decode())


def result_from_tensor(t: torch.Tensor) -> gac_result:
    """Decodes a gac_result held in a uint8 tensor (copied to the host here)."""
    raw = bytes(t.detach().cpu().numpy().tobytes()[: ctypes.sizeof(gac_result)])
    return gac_result.from_buffer_copy(raw)


@dataclass
class AdamW:
    """AdamW hyper-parameters; defaults are the paper's (Table 2)."""
    lr: float = 1e-6
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 1e-2

    def c(self) -> gac_adamw:
        return gac_adamw(self.lr, self.beta1, self.beta2, self.eps, self.weight_decay)


def gac_attach_adamw(ctx: GacContext, p_list: Sequence[torch.Tensor], m_list: Sequence[torch.Tensor],
                     v_list: Sequence[torch.Tensor], applied_steps: int = 0) -> None:
    """Binds float32 parameters and AdamW moments (one per tensor of the context's list)."""
    n = len(p_list)
    arr = (gac_opt_tensor * max(n, 1))()
    for i, (p, m, v) in enumerate(zip(p_list, m_list, v_list)):
        for t in (p, m, v):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.float32):
                raise ValueError("p, m, v must be contiguous float32 CUDA tensors")
            if t.numel() != ctx._keep[0][i].numel():
                raise ValueError(f"tensor {i}: optimizer state differs in numel from the gradient")
        arr[i] = gac_opt_tensor(p.data_ptr(), m.data_ptr(), v.data_ptr())
    ctx._check(load_library().gac_attach_adamw(ctx.handle, arr, n, applied_steps))
    ctx._keep_opt = (list(p_list), list(m_list), list(v_list))


def gac_project_adamw(ctx: GacContext, opt: AdamW, stream=None, coef_override: Optional[float] = None,
                      fetch: bool = False) -> Optional[gac_result]:
    L = load_library()
    res = gac_result() if fetch else None
    k = ctypes.c_float(coef_override) if coef_override is not None else None
    copt = opt.c()
    rc = L.gac_project_adamw(ctx.handle, _stream_ptr(stream), ctypes.byref(copt),
                             ctypes.byref(k) if k is not None else None,
                             ctypes.byref(res) if fetch else None)
    ctx._check(rc, allow_nonfinite=True)
    return res


def gac_rebind(ctx: GacContext, g_list: Sequence[torch.Tensor], d_list: Sequence[torch.Tensor]) -> None:
    """Points the context at moved buffers of the same sizes (gac_rebind of the C ABI)."""
    n = len(g_list)
    arr = (gac_tensor * max(n, 1))()
    for i, (g, d) in enumerate(zip(g_list, d_list)):
        if not (g.is_cuda and d.is_cuda and g.is_contiguous() and d.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
        arr[i] = gac_tensor(g.data_ptr(), d.data_ptr(), g.numel())
    ctx._check(load_library().gac_rebind(ctx.handle, arr, n))
    ctx._keep = (list(g_list), list(d_list))
