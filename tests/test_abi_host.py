"""Host-only checks of the C ABI: the library loads without a GPU, exports
every function the header declares, its structs have the layout the Python
binding assumes, and argument errors are reported before any device work."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gac.h")


@pytest.fixture(scope="module")
def lib():
    gbuild.build()
    return gb.load_library()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gac_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert {"gac_init", "gac_stats", "gac_project", "gac_free"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in gac.h but not exported"
    assert sorted(gb.EXPORTS) == [n for n in names if n in gb.EXPORTS]
    assert set(names) <= set(gb.EXPORTS), set(names) - set(gb.EXPORTS)


def test_struct_layouts_match_the_header(tmp_path):
    src = tmp_path / "layout.c"
    src.write_text(r'''
#include <stdio.h>
#include <stddef.h>
#include "gac.h"
int main(void) {
  printf("%zu %zu %zu %zu\n", sizeof(gac_tensor), sizeof(gac_hparams), sizeof(gac_result), sizeof(gac_info));
  printf("%zu %zu %zu %zu %zu\n", offsetof(gac_hparams, mode), offsetof(gac_hparams, alpha_fixed),
         offsetof(gac_hparams, zero_on_violation), offsetof(gac_result, coef), offsetof(gac_result, step));
  return 0; }
''')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()
    got = list(map(int, out))
    want = [ctypes.sizeof(gb.gac_tensor), ctypes.sizeof(gb.gac_hparams), ctypes.sizeof(gb.gac_result),
            ctypes.sizeof(gb.gac_info), gb.gac_hparams.mode.offset, gb.gac_hparams.alpha_fixed.offset,
            gb.gac_hparams.zero_on_violation.offset, gb.gac_result.coef.offset,
            gb.gac_result.step.offset]
    assert got == want


def test_default_hparams_are_the_papers(lib):
    hp = gb.gac_hparams()
    lib.gac_default_hparams(ctypes.byref(hp))
    assert (hp.c_low, hp.c_high, hp.eps, hp.beta) == (0.05, 0.3, 1e-8, 1.0)
    assert (hp.mode, hp.state_mode, hp.zero_on_violation) == (0, 0, 0)


def _init(lib, tensors, g_dt=0, d_dt=0, **over):
    hp = gb.gac_hparams()
    lib.gac_default_hparams(ctypes.byref(hp))
    for k, v in over.items():
        setattr(hp, k, v)
    arr = (gb.gac_tensor * max(1, len(tensors)))(*[gb.gac_tensor(*t) for t in tensors])
    out = ctypes.c_void_p()
    rc = lib.gac_init(ctypes.byref(out), arr, len(tensors), g_dt, d_dt, ctypes.byref(hp), 0)
    assert not out.value or rc == 0
    return rc, lib.gac_last_error(None).decode()


def test_argument_errors_need_no_device(lib):
    ok = (4096, 8192, 16)
    assert _init(lib, [])[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [(0, 8192, 16)])[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [(4096, 8192, 0)])[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], g_dt=0, d_dt=1)[0] == gb.GAC_ERR_DTYPE
    assert _init(lib, [ok], g_dt=7)[0] == gb.GAC_ERR_DTYPE
    assert _init(lib, [ok], c_low=0.3, c_high=0.3)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], c_low=0.0)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], c_low=-0.1)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], eps=-1.0)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], beta=float("nan"))[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], mode=5)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], state_mode=4)[0] == gb.GAC_ERR_INVALID_ARG
    # exchange mode swaps the roles of the two buffer sets: one element type for both
    rc, msg = _init(lib, [ok], g_dt=1, d_dt=0, state_mode=gb.GAC_STATE_EXCHANGE)
    assert rc == gb.GAC_ERR_DTYPE and "exchange" in msg
    assert _init(lib, [ok], state_mode=gb.GAC_STATE_EXCHANGE)[0] in (gb.GAC_OK, gb.GAC_ERR_CUDA)
    assert _init(lib, [ok], mode=1, alpha_fixed=-1.0)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], reserved=1)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [(4097, 8192, 16)])[0] == gb.GAC_ERR_INVALID_ARG       # not element-aligned
    rc, msg = _init(lib, [(4096, 4100, 16)])                                   # g and d overlap
    assert rc == gb.GAC_ERR_INVALID_ARG and "overlap" in msg
    rc, msg = _init(lib, [(4096, 8192, 16), (16384, 4096 + 32, 16)])          # d of tensor 1 inside g of tensor 0
    assert rc == gb.GAC_ERR_INVALID_ARG and "overlap" in msg
    assert _init(lib, [ok], clip_max_norm=-1.0)[0] == gb.GAC_ERR_INVALID_ARG
    assert _init(lib, [ok], g_dt=1, d_dt=1)[0] in (gb.GAC_OK, gb.GAC_ERR_CUDA)   # bf16/bf16 is a supported pair
    rc, msg = _init(lib, [ok])
    # with valid arguments the only thing that can fail here is the missing device
    import torch
    if not torch.cuda.is_available():
        assert rc == gb.GAC_ERR_CUDA and "device" in msg


def test_static_entry_argument_errors_need_no_device(lib):
    """gac_stats_static checks its arguments before it touches CUDA: a misaligned record pointer (the
    record holds doubles, a 4-byte aligned address would make the device stores fault) is refused on
    the host, with a message."""
    hp = gb.gac_hparams()
    lib.gac_default_hparams(ctypes.byref(hp))
    arr = (gb.gac_tensor * 1)(gb.gac_tensor(4096, 8192, 16))

    def call(result_ptr, step=2, n=1, g_dt=0, d_dt=0):
        rc = lib.gac_stats_static(arr, n, g_dt, d_dt, ctypes.byref(hp), step, 0, 0, None, result_ptr)
        return rc, lib.gac_last_error(None).decode()

    rc, msg = call(0x10004)
    assert rc == gb.GAC_ERR_INVALID_ARG and "8-byte aligned" in msg
    assert call(None)[0] == gb.GAC_ERR_INVALID_ARG
    assert call(0x10000, step=0)[0] == gb.GAC_ERR_INVALID_ARG
    assert call(0x10000, n=0)[0] == gb.GAC_ERR_INVALID_ARG
    assert call(0x10000, g_dt=0, d_dt=1)[0] == gb.GAC_ERR_DTYPE


def test_null_context_is_rejected(lib):
    r = gb.gac_result()
    assert lib.gac_stats(None, 1, 0, None, ctypes.byref(r)) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_project(None, None, None, None) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_stats_partial(None, 1, 0, None, None) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_decide(None, None, None, None) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_set_launch(None, 0, 0) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_next_gradient_set(None, None) == gb.GAC_ERR_INVALID_ARG
    assert lib.gac_free(None) == gb.GAC_OK
    assert lib.gac_last_error(None) is not None


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(gb, "_lib", None)
    monkeypatch.setattr(gb, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        gb.load_library()


def test_product_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2603_01501_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
