"""The C-ABI boundary without a GPU: the shared library loads, exports every function that
include/*.h declare (and the binding lists the same names), the ctypes structures have the
layout the C compiler gives the header's structs, and the calls that need no device answer."""
import ctypes as C
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
HEADER = os.path.join(ROOT, "include", "scd.h")
HEADERS = [HEADER, os.path.join(ROOT, "include", "scd_hooks.h")]

from paper_2510_24211_b200 import binding as scd  # noqa: E402


def _declared():
    text = "".join(open(h).read() for h in HEADERS)
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)          # comments mention function names too
    return re.findall(r"^\s*(?:int|int64_t|const char \*)\s*\*?\s*(scd_\w+)\s*\(", text, flags=re.M)


def test_library_exports_every_declared_function():
    names = _declared()
    assert len(names) >= 20 and len(set(names)) == len(names)
    lib = C.CDLL(scd.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(names) == set(scd.EXPORTS)


def test_ctypes_structures_match_the_header(tmp_path):
    fields = {
        "scd_model_config_t": (scd.ModelConfig, [f[0] for f in scd.ModelConfig._fields_]),
        "scd_decode_config_t": (scd.DecodeConfig, [f[0] for f in scd.DecodeConfig._fields_]),
        "scd_stats_t": (scd.Stats, [f[0] for f in scd.Stats._fields_]),
        "scd_weights_t": (scd.Weights, [f[0] for f in scd.Weights._fields_]),
    }
    lines = ['#include <stdio.h>', '#include <stddef.h>', f'#include "{HEADER}"', "int main(void) {"]
    for ctype, (_, names) in fields.items():
        lines.append(f'  printf("{ctype} %zu\\n", sizeof({ctype}));')
        for n in names:
            lines.append(f'  printf("{ctype}.{n} %zu\\n", offsetof({ctype}, {n}));')
    lines += ["  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-std=c99", "-o", str(exe), str(src)])
    out = dict(line.split() for line in subprocess.check_output([str(exe)]).decode().splitlines())
    for ctype, (cls, names) in fields.items():
        assert int(out[ctype]) == C.sizeof(cls), ctype
        for n in names:
            assert int(out[f"{ctype}.{n}"]) == getattr(cls, n).offset, f"{ctype}.{n}"


def test_calls_that_need_no_device():
    lib = scd.lib()
    lib.scd_strerror.restype = C.c_char_p
    texts = {code: lib.scd_strerror(code).decode() for code in range(-8, 1)}
    assert texts[0] and len(set(texts.values())) >= 8             # one text per status code
    assert scd.scd_kernel_launches() >= 0
    assert scd.scd_selftest_device_once() == 0                    # per-device set-up bookkeeping (host only)
    # argument checks run on the host, before any CUDA call
    bad = scd.decode_config(batch=0, window_L=4, allowed_hi=10)
    assert lib.scd_verify_workspace_bytes(C.byref(bad), 10) < 0
    good = scd.decode_config(batch=2, window_L=4, allowed_hi=10)
    assert lib.scd_verify_workspace_bytes(C.byref(good), 10) > 0
    assert lib.scd_verify_noalloc_max_bytes() == 16 << 20
    assert lib.scd_gemm_workspace_bytes(64, 4096, 4096) > 0
    assert lib.scd_gemm_workspace_bytes(64, 4096, 100) < 0       # K not a multiple of 64
    assert lib.scd_gemm_workspace_bytes(300, 4096, 4096) < 0     # more than 256 window rows
    with pytest.raises(scd.ScdError):
        scd._check(lib.scd_prefill(None, None, 1, 1, None))
    assert lib.scd_session_attention_min_ctx(None, 0) < 0           # null session
