"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, agrees with the binding on the parameter block, and rejects bad
arguments before touching the device."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "rattn.h")


@pytest.fixture(scope="module")
def B():
    from paper_2506_15545_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rattn_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = _declared_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(B.lib(), n), n


def test_debug_library_exports_its_one_extra_entry_point(B):
    """include/rattn_debug.h: declared there, exported by librattn_dbg.so only."""
    from paper_2506_15545_b200 import build
    dbg = ctypes.CDLL(build.build(debug=True))
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "rattn_debug.h")).read(), flags=re.S)
    names = sorted(set(re.findall(r"\b(rattn_[a-z_]+)\s*\(", text)))
    assert names == ["rattn_debug_withhold_arrival"]
    assert hasattr(dbg, names[0]) and not hasattr(B.lib(), names[0])
    for n in B.EXPORTS:
        assert hasattr(dbg, n), n


def test_header_is_plain_c_and_struct_matches_binding(B, tmp_path):
    src = tmp_path / "sz.c"
    src.write_text('#include "rattn.h"\n#include <stdio.h>\n#include <stddef.h>\n'
                   'int main(void){printf("%zu %zu %zu %zu\\n", sizeof(rattn_params),'
                   'offsetof(rattn_params, workspace_bytes), offsetof(rattn_params, dout),'
                   'offsetof(rattn_params, flags));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe)])
    size, off_ws, off_dout, off_flags = map(int, subprocess.check_output([str(exe)]).split())
    P = B.RattnParams
    assert size == ctypes.sizeof(P)
    assert off_ws == P.workspace_bytes.offset
    assert off_dout == P.dout.offset
    assert off_flags == P.flags.offset


def test_strerror_and_workspace_bytes(B):
    L = B.lib()
    assert L.rattn_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert L.rattn_strerror(code) not in (b"ok", b"unknown status")
    assert L.rattn_strerror(-99) == b"unknown status"
    n = B.rattn_workspace_bytes(4, 16, 16, 4096, 128, 512)
    assert n > 0 and n % 256 == 0
    assert B.rattn_workspace_bytes(4, 16, 16, 4096, 128, 512) == n          # pure function
    assert B.rattn_workspace_bytes(8, 16, 16, 4096, 128, 512) > n
    assert B.rattn_workspace_bytes(4, 16, 16, 4096, 96, 512) == 0           # unsupported d
    assert B.rattn_workspace_bytes(4, 16, 5, 4096, 128, 512) == 0           # H_q % H_kv != 0
    assert B.rattn_workspace_bytes(0, 16, 16, 4096, 128, 512) == 0


def test_workspace_size_follows_mode_and_flags(B):
    """An inference forward keeps only what it uses: the status block on the portable kernels,
    status + one progress word per K/V head + bf16 chunk states on the tensor-core kernels; training
    adds the residuals."""
    c5 = (32, 32, 8, 32768, 128, 512)
    infer = B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, B.MODE_RATTN, 0)
    states = 32 * 8 * 256 * 128 * 128 * 2
    assert infer == 256 + 1024 + states                                  # 2.1 GB, not 78 GB
    assert B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, B.MODE_SWA_ONLY, 0) == 256
    assert B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, B.MODE_RATTN, B.FLAG_FORCE_GENERIC) == 256
    train = B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, B.MODE_RATTN, B.FLAG_SAVE_RESIDUALS)
    train_generic = B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, B.MODE_RATTN,
                                               B.FLAG_SAVE_RESIDUALS | B.FLAG_FORCE_GENERIC)
    assert infer < train < train_generic                                 # bf16 against fp32 residuals
    assert B.rattn_workspace_bytes(*c5) == max(train, train_generic)     # the bound covers every case
    assert B.rattn_workspace_bytes_ex(*c5, B.RATTN_BF16, 7, 0) == 0      # unknown mode
    few = (1, 4, 2, 1024, 128, 128)
    assert B.rattn_workspace_bytes_ex(*few, B.RATTN_BF16, B.MODE_RATTN, 0) == 256 + 256 + 2 * 8 * 128 * 128 * 2


def _p(bind, **kw):
    p = bind.RattnParams()
    fake = 0x10000                       # non-null, 16-byte aligned; never dereferenced
    p.q = p.k = p.v = p.out = fake
    p.B, p.H_q, p.H_kv, p.T, p.d, p.w = 1, 4, 2, 64, 64, 8
    p.dtype, p.mode, p.scale, p.eps = bind.RATTN_F32, bind.MODE_RATTN, 1.0, 1e-6
    for k, v in kw.items():
        setattr(p, k, v)
    return p


@pytest.mark.parametrize("kw,code", [
    (dict(B=0), -1), (dict(T=0), -1), (dict(w=0), -1), (dict(H_kv=3), -1), (dict(eps=0.0), -1),
    (dict(d=96), -4), (dict(dtype=7), -4), (dict(mode=5), -4),
    (dict(q=0), -2), (dict(out=0), -2),
    (dict(k=0x10008), -3), (dict(gamma_swa=0x10004), -3),
    (dict(flags=2), -5),                                   # residuals wanted, no workspace
    (dict(workspace=0x10100, workspace_bytes=16), -5),     # too small
    (dict(workspace=0x10010, workspace_bytes=1 << 40), -3),  # workspace not 256-byte aligned
    (dict(k_ring_out=0x10000), -2),                        # only one of the two rings
    # shapes of the tensor-core path: it needs a workspace for its chunk states and a positive scale
    (dict(d=128, w=128, dtype=0), -5),
    (dict(d=128, w=128, dtype=0, scale=-1.0, workspace=0x10100, workspace_bytes=1 << 40), -4),
    (dict(d=128, w=128, dtype=0, scale=0.0, workspace=0x10100, workspace_bytes=1 << 40), -4),
])
def test_forward_rejects_bad_arguments_without_launching(B, kw, code):
    before = B.rattn_launch_count()
    assert B.lib().rattn_forward_ex(ctypes.byref(_p(B, **kw)), None) == code
    assert B.rattn_launch_count() == before


def test_null_params_and_backward_and_decode_checks(B):
    L = B.lib()
    assert L.rattn_forward_ex(None, None) == -2
    assert L.rattn_backward_ex(ctypes.byref(_p(B)), None) == -2           # no dout/dq/dk/dv
    p = _p(B, dout=0x10000, dq=0x10000, dk=0x10000, dv=0x10000)
    assert L.rattn_backward_ex(ctypes.byref(p), None) == -5               # no workspace
    assert L.rattn_decode_step_ex(ctypes.byref(_p(B)), None, None, None, 0, None) == -2
    assert L.rattn_decode_step_ex(ctypes.byref(_p(B)), 0x10000, 0x10000, 0x10000, -1, None) == -1
    assert L.rattn_decode_step_ex(ctypes.byref(_p(B)), 0x10000, 0x10008, 0x10000, 0, None) == -3
    assert L.rattn_read_status(None, None) == -2


def test_path_selection_is_a_pure_host_decision(B):
    assert not B.rattn_uses_tensor_path(64, 128)                         # d = 64: portable path
    assert not B.rattn_uses_tensor_path(128, 100)                        # w not a tile multiple
    assert not B.rattn_uses_tensor_path(128, 512, dtype=B.RATTN_F32)
    assert not B.rattn_uses_tensor_path(128, 512, flags=B.FLAG_FORCE_GENERIC)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2506_15545_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2506_15545_b200" not in open(os.path.join(ROOT, "oracle", f)).read()


def test_qk_prologue_struct_and_argument_checks(B, tmp_path):
    """rattn_qk_params has the binding's size and field offsets, and both prologue entry points
    refuse bad arguments before any launch (there is no GPU here, so a launch would fail)."""
    src = tmp_path / "qk.c"
    src.write_text('#include "rattn.h"\n#include <stdio.h>\n#include <stddef.h>\n'
                   'int main(void){printf("%zu %zu %zu %zu\\n", sizeof(rattn_qk_params),'
                   'offsetof(rattn_qk_params, B), offsetof(rattn_qk_params, eps),'
                   'offsetof(rattn_qk_params, pos));return 0;}\n')
    exe = tmp_path / "qk"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe)])
    size, off_b, off_eps, off_pos = map(int, subprocess.check_output([str(exe)]).split())
    P = B.RattnQkParams
    assert (size, off_b, off_eps, off_pos) == (ctypes.sizeof(P), P.B.offset, P.eps.offset, P.pos.offset)

    L = B.lib()

    def params(**kw):
        p = P()
        p.q = p.k = p.q_out = p.k_out = 0x1000
        p.B, p.H_q, p.H_kv, p.T, p.d, p.dtype = 2, 4, 2, 64, 128, B.RATTN_BF16
        p.eps, p.theta = 1e-6, 5.0e5
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    cases = [(dict(B=0), -1), (dict(T=0), -1), (dict(H_kv=-1), -1), (dict(pos0=-5), -1),
             (dict(eps=float("nan")), -1), (dict(eps=-1.0), -1), (dict(theta=float("inf")), -1),
             (dict(d=96), -4), (dict(dtype=7), -4), (dict(q=None), -2), (dict(k=None), -2),
             (dict(q_out=None), -2), (dict(k_out=None), -2), (dict(q=0x1008), -3), (dict(k_out=0x1004), -3),
             (dict(q_gain=0x2004), -3), (dict(pos=0x3002), -3), (dict(B=1 << 20, T=1 << 20), -1)]
    for kw, code in cases:
        assert L.rattn_qk_prologue(ctypes.byref(params(**kw)), None) == code, kw
    assert L.rattn_qk_prologue(None, None) == -2
    p = params()
    assert L.rattn_qk_prologue_backward(ctypes.byref(p), None, 0x1000, 0x1000, 0x1000, None, None, None, 0, None) == -2
    assert L.rattn_qk_prologue_backward(ctypes.byref(p), 0x1000, 0x1000, 0x1000, 0x1000, 0x4000, None, None, 0,
                                        None) == -5
    assert L.rattn_qk_prologue_backward(ctypes.byref(p), 0x1000, 0x1000, 0x1000, 0x1000, 0x4000, None, 0x5000, 16,
                                        None) == -5
    assert L.rattn_qk_prologue_backward(ctypes.byref(params(H_kv=0, k=None, k_out=None)), 0x1000, None, 0x1000, None,
                                        None, 0x4000, None, 0, None) == -1
    n = B.rattn_qk_prologue_workspace_bytes(4, 16, 16, 4096, 128)
    assert n % 256 == 0 and 0 < n <= 2 * 2048 * 128 * 4
    assert B.rattn_qk_prologue_workspace_bytes(4, 16, 16, 4096, 96) == 0
