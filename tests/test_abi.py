"""Host-only checks of the C-ABI library: it loads, exports every function the
header declares, and rejects bad arguments before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200 import build as _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    _build.build()


def _declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(qalora_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = Q.load()
    declared = _declared_functions()
    assert set(Q.EXPORTS) <= set(declared) and len(declared) >= 8
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings():
    assert Q.qalora_version() % 100 == 1
    assert Q.status_string(0) == "ok"
    for s in range(-6, 0):
        assert Q.status_string(s) not in ("ok", "unknown status")
    assert Q.status_string(-99) == "unknown status"


def test_packed_and_workspace_sizes():
    d = Q.desc(4096, 11008, 32, 4, 64, 1.0)
    cb, qb = Q.qalora_packed_bytes(d)
    assert cb == 4096 * 11008 // 2 and qb == (4096 // 32) * 11008 * 8
    assert Q.qalora_packed_bytes(Q.desc(4096, 4096, 32, 3, 0, 1.0))[0] == 4096 * 4096 * 3 // 8
    assert Q.qalora_packed_bytes(Q.desc(4096, 4096, 128, 2, 0, 1.0)) == (4096 * 4096 // 4, 32 * 4096 * 8)
    fwd = Q.qalora_workspace_bytes(d, 8192, Q.OP_FORWARD)
    bwd = Q.qalora_workspace_bytes(d, 8192, Q.OP_BACKWARD)
    assert 0 < fwd <= bwd < (1 << 30)
    assert Q.qalora_workspace_bytes(d, 0, Q.OP_FORWARD) >= 0


@pytest.mark.parametrize("args,status", [
    ((0, 512, 32, 4, 16, 1.0), -1), ((512, 512, 32, 5, 16, 1.0), -1), ((512, 512, 32, 4, -8, 1.0), -1),
    ((512, 512, 32, 4, 16, float("nan")), -1),
    ((512, 512, 48, 4, 16, 1.0), -3), ((500, 512, 32, 4, 16, 1.0), -3), ((512, 516, 32, 4, 16, 1.0), -3),
    ((512, 512, 32, 4, 12, 1.0), -3), ((512, 512, 32, 4, 512, 1.0), -3),
])
def test_bad_descriptors_are_rejected(args, status):
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_packed_bytes(Q.desc(*args))
    assert e.value.status == status


def test_null_and_misaligned_pointers_are_rejected_without_a_launch():
    lib = Q.load()
    d = Q.desc(512, 512, 32, 4, 16, 1.0)
    p = ctypes.c_void_p
    buf = ctypes.create_string_buffer(64)          # host memory: must never be dereferenced
    a = ctypes.addressof(buf)
    a16 = (a + 15) // 16 * 16
    r = ctypes.byref
    assert lib.qalora_quantize(r(d), None, p(a16), p(a16), None, None) == -2
    assert lib.qalora_quantize(r(d), p(a16 + 4), p(a16), p(a16), None, None) == -4
    assert lib.qalora_merge(r(d), p(a16), None, p(a16), p(a16), None) == -2
    assert lib.qalora_forward(r(d), -1, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -1
    assert lib.qalora_forward(r(d), (1 << 22) + 1, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -1
    size = ctypes.c_size_t(0)
    assert lib.qalora_workspace_bytes(r(d), 1 << 22, Q.OP_TRAIN, r(size)) == 0 and size.value > 0
    assert lib.qalora_workspace_bytes(r(d), (1 << 22) + 1, Q.OP_TRAIN, r(size)) == -1
    assert lib.qalora_forward(r(d), 8, None, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -2
    assert lib.qalora_forward(r(d), 8, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 0, None) == -5
    assert lib.qalora_forward(r(d), 8, p(a16 + 2), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -4
    assert lib.qalora_backward(r(d), 8, p(a16), None, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -2
    d0 = Q.desc(512, 512, 32, 4, 0, 1.0)
    assert lib.qalora_backward(r(d0), 8, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), 1 << 30, None) == -1
    assert lib.qalora_forward(r(d), 0, None, None, None, None, None, None, None, 0, None) == 0


def test_static_scratch_forward_checks_its_arguments_before_anything_else():
    """qalora_forward_static must turn a bad argument down before it looks up its scratch
    array or enqueues the clearing of the status word: on a machine without a GPU a call
    that reached the CUDA runtime first would come back as a CUDA error (-6) instead."""
    lib = Q.load()
    d = Q.desc(512, 512, 32, 4, 16, 1.0)
    p = ctypes.c_void_p
    buf = ctypes.create_string_buffer(64)          # host memory: must never be dereferenced
    a16 = (ctypes.addressof(buf) + 15) // 16 * 16
    r = ctypes.byref
    assert lib.qalora_forward_static(r(d), 8, None, p(a16), p(a16), p(a16), p(a16), p(a16), None) == -2
    assert lib.qalora_forward_static(r(d), 8, p(a16), p(a16), p(a16), None, p(a16), p(a16), None) == -2
    assert lib.qalora_forward_static(r(d), 8, p(a16 + 2), p(a16), p(a16), p(a16), p(a16), p(a16), None) == -4
    assert lib.qalora_forward_static(r(d), -3, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), None) == -1
    assert lib.qalora_forward_static(r(d), 1 << 20, p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), None) == -7
    assert lib.qalora_forward_static(r(d), 0, None, None, None, None, None, None, None) == 0


def test_forward_group_argument_checks_need_no_gpu():
    lib = Q.load()
    buf = ctypes.create_string_buffer(64)          # host memory: must never be dereferenced
    a16 = (ctypes.addressof(buf) + 15) // 16 * 16
    good = Q.GroupLayer(Q.desc(512, 512, 32, 4, 0, 1.0), a16, a16, a16, None, None, a16)
    bad_desc = Q.GroupLayer(Q.desc(512, 512, 48, 4, 0, 1.0), a16, a16, a16, None, None, a16)
    no_x = Q.GroupLayer(Q.desc(512, 512, 32, 4, 0, 1.0), None, a16, a16, None, None, a16)
    need_ab = Q.GroupLayer(Q.desc(512, 512, 32, 4, 16, 1.0), a16, a16, a16, None, None, a16)
    arr = lambda *ls: (Q.GroupLayer * len(ls))(*ls)
    size = ctypes.c_size_t()
    assert lib.qalora_forward_group_workspace_bytes(arr(good, good), 2, 4, ctypes.byref(size)) == 0 and size.value >= 256
    assert lib.qalora_forward_group_workspace_bytes(arr(good, bad_desc), 2, 4, ctypes.byref(size)) == -3
    assert lib.qalora_forward_group_workspace_bytes(None, 2, 4, ctypes.byref(size)) == -2
    ws = ctypes.c_void_p(a16)
    assert lib.qalora_forward_group(None, 1, 4, ws, 1 << 20, None) == -2
    assert lib.qalora_forward_group(arr(good), -1, 4, ws, 1 << 20, None) == -1
    assert lib.qalora_forward_group(arr(good, bad_desc), 2, 4, ws, 1 << 20, None) == -3
    assert lib.qalora_forward_group(arr(good, no_x), 2, 4, ws, 1 << 20, None) == -2       # the second layer spoils the call
    assert lib.qalora_forward_group(arr(good, need_ab), 2, 4, ws, 1 << 20, None) == -2
    assert lib.qalora_forward_group(arr(good), 1, 4, ws, 8, None) == -5
    assert lib.qalora_forward_group(arr(good), 1, 4, ctypes.c_void_p(a16 + 4), 1 << 20, None) == -4
    assert lib.qalora_forward_group(arr(good), 0, 4, ws, 1 << 20, None) == 0
    assert lib.qalora_forward_group(arr(good), 1, 0, ws, 1 << 20, None) == 0


def test_adamw_argument_checks_need_no_gpu():
    lib = Q.load()
    p = ctypes.c_void_p
    buf = ctypes.create_string_buffer(64)          # host memory: must never be dereferenced
    a16 = (ctypes.addressof(buf) + 15) // 16 * 16
    r = ctypes.byref
    good = Q.adamw_hyper(1, 2e-5)
    args = lambda h, n=8, g=a16, ws=1 << 20: (r(h) if h is not None else None, n, p(g), p(a16), p(a16), p(a16), p(a16),
                                              None, p(a16), ws, None)
    assert lib.qalora_adamw_step(*args(None)) == -2
    assert lib.qalora_adamw_step(*args(Q.adamw_hyper(0, 2e-5))) == -1
    assert lib.qalora_adamw_step(*args(Q.adamw_hyper(1, 2e-5, beta2=1.0))) == -1
    assert lib.qalora_adamw_step(*args(good, n=-1)) == -1
    assert lib.qalora_adamw_step(*args(good, g=a16 + 4)) == -4
    assert lib.qalora_adamw_step(*args(good, ws=8)) == -5
    assert lib.qalora_adamw_step(*args(good, n=0)) == 0
    assert Q.qalora_adamw_workspace_bytes() >= 4096
