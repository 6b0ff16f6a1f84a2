"""The bounds-check build (-DQALORA_DEBUG) run over the small parity shapes.

The library compiled with the checks tests every computed index, offset, tensor-memory column
and copy coordinate against its limit and surrounds the workspace regions with guard words.
Here the small-shape parity, grouped-forward and fine-tuning-step tests run once more in a
child process that loads that build; `conftest.py` reads the record words after every test of
that process and fails the test if a check failed or a guard word was overwritten.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = ["tests/test_parity_gpu.py", "tests/test_forward_group_gpu.py", "tests/test_finetune_step_gpu.py",
         "tests/test_formats_gpu.py", "tests/test_optimizer_gpu.py", "tests/test_debug_build_gpu.py"]


def test_release_library_reports_no_checks():
    from paper_2309_14717_b200 import binding as Q
    if Q.DEBUG_LIBRARY:
        pytest.skip("this process runs the bounds-check build")
    assert Q.qalora_debug_checks() is False
    assert Q.qalora_debug_report() == [0] * 8


@pytest.mark.gpu
def test_small_parity_shapes_pass_the_bounds_check_build():
    if os.environ.get("QALORA_LIBRARY") == "debug":
        pytest.skip("already inside the bounds-check run")
    from paper_2309_14717_b200 import build as B
    B.build(debug=True)
    env = dict(os.environ, QALORA_LIBRARY="debug")
    env.pop("QALORA_PARITY_MARGINS", None)
    cases = [c for c in CASES if os.path.exists(os.path.join(ROOT, c))]
    p = subprocess.run([sys.executable, "-m", "pytest", "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"] + cases,
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = "\n".join((p.stdout + p.stderr).splitlines()[-40:])
    assert p.returncode == 0, tail
    assert " passed" in p.stdout and "bounds-check build" in p.stdout, tail


@pytest.mark.gpu
def test_the_record_catches_a_refused_index_and_an_overwritten_guard_word():
    """Runs only inside the bounds-check process.  The library's self-test asks for index 5 of an
    array of 4 (refused, nothing is accessed) and overwrites one word of a guard that lies inside
    the buffer it was given: both must show in the record, which this test then leaves clean."""
    import ctypes

    import torch

    from paper_2309_14717_b200 import binding as Q
    if not Q.DEBUG_LIBRARY:
        pytest.skip("needs QALORA_LIBRARY=debug")
    lib = Q.load()
    lib.qalora_debug_selftest.restype = ctypes.c_int
    lib.qalora_debug_selftest.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    assert Q.qalora_debug_report() == [0] * 8
    buf = torch.zeros(512, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.qalora_debug_selftest(ctypes.c_void_p(buf.data_ptr()), ctypes.c_void_p(stream)) == 0
    words = Q.qalora_debug_report()
    assert words[0] == 6 and words[2] == 5 and words[3] == 0 and words[4] == 4 and words[5] == 0
    assert words[1] // 100000 == 1 and words[6] == 1 and words[7] == 0 * 65536 + 3 + 1
    assert Q.qalora_debug_report() == [0] * 8
