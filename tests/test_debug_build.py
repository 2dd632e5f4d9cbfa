"""The checked builds: the CUDA library with -DSPADE_DEBUG (index checks that record instead of trapping, guard
words behind the workspace regions) and the CPU-side code under AddressSanitizer / UBSan."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _asan():
    out = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    return out if os.path.isabs(out) and os.path.exists(out) else None


def test_debug_library_builds_and_exports_the_same_symbols():
    import ctypes as C
    import re
    from paper_2608_03335_b200.build import build_library
    L = C.CDLL(build_library(debug=True))
    hdr = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "spade.h")).read(), flags=re.S)
    for n in set(re.findall(r"\b(spade_[a-z_]+)\s*\(", hdr)):
        assert hasattr(L, n), n


def test_oracle_pins_pass_under_address_and_ub_sanitizers():
    """The oracle rebuilt with -fsanitize=address,undefined runs a slice of its pins (geometry, SICS, selection,
    attention on ragged grids): any out-of-bounds index or undefined operation aborts the child."""
    asan = _asan()
    if asan is None:
        pytest.skip("libasan is not installed")
    env = dict(os.environ, SPADE_ORACLE_SANITIZE="1", LD_PRELOAD=asan, ASAN_OPTIONS="detect_leaks=0:halt_on_error=1",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "tests/test_oracle_pins.py",
                        "-k", "geometry or sics or topk or topp or attention or static or minmax"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert "passed" in r.stdout


def test_host_argument_checks_pass_under_address_sanitizer():
    """The library's host side (argument validation, geometry and layout planning) rebuilt with AddressSanitizer
    runs the ABI argument tests; a plan for the largest shapes is laid out and torn down where a device exists."""
    asan = _asan()
    if asan is None:
        pytest.skip("libasan is not installed")
    build = (
        "import os, sys; sys.path.insert(0, '.');"
        "from paper_2608_03335_b200 import build;"
        "build.LIB = build.LIB.replace('.so', '_asan.so');"
        "os.environ['SPADE_NVCC_EXTRA'] = '-Xcompiler -fsanitize=address -Xcompiler -fno-omit-frame-pointer';"
        "print(build.build_library())"
    )
    r = subprocess.run([sys.executable, "-c", build], cwd=ROOT, capture_output=True, text=True, timeout=1800)   # the compiler runs unsanitized
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    lib = r.stdout.strip().splitlines()[-1]
    code = (
        "import sys; sys.path.insert(0, '.');"
        f"import paper_2608_03335_b200.binding as b; b.LIB = {lib!r};"
        "import pytest; sys.exit(pytest.main(['-x', '-q', '-p', 'no:cacheprovider', 'tests/test_abi.py', '-k', 'rejects or null_plan']))"
    )
    env = dict(os.environ, LD_PRELOAD=asan, ASAN_OPTIONS="detect_leaks=0:halt_on_error=1:protect_shadow_gap=0")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1800)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert "passed" in r.stdout


@pytest.mark.gpu
def test_tiny_and_ragged_layers_run_clean_under_the_debug_library():
    """Tiny (both budgets), a ragged grid with odd block counts and a text tail, all four stages checked against
    the oracle as usual, through the library built with -DSPADE_DEBUG: no index check may fire and every guard
    word must be intact (spade_status would raise SPADE_ERR_DEBUG_CHECK)."""
    code = (
        "import sys; sys.path.insert(0, '.');"
        "from paper_2608_03335_b200 import binding;"
        "from paper_2608_03335_b200.workloads import WORKLOADS, small_variant;"
        "from tests.parity_util import run_layer_parity;"
        "assert binding.lib()._name.endswith('_debug.so');"
        "run_layer_parity(WORKLOADS['tiny']); run_layer_parity(WORKLOADS['tiny_topp']);"
        "run_layer_parity(small_variant(WORKLOADS['wan1p3b'], heads=3, grid=(5, 14, 20)));"
        "run_layer_parity(small_variant(WORKLOADS['hunyuan'], heads=4, grid=(16, 9, 12), n_text=100));"
        "run_layer_parity(small_variant(WORKLOADS['wan14b'], heads=2, grid=(9, 10, 12)), forced=[3, 0], static=dict(window=1, sink_tokens=70));"
        "print('debug build clean')"
    )
    env = dict(os.environ, SPADE_DEBUG="1")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "debug build clean" in r.stdout, r.stdout[-3000:] + r.stderr[-3000:]
