"""Host-side checks of the C-ABI library that need no GPU: it builds, loads, exports every
symbol the header declares, and its host-only entry points behave."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "swiftprune.h")


@pytest.fixture(scope="module")
def lib_path():
    from paper_2501_16376_b200 import build
    return build.build()


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_calls_of_the_pruning_pass():
    names = _declared_symbols()
    for required in ("sp_calib_accumulate", "sp_score", "sp_select_unstructured", "sp_select_nm",
                     "sp_apply_mask"):
        assert required in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_debug_build_exports_the_same_symbols():
    from paper_2501_16376_b200 import build
    lib = ctypes.CDLL(build.build(debug=True))
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2501_16376_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_symbols()


def test_table3_lookup_in_the_library(lib_path):
    from paper_2501_16376_b200 import binding
    golden = {}
    with open(os.path.join(ROOT, "tests", "golden", "table2_table3.txt")) as f:
        for line in f:
            if line.startswith("la_"):
                k, v = line.split()
                golden[int(k[3:])] = float(v)
    for pct, la in golden.items():
        assert binding.sp_la_for_sparsity(pct / 100.0) == pytest.approx(la, abs=1e-7)
    assert binding.sp_la_for_sparsity(0.55) == pytest.approx(0.35, abs=1e-6)
    assert binding.sp_la_for_sparsity(0.95) == pytest.approx(-1.8, abs=1e-6)
    assert binding.sp_la_for_sparsity(0.40) == pytest.approx(0.8, abs=1e-6)
    with pytest.raises(binding.SpError):
        binding.sp_la_for_sparsity(0.0)


def test_status_strings_and_null_arguments(lib_path):
    from paper_2501_16376_b200 import binding
    lib = binding.lib
    assert lib.sp_status_string(0) == b"ok"
    assert b"shape" in lib.sp_status_string(binding.SP_ERR_SHAPE)
    assert lib.sp_create(None, 16, 0) == binding.SP_ERR_INVALID_ARG
    assert lib.sp_destroy(None) == binding.SP_OK
    assert lib.sp_calib_reset(None, None) == binding.SP_ERR_INVALID_ARG
    assert lib.sp_apply_mask(None, 0, 1, 1, 1, None, None, 1, None) == binding.SP_ERR_INVALID_ARG
    assert lib.sp_apply_mask(None, 0, 0, 8, 8, None, None, 8, None) == binding.SP_OK
    assert lib.sp_select_nm(None, None, 0, 1, 1, 2, 4, None, None, 1, None) == \
        binding.SP_ERR_INVALID_ARG


def test_create_without_a_device_fails_cleanly(lib_path):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2501_16376_b200 import binding
    with pytest.raises(binding.SpError) as e:
        binding.Context(64, device=0)
    assert e.value.status in (binding.SP_ERR_CUDA, binding.SP_ERR_INVALID_ARG)


def test_product_path_fails_loudly_without_the_library_or_a_device(tmp_path):
    # no CPU fallback anywhere: a missing library is an ImportError, a missing GPU a refusal
    import subprocess
    import sys
    env = dict(os.environ, SWIFTPRUNE_LIBRARY=str(tmp_path / "not_built.so"))
    proc = subprocess.run([sys.executable, "-c", "import paper_2501_16376_b200.binding"],
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert proc.returncode != 0 and "no CPU fallback" in proc.stderr
    import torch
    if not torch.cuda.is_available():
        proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "single-512",
                               "--no-cpu-baseline"], cwd=ROOT, capture_output=True, text=True, timeout=300)
        assert proc.returncode != 0 and "CUDA device" in proc.stderr
        # and nothing in the package reaches for the oracle
        src = ""
        pkg = os.path.join(ROOT, "paper_2501_16376_b200")
        for name in os.listdir(pkg):
            if name.endswith(".py"):
                with open(os.path.join(pkg, name)) as f:
                    src += f.read()
        assert "import oracle" not in src and "from oracle" not in src
