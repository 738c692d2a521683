"""Host-only checks of the C-ABI library: it loads, exports every symbol that
include/sama.h declares, and its pure-host helpers work.  No kernel runs."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2310_05674_b200 import build
    build.build()
    from paper_2310_05674_b200 import binding as b
    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sama.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sama_[a-z_]+)\s*\(", text)))


def test_header_declares_the_four_path_entry_points():
    names = declared_functions()
    for n in ["sama_adapt", "sama_perturb", "sama_fd_metagrad", "sama_step"]:
        assert n in names


def test_library_exports_every_declared_symbol(binding):
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_param_count_and_status_strings(binding):
    assert binding.sama_mlp_param_count(binding.MLP((784, 256, 10))) == 203530
    assert binding.sama_mlp_param_count(binding.MLP((4096, 4096, 4096, 1000))) == 37659624
    assert binding.sama_mlp_param_count(binding.MLP((3, 0, 2))) == -1
    seen = {binding.sama_status_string(c) for c in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert binding.sama_status_string(-99) == "unknown status"


def test_create_fails_cleanly_without_a_device(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(binding.SamaError) as e:
        binding.sama_create(0, 1024, 8, None)
    assert e.value.status == binding.SAMA_ERR_CUDA


def test_null_context_is_rejected_on_the_host(binding):
    a = binding.Adam()
    with pytest.raises(binding.SamaError) as e:
        binding.sama_adapt(None, 4, 16, 32, None, 48, a, 64, None, stream=0)
    assert e.value.status == binding.SAMA_ERR_NULL
    with pytest.raises(binding.SamaError):
        binding.sama_perturb(None, 4, 16, 32, None, 1.0, 48, 64, None, stream=0)


def test_product_package_does_not_import_the_checker():
    pkg = os.path.join(ROOT, "paper_2310_05674_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
