"""The C-ABI library builds, loads, and exports every symbol the header declares (no GPU needed)."""
import os
import re

from paper_2410_05265_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_loads_and_exports_header_symbols():
    build.build()
    lib = binding.load_library()
    header = open(os.path.join(ROOT, "include", "pq.h")).read()
    code = re.sub(r"/\*.*?\*/", "", header, flags=re.S)  # declarations only, comments stripped
    declared = set(re.findall(r"\b(pq_[a-z0-9_]+)\s*\(", code))
    assert declared, "no declarations found in include/pq.h"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in pq.h but not exported"
    assert set(binding.EXPORTS) == declared
    assert lib.pq_status_string(0) == b"PQ_OK" and lib.pq_status_string(6) == b"PQ_ERR_TIMEOUT"
    assert lib.pq_w4a4_gemm_workspace_bytes(1, 1, 32) == 0


def test_product_path_has_no_cpu_fallback():
    import pytest
    import torch

    if torch.cuda.is_available():
        pytest.skip("checks the failure mode on a box without a GPU")
    with pytest.raises(RuntimeError):
        binding.Context()
