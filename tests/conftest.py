import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


SWITCHES = ("attn_mma_sync", "attn_one_tile", "attn_persistent", "attn_section", "attn_variant", "gemm_cta_group", "gemm_group_m",
            "gemm_heavy_first", "gemm_split", "gemm_loader", "row_tma", "row_team", "row_reduce")


@pytest.fixture(autouse=True)
def reset_library_switches():
    """Tests force kernel forms through ja_debug_set; every test starts and ends with nothing forced and the default wait limit."""
    yield
    import paper_2609_03905_b200 as ja
    for name in SWITCHES:
        ja.ja_debug_set(name, -1)
    ja.ja_debug_set("wait_cap_ns", 2_000_000_000)
