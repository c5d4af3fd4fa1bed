"""The shared library loads without a GPU and exports every symbol include/aero.h declares."""
import ctypes
import os
import re

from paper_2602_14338_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "aero.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aero_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    from paper_2602_14338_b200 import build

    build.build()
    lib = ctypes.CDLL(B.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_host_side_calls_without_gpu():
    lib = B.load_library()
    assert lib.aero_version() >= 100
    cfg = B.cfg_default()
    assert cfg.k_ratio == 1 and cfg.n_keep_uniform == 4 and abs(cfg.clip_hi - 0.2) < 1e-7
    assert lib.aero_error_string(-3) == b"workspace too small"
    assert lib.aero_group_workspace_bytes(64, 512) > 0
    # the dz block dominates the backward workspace: rows * padded V * 2 bytes
    assert lib.aero_bwd_workspace_bytes(1000, 128, 1000, 10, 256) >= 256 * 1024 * 2
    assert lib.aero_step_workspace_bytes(4, 16, 640, 64, 512, 128, B.AERO_BF16) > 640 * 64 * 2
