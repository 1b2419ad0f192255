"""The C-ABI library builds, loads without a GPU, and exports every symbol the header
declares (no compute calls here)."""
import ctypes
import os
import re

import paper_2512_04939_b200 as pkg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(litevggt_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    if not os.path.exists(pkg.library_path()):
        from paper_2512_04939_b200.build import build
        build()
    lib = ctypes.CDLL(pkg.library_path())
    declared = _declared_symbols()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"


def test_status_strings_and_default_config_without_gpu():
    lib = pkg.load_library()
    assert lib.litevggt_status_string(0) == b"ok"
    assert b"timed out" in lib.litevggt_status_string(9)
    from paper_2512_04939_b200.binding import Config
    cfg = Config()
    assert lib.litevggt_default_config(4, 16, 16, 0.5, ctypes.byref(cfg)) == 0
    assert (cfg.patch_px, cfg.n_special, cfg.dim, cfg.heads, cfg.recompute_interval) == (14, 5, 1024, 16, 6)
    assert lib.litevggt_default_config(0, 16, 16, 0.5, ctypes.byref(cfg)) == 2      # bad config
    assert lib.litevggt_default_config(4, 16, 16, 1.5, ctypes.byref(cfg)) == 2
    assert lib.litevggt_default_config(4, 16, 16, 0.5, None) == 1                   # null
    # handle-taking calls reject NULL handles without touching a device
    assert lib.litevggt_sizes(None, None, None, None, None, None) == 1
    assert lib.litevggt_merge(None, None, None, None, None) == 1
    assert lib.litevggt_plan_destroy(None) == 0 and lib.litevggt_destroy(None) == 0
