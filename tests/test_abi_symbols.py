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


def test_static_attention_wrapper_refuses_bad_arguments_before_any_launch():
    """litevggt_global_attn_static is told only m and trusts every extent; its Python wrapper must
    turn a wrong shape, dtype or device into an error on the host (no GPU is touched here)."""
    import pytest
    import torch

    import paper_2512_04939_b200 as pkg

    bf = torch.bfloat16
    good = dict(xm=torch.zeros(16, 1024, dtype=bf), w_qkv=torch.zeros(3072, 1024, dtype=bf),
                b_qkv=torch.zeros(3072, dtype=bf), w_o=torch.zeros(1024, 1024, dtype=bf), b_o=torch.zeros(1024, dtype=bf))
    bad = [
        dict(xm=torch.zeros(16, 512, dtype=bf)),                      # half-width rows
        dict(xm=torch.zeros(pkg.STATIC_ATTN_MAX_ROWS + 1, 1024, dtype=bf)),
        dict(w_qkv=torch.zeros(1024, 1024, dtype=bf)),                # one projection instead of three
        dict(w_o=torch.zeros(1024, 512, dtype=bf)),
        dict(b_qkv=torch.zeros(1024, dtype=bf)),                      # short bias
        dict(b_o=torch.zeros(8, dtype=bf)),
        dict(xm=torch.zeros(16, 1024, dtype=torch.float32)),          # wrong dtype
        dict(w_o=torch.zeros(1024, 2048, dtype=bf)[:, ::2]),          # not contiguous
        dict(out=torch.zeros(8, 1024, dtype=bf)),                     # short output
        dict(device_status=torch.zeros(2, dtype=torch.int32)),
        dict(device_status=torch.zeros(1, dtype=torch.int64)),
    ]
    for change in bad:
        args = dict(good, out=None, device_status=None)
        args.update(change)
        with pytest.raises(ValueError):
            pkg.global_attn_static(args["xm"], args["w_qkv"], args["b_qkv"], args["w_o"], args["b_o"], out=args["out"],
                                   device_status=args["device_status"])
    # right shapes, but host tensors: refused as well (the entry point works on the current CUDA device)
    with pytest.raises(ValueError, match="CUDA"):
        pkg.global_attn_static(good["xm"], good["w_qkv"], good["b_qkv"], good["w_o"], good["b_o"])
