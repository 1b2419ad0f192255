"""ctypes binding of the C ABI in ``include/litevggt.h``.

Argument marshalling only: every step of the path runs inside the CUDA library.  Tensors
are torch CUDA tensors (device memory and streams are PyTorch's); the binding passes
``data_ptr()`` and the current stream's handle.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

CLS_PROTECTED, CLS_GA, CLS_DST, CLS_SRC = 0, 1, 2, 3

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class LiteVGGTError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().litevggt_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code})")


class Config(C.Structure):
    _fields_ = [
        ("frames", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32), ("patch_px", C.c_int32),
        ("n_special", C.c_int32), ("dim", C.c_int32), ("heads", C.c_int32), ("merge_ratio", C.c_float),
        ("ga_keep_frac", C.c_float), ("alpha", C.c_float), ("beta", C.c_float), ("cell_h", C.c_int32),
        ("cell_w", C.c_int32), ("var_window", C.c_int32), ("recompute_interval", C.c_int32),
        ("qkv_dtype", C.c_int32),
    ]


def library_path() -> str:
    return os.path.join(_HERE, "liblitevggt.so")


class AttnExt(C.Structure):
    """Mirror of litevggt_attn_ext."""
    _fields_ = [("q_norm_gamma", C.c_void_p), ("q_norm_beta", C.c_void_p), ("k_norm_gamma", C.c_void_p),
                ("k_norm_beta", C.c_void_p), ("norm_eps", C.c_float), ("rope", C.c_int32), ("rope_base", C.c_float)]


def load_library():
    """Load liblitevggt.so (once).  Raises if it has not been built: there is no fallback."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2512_04939_b200.build`")
    lib = C.CDLL(path)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
    P = C.POINTER
    sigs = {
        "litevggt_default_config": [i32, i32, i32, C.c_float, P(Config)],
        "litevggt_create": [P(Config), C.c_int, P(vp)],
        "litevggt_destroy": [vp],
        "litevggt_sizes": [vp, P(i64), P(i64), P(i64), P(i64), P(C.c_size_t)],
        "litevggt_grad_map": [vp, vp, vp, vp],
        "litevggt_merge_plan": [vp, vp, vp, P(vp), vp],
        "litevggt_merge_plan_with_partition": [vp, vp, vp, P(vp), vp],
        "litevggt_merge": [vp, vp, vp, vp, vp],
        "litevggt_global_attn": [vp, vp, i64, vp, vp, vp, vp, vp, vp],
        "litevggt_global_attn_static": [vp, i64, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_global_attn_ext": [vp, vp, vp, i64, vp, vp, vp, vp, P(AttnExt), vp, vp],
        "litevggt_unmerge": [vp, vp, vp, vp, vp, vp],
        "litevggt_layernorm": [vp, vp, i64, vp, vp, C.c_float, vp, vp],
        "litevggt_frame_attn": [vp, vp, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_mlp": [vp, vp, i64, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_global_layer_host": [vp, P(vp), vp, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_global_layer_host_pipelined": [vp, P(vp), vp, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_host_drain": [vp, vp],
        "litevggt_timers_reset": [vp],
        "litevggt_timer_read": [vp, C.c_int, P(C.c_float), P(i32)],
        "litevggt_timer_samples": [vp, C.c_int, P(C.c_float), i32, P(i32)],
        "litevggt_linear": [vp, vp, i64, i64, vp, i64, vp, vp, vp],
        "litevggt_should_refresh": [vp, vp, i32, P(i32)],
        "litevggt_plan_export": [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp],
        "litevggt_plan_import": [vp, vp, P(vp)],
        "litevggt_plan_destroy": [vp],
        "litevggt_debug_buffer": [vp, C.c_int, P(vp), P(C.c_size_t)],
        "litevggt_poll_device_status": [vp, vp],
        "litevggt_selftest_bounded_wait": [vp, i64, P(C.c_uint32), vp],
        "litevggt_launch_count": [vp, P(i64)],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.litevggt_status_string.argtypes = [C.c_int]
    lib.litevggt_status_string.restype = C.c_char_p
    _LIB = lib
    return lib


def _check(code: int, where: str):
    if code != 0:
        raise LiteVGGTError(code, where)


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


STATIC_ATTN_MAX_ROWS = 1024


def _check_static_attn_args(xm, w_qkv, b_qkv, w_o, b_o, out, device_status):
    """The C entry point is told only m and trusts every extent, so a wrong shape, dtype or device
    would send its kernels past the end of an allocation: refuse such arguments here, before any
    launch.  Shapes first, so that the message names the actual mistake."""
    d = 1024
    if xm.dim() != 2 or xm.shape[1] != d or not 1 <= xm.shape[0] <= STATIC_ATTN_MAX_ROWS:
        raise ValueError(f"x_merged must be [m, {d}] with 1 <= m <= {STATIC_ATTN_MAX_ROWS}, got {tuple(xm.shape)}")
    wanted = {"w_qkv": (w_qkv, (3 * d, d)), "w_o": (w_o, (d, d)), "b_qkv": (b_qkv, (3 * d,)), "b_o": (b_o, (d,)),
              "out": (out, tuple(xm.shape))}
    for name, (t, shape) in wanted.items():
        if t is None:
            if name in ("b_qkv", "b_o"):
                continue
            raise ValueError(f"{name} is required")
        if tuple(t.shape) != shape:
            raise ValueError(f"{name} must have shape {shape}, got {tuple(t.shape)}")
    for name, t in (("x_merged", xm), ("w_qkv", w_qkv), ("b_qkv", b_qkv), ("w_o", w_o), ("b_o", b_o), ("out", out)):
        if t is None:
            continue
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous bfloat16 tensor")
    if device_status is not None and (device_status.dtype != torch.int32 or device_status.numel() != 1):
        raise ValueError("device_status must be one int32 element")
    tensors = [t for t in (xm, w_qkv, b_qkv, w_o, b_o, out, device_status) if t is not None]
    if not all(t.is_cuda for t in tensors):
        raise ValueError("every tensor must live on a CUDA device")
    current = torch.cuda.current_device()
    if any(t.device.index != current for t in tensors):
        raise ValueError(f"every tensor must live on the current device (cuda:{current}): the entry point works there")


def global_attn_static(xm, w_qkv, b_qkv, w_o, b_o, out=None, device_status=None):
    """Attention layer over up to STATIC_ATTN_MAX_ROWS merged rows through the entry point that
    allocates nothing (no context; intermediates in the library's own fixed device array).  The
    output tensor is the caller's; pass ``out`` to keep this wrapper from allocating one.
    ``device_status``: optional int32 CUDA tensor of one element that receives the kernels' flag.
    Shapes, dtypes and devices are checked here, because the C entry point cannot."""
    lib = load_library()
    if out is None:
        out = torch.empty_like(xm)
    _check_static_attn_args(xm, w_qkv, b_qkv, w_o, b_o, out, device_status)
    _check(lib.litevggt_global_attn_static(_ptr(xm), xm.shape[0], _ptr(w_qkv), _ptr(b_qkv), _ptr(w_o), _ptr(b_o),
                                           _ptr(out), _ptr(device_status), _stream()), "global_attn_static")
    return out


class _DeviceBuffer:
    """Exposes a raw device pointer to torch through the CUDA array interface (int16 words)."""

    def __init__(self, ptr: int, shape):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": "<i2", "data": (ptr, False), "version": 2}


class Plan:
    """The cached merge indices (index-cache handle)."""

    def __init__(self, owner: "LiteVGGT", handle):
        self.owner = owner
        self.handle = handle

    def destroy(self):
        if self.handle is not None and self.handle.value:
            load_library().litevggt_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.destroy()
        except Exception:
            pass


class LiteVGGT:
    """One context = one sequence shape (frames, patch grid, merge ratio) on one GPU."""

    def __init__(self, frames, grid_h, grid_w, merge_ratio, device=0, **overrides):
        lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2512_04939_b200 needs a CUDA device (sm_100); there is no CPU path")
        self.lib = lib
        cfg = Config()
        _check(lib.litevggt_default_config(frames, grid_h, grid_w, merge_ratio, C.byref(cfg)), "default_config")
        for k, v in overrides.items():
            setattr(cfg, k, v)
        self.cfg = cfg
        self.device = torch.device("cuda", device)
        self.handle = C.c_void_p()
        _check(lib.litevggt_create(C.byref(cfg), device, C.byref(self.handle)), "create")
        n, m, ns, nd, wb = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64(), C.c_size_t()
        _check(lib.litevggt_sizes(self.handle, C.byref(n), C.byref(m), C.byref(ns), C.byref(nd), C.byref(wb)), "sizes")
        self.n_tokens, self.n_merged, self.n_src, self.n_dst = n.value, m.value, ns.value, nd.value
        self.workspace_bytes = wb.value
        self.dim = cfg.dim

    def close(self):
        if self.handle is not None and self.handle.value:
            self.lib.litevggt_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ path
    def grad_map(self, images: torch.Tensor) -> torch.Tensor:
        c = self.cfg
        assert images.dtype == torch.float32 and images.shape == (c.frames, 3, c.grid_h * c.patch_px, c.grid_w * c.patch_px)
        grad = torch.empty(c.frames, c.grid_h, c.grid_w, dtype=torch.float32, device=self.device)
        _check(self.lib.litevggt_grad_map(self.handle, _ptr(images), _ptr(grad), _stream()), "grad_map")
        return grad

    def merge_plan(self, x: torch.Tensor, grad: torch.Tensor, plan: Plan | None = None) -> Plan:
        assert x.dtype == torch.bfloat16 and x.shape == (self.n_tokens, self.dim)
        h = plan.handle if plan is not None else C.c_void_p()
        _check(self.lib.litevggt_merge_plan(self.handle, _ptr(x), _ptr(grad), C.byref(h), _stream()), "merge_plan")
        return plan if plan is not None else Plan(self, h)

    def merge_plan_with_partition(self, x: torch.Tensor, cls: torch.Tensor, plan: Plan | None = None) -> Plan:
        assert x.dtype == torch.bfloat16 and x.shape == (self.n_tokens, self.dim)
        assert cls.dtype == torch.uint8 and cls.numel() == self.n_tokens
        h = plan.handle if plan is not None else C.c_void_p()
        _check(self.lib.litevggt_merge_plan_with_partition(self.handle, _ptr(x), _ptr(cls), C.byref(h), _stream()),
               "merge_plan_with_partition")
        return plan if plan is not None else Plan(self, h)

    def merge(self, plan: Plan, x: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.dtype == torch.bfloat16 and x.shape == (self.n_tokens, self.dim)
        if out is None:
            out = torch.empty(self.n_merged, self.dim, dtype=torch.bfloat16, device=self.device)
        _check(self.lib.litevggt_merge(self.handle, plan.handle, _ptr(x), _ptr(out), _stream()), "merge")
        return out

    def global_attn(self, xm, w_qkv, b_qkv, w_o, b_o, out: torch.Tensor | None = None) -> torch.Tensor:
        assert xm.dtype == torch.bfloat16 and xm.shape == (self.n_merged, self.dim)
        assert w_qkv.shape == (3 * self.dim, self.dim) and w_o.shape == (self.dim, self.dim)
        if out is None:
            out = torch.empty_like(xm)
        _check(self.lib.litevggt_global_attn(self.handle, _ptr(xm), self.n_merged, _ptr(w_qkv), _ptr(b_qkv),
                                             _ptr(w_o), _ptr(b_o), _ptr(out), _stream()), "global_attn")
        return out

    def global_attn_ext(self, plan, xm, w_qkv, b_qkv, w_o, b_o, q_norm=None, k_norm=None, norm_eps=1e-5,
                        rope=False, rope_base=100.0, out: torch.Tensor | None = None) -> torch.Tensor:
        """global_attn with per-head LayerNorm of Q and K (q_norm, k_norm: (gamma, beta) pairs of bf16 [64]
        tensors, both or neither) and / or the 2-D rotary embedding (positions come from ``plan``)."""
        assert xm.dtype == torch.bfloat16 and xm.shape == (self.n_merged, self.dim)
        if out is None:
            out = torch.empty_like(xm)
        ext = AttnExt()
        qg, qb = q_norm if q_norm is not None else (None, None)
        kg, kb = k_norm if k_norm is not None else (None, None)
        ext.q_norm_gamma, ext.q_norm_beta, ext.k_norm_gamma, ext.k_norm_beta = _ptr(qg), _ptr(qb), _ptr(kg), _ptr(kb)
        ext.norm_eps = norm_eps
        ext.rope = 1 if rope else 0
        ext.rope_base = rope_base
        h = plan.handle if plan is not None else None
        _check(self.lib.litevggt_global_attn_ext(self.handle, h, _ptr(xm), self.n_merged, _ptr(w_qkv), _ptr(b_qkv),
                                                 _ptr(w_o), _ptr(b_o), C.byref(ext), _ptr(out), _stream()),
               "global_attn_ext")
        return out

    def unmerge(self, plan: Plan, ym, residual=None, out: torch.Tensor | None = None) -> torch.Tensor:
        assert ym.dtype == torch.bfloat16 and ym.shape == (self.n_merged, self.dim)
        if out is None:
            out = torch.empty(self.n_tokens, self.dim, dtype=torch.bfloat16, device=self.device)
        _check(self.lib.litevggt_unmerge(self.handle, plan.handle, _ptr(ym), _ptr(residual), _ptr(out), _stream()),
               "unmerge")
        return out

    def global_layer_host(self, plan: Plan | None, x_host, w_qkv, b_qkv, w_o, b_o, out_host, grad=None) -> Plan:
        """x_host / out_host: CPU bf16 tensors [N, D] (pinned for asynchronous copies).  With
        ``grad`` the plan is (re)built from the uploaded tokens first.  Returns the plan."""
        assert x_host.device.type == "cpu" and out_host.device.type == "cpu"
        assert x_host.shape == (self.n_tokens, self.dim) and out_host.shape == x_host.shape
        h = plan.handle if plan is not None else C.c_void_p()
        _check(self.lib.litevggt_global_layer_host(self.handle, C.byref(h), _ptr(grad), _ptr(x_host), _ptr(w_qkv),
                                                   _ptr(b_qkv), _ptr(w_o), _ptr(b_o), _ptr(out_host), _stream()),
               "global_layer_host")
        return plan if plan is not None else Plan(self, h)

    def global_layer_host_pipelined(self, plan: Plan | None, x_host, w_qkv, b_qkv, w_o, b_o, out_host,
                                    grad=None) -> Plan:
        """global_layer_host for independent calls in a row: the copies run on the context's copy
        streams and overlap the neighbouring calls' kernels.  ``out_host`` is complete only after
        ``host_drain()`` and a synchronisation of the current stream."""
        assert x_host.device.type == "cpu" and out_host.device.type == "cpu"
        assert x_host.shape == (self.n_tokens, self.dim) and out_host.shape == x_host.shape
        h = plan.handle if plan is not None else C.c_void_p()
        _check(self.lib.litevggt_global_layer_host_pipelined(self.handle, C.byref(h), _ptr(grad), _ptr(x_host),
                                                             _ptr(w_qkv), _ptr(b_qkv), _ptr(w_o), _ptr(b_o),
                                                             _ptr(out_host), _stream()), "global_layer_host_pipelined")
        return plan if plan is not None else Plan(self, h)

    def host_drain(self):
        _check(self.lib.litevggt_host_drain(self.handle, _stream()), "host_drain")

    def layernorm(self, x, gamma, beta, eps=1e-6, out=None) -> torch.Tensor:
        assert x.dtype == torch.bfloat16 and x.shape[1] == self.dim
        if out is None:
            out = torch.empty_like(x)
        _check(self.lib.litevggt_layernorm(self.handle, _ptr(x), x.shape[0], _ptr(gamma), _ptr(beta), eps, _ptr(out),
                                           _stream()), "layernorm")
        return out

    def frame_attn(self, x, w_qkv, b_qkv, w_o, b_o, residual=None, out=None) -> torch.Tensor:
        assert x.dtype == torch.bfloat16 and x.shape == (self.n_tokens, self.dim)
        if out is None:
            out = torch.empty_like(x)
        _check(self.lib.litevggt_frame_attn(self.handle, _ptr(x), _ptr(w_qkv), _ptr(b_qkv), _ptr(w_o), _ptr(b_o),
                                            _ptr(residual), _ptr(out), _stream()), "frame_attn")
        return out

    def mlp(self, x, w1, b1, w2, b2, residual=None, out=None) -> torch.Tensor:
        assert x.dtype == torch.bfloat16 and x.shape[1] == self.dim
        if out is None:
            out = torch.empty_like(x)
        _check(self.lib.litevggt_mlp(self.handle, _ptr(x), x.shape[0], _ptr(w1), _ptr(b1), _ptr(w2), _ptr(b2),
                                     _ptr(residual), _ptr(out), _stream()), "mlp")
        return out

    def linear(self, a, w, bias=None) -> torch.Tensor:
        m, k = a.shape
        n = w.shape[0]
        out = torch.empty(m, n, dtype=torch.bfloat16, device=self.device)
        _check(self.lib.litevggt_linear(self.handle, _ptr(a), m, k, _ptr(w), n, _ptr(bias), _ptr(out), _stream()),
               "linear")
        return out

    # ------------------------------------------------------------------ cache handle
    def should_refresh(self, plan: Plan | None, global_layer_idx: int) -> bool:
        yes = C.c_int32()
        h = plan.handle if plan is not None else None
        _check(self.lib.litevggt_should_refresh(self.handle, h, global_layer_idx, C.byref(yes)), "should_refresh")
        return bool(yes.value)

    def plan_export(self, plan: Plan) -> dict:
        c = self.cfg
        fp = c.frames * c.grid_h * c.grid_w
        out = dict(
            dst_of=np.empty(self.n_tokens, np.int32), size=np.empty(self.n_merged, np.int32),
            kept_idx=np.empty(self.n_merged, np.int32), cls=np.empty(self.n_tokens, np.uint8),
            best_dst=np.empty(self.n_src, np.int32), best_sim=np.empty(self.n_src, np.float32),
            var=np.empty(fp, np.float32), ga=np.empty(fp, np.float32),
        )
        ptrs = [out[k].ctypes.data_as(C.c_void_p) for k in
                ("dst_of", "size", "kept_idx", "cls", "best_dst", "best_sim", "var", "ga")]
        _check(self.lib.litevggt_plan_export(self.handle, plan.handle, *ptrs, _stream()), "plan_export")
        out["var"] = out["var"].reshape(c.frames, c.grid_h, c.grid_w)
        out["ga"] = out["ga"].reshape(c.frames, c.grid_h, c.grid_w)
        return out

    def plan_import(self, dst_of: np.ndarray) -> Plan:
        arr = np.ascontiguousarray(dst_of, dtype=np.int32)
        assert arr.size == self.n_tokens
        h = C.c_void_p()
        _check(self.lib.litevggt_plan_import(self.handle, arr.ctypes.data_as(C.c_void_p), C.byref(h)), "plan_import")
        return Plan(self, h)

    def debug_buffer(self, which: int) -> torch.Tensor:
        """View of an internal buffer of the last global_attn call, copied to a new tensor
        (0: qkv [M,3D], 1: attention output [M,D])."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(self.lib.litevggt_debug_buffer(self.handle, which, C.byref(ptr), C.byref(nbytes)), "debug_buffer")
        cols = 3 * self.dim if which == 0 else self.dim
        view = _DeviceBuffer(ptr.value, (self.n_merged, cols))
        return torch.as_tensor(view, device=self.device).view(torch.bfloat16).clone()

    def debug_fp8_buffers(self) -> dict:
        """The E4M3 operands of the last global_attn call of a context made with qkv_dtype=1, copied
        out: q8, k8 uint8 [M, D]; v8t uint8 [D, round_up(M, 128)] (V transposed: row = head * 64 +
        channel, column = key, zero beyond M); amax float32 [3, heads] of Q, K, V."""
        out = {}
        m_pad = (self.n_merged + 127) // 128 * 128
        shapes = {2: ("q8", (self.n_merged, self.dim)), 3: ("k8", (self.n_merged, self.dim)), 4: ("v8t", (self.dim, m_pad))}
        for which, (name, shape) in shapes.items():
            ptr, nbytes = C.c_void_p(), C.c_size_t()
            _check(self.lib.litevggt_debug_buffer(self.handle, which, C.byref(ptr), C.byref(nbytes)), "debug_buffer")
            assert nbytes.value == shape[0] * shape[1]
            iface = {"shape": shape, "typestr": "|u1", "data": (ptr.value, False), "version": 2}
            holder = type("_U8", (), {"__cuda_array_interface__": iface})()
            out[name] = torch.as_tensor(holder, device=self.device).clone()
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(self.lib.litevggt_debug_buffer(self.handle, 5, C.byref(ptr), C.byref(nbytes)), "debug_buffer")
        iface = {"shape": (3, 16), "typestr": "<f4", "data": (ptr.value, False), "version": 2}
        holder = type("_F4", (), {"__cuda_array_interface__": iface})()
        out["amax"] = torch.as_tensor(holder, device=self.device).clone()
        return out

    TIMER_NAMES = ("grad_map", "var_map", "partition", "match", "index_build", "merge", "qkv_proj",
                   "attention", "out_proj", "unmerge", "layernorm", "frame_attn", "mlp", "qk_embed", "qkv_quantize")

    def timers_reset(self):
        _check(self.lib.litevggt_timers_reset(self.handle), "timers_reset")

    def timers_read(self) -> dict:
        """{step name: (total device ms, launches recorded)} since the last reset (synchronises)."""
        out = {}
        for i, name in enumerate(self.TIMER_NAMES):
            ms, cnt = C.c_float(), C.c_int32()
            _check(self.lib.litevggt_timer_read(self.handle, i, C.byref(ms), C.byref(cnt)), "timer_read")
            out[name] = (ms.value, cnt.value)
        return out

    def timers_samples(self) -> dict:
        """{step name: [device ms of each record since the last reset, oldest first]} (synchronises)."""
        out = {}
        buf = (C.c_float * 64)()
        for i, name in enumerate(self.TIMER_NAMES):
            cnt = C.c_int32()
            _check(self.lib.litevggt_timer_samples(self.handle, i, buf, 64, C.byref(cnt)), "timer_samples")
            out[name] = [float(buf[k]) for k in range(cnt.value)]
        return out

    def poll(self):
        """Synchronise the current stream; raise if a kernel flagged a timeout / bad index."""
        _check(self.lib.litevggt_poll_device_status(self.handle, _stream()), "poll_device_status")

    def selftest_bounded_wait(self, limit_cycles: int = 1_000_000) -> int:
        """Run the one-CTA kernel that waits on a barrier nobody arrives on; returns its outcome
        word (4 = ran to its end, no wait reported a false completion).  The next poll() raises
        LITEVGGT_ERR_DEVICE_TIMEOUT, the one after that is clean."""
        word = C.c_uint32(0)
        _check(self.lib.litevggt_selftest_bounded_wait(self.handle, int(limit_cycles), C.byref(word), _stream()),
               "selftest_bounded_wait")
        return int(word.value)

    def launch_count(self) -> int:
        n = C.c_int64()
        _check(self.lib.litevggt_launch_count(self.handle, C.byref(n)), "launch_count")
        return n.value
