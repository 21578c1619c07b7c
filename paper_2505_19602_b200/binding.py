"""ctypes binding of libscalekv.so: argument marshalling only.

Function names equal the C ABI's (include/scalekv.h).  PyTorch provides device memory and
streams; every step of the path runs inside the library's CUDA kernels.  There is no CPU
fallback: a missing or unloadable library raises.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libscalekv.so")
SOURCES = [os.path.join(_HERE, "csrc", f) for f in ("scalekv.cu", "select_static.cu", "kernels_simt.cuh", "attend_tc.cuh", "common.cuh")]
HEADER = os.path.join(os.path.dirname(_HERE), "include", "scalekv.h")

KEEP_ALL = -1
MAX_WINDOW = 64
BF16, F32 = 0, 1
STATUS_NAMES = ["OK", "INVALID_ARG", "BAD_STATE", "CAPACITY", "UNSUPPORTED", "CUDA", "TIMEOUT", "DEVICE_CHECK"]
KERNEL_CLASSES = ["append", "attend", "score", "select", "compact", "other", "compress"]


class ScaleKVError(RuntimeError):
    def __init__(self, status, text=""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"scalekv status {name}: {text}")


class scalekv_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("dtype", C.c_int32), ("n_scales", C.c_int32),
        ("scale_h", C.POINTER(C.c_int32)), ("scale_w", C.POINTER(C.c_int32)), ("budgets", C.POINTER(C.c_int32)),
        ("max_window", C.c_int32), ("softmax_scale", C.c_float), ("page_tokens", C.c_int32),
        ("pool", C.c_void_p), ("pool_bytes", C.c_size_t),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("stream_main", C.c_void_p), ("stream_side", C.c_void_p), ("device", C.c_int32), ("window_patches", C.c_int32),
        ("window_kind", C.c_int32),
    ]


class scalekv_select_opts(C.Structure):
    _fields_ = [("policy", C.c_int32), ("pool_kernel", C.c_int32), ("n_sink", C.c_int32), ("head_shared", C.c_int32),
                ("head_budgets", C.POINTER(C.c_int32)), ("separate_kernels", C.c_int32)]


class scalekv_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_t", C.c_int64)]


def build_library(force=False, verbose=False):
    """Compiles the CUDA sources for sm_100a into libscalekv.so (in-tree) when out of date."""
    if not force and os.path.exists(LIB_PATH):
        newest = max(os.path.getmtime(p) for p in SOURCES + [HEADER] if os.path.exists(p))
        if os.path.getmtime(LIB_PATH) >= newest:
            return LIB_PATH
    cmd = ["nvcc", "-shared", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-O3", "-std=c++17", SOURCES[0], SOURCES[1], "-o", LIB_PATH]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return LIB_PATH


_lib = None


def load_library():
    """Loads libscalekv.so and declares every entry point of the header."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        build_library()
    lib = C.CDLL(LIB_PATH)
    ctx_p = C.c_void_p
    i32, i64, f64 = C.c_int32, C.c_int64, C.c_double
    T = scalekv_tensor
    P = C.POINTER
    sig = {
        "scalekv_query_sizes": [P(scalekv_config), P(C.c_size_t), P(C.c_size_t)],
        "scalekv_init": [P(scalekv_config), P(ctx_p)],
        "scalekv_reset": [ctx_p],
        "scalekv_destroy": [ctx_p],
        "scalekv_append": [ctx_p, i32, i32, T, T],
        "scalekv_attend": [ctx_p, i32, T, T, C.c_void_p],
        "scalekv_compress": [ctx_p, i32, T, i32, P(i32), i32],
        "scalekv_compress_ex": [ctx_p, i32, T, i32, P(i32), i32, P(scalekv_select_opts)],
        "scalekv_step": [ctx_p, i32, i32, T, T, T, T, P(C.c_float), i32, P(i32)],
        "scalekv_step_ex": [ctx_p, i32, i32, T, T, T, T, P(C.c_float), i32, i32, P(i32), P(scalekv_select_opts)],
        "scalekv_step_host": [ctx_p, i32, i32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, i32, P(i32)],
        "scalekv_layer_stats": [ctx_p, i32, T, i32, i32, P(f64), P(f64)],
        "scalekv_layer_stats_ex": [ctx_p, i32, T, i32, i32, P(f64), P(f64), P(f64), P(f64), P(f64)],
        "scalekv_window_centroids": [i32, i32, i32, P(i32), P(i32)],
        "scalekv_assign_roles": [P(f64), i32, i32, i32, i32, f64, P(C.c_uint8)],
        "scalekv_make_budgets": [P(C.c_uint8), i32, i32, f64, f64, f64, P(i32)],
        "scalekv_lengths": [ctx_p, i32, P(i32)],
        "scalekv_export_slice": [ctx_p, i32, i32, i32, P(i32), C.c_void_p, C.c_void_p, i32, P(i32)],
        "scalekv_export_scores": [ctx_p, i32, i32, P(C.c_float), i32, P(i32)],
        "scalekv_sync": [ctx_p],
        "scalekv_join": [ctx_p],
        "scalekv_budget_tokens": [f64, P(i32), P(i32), i32, P(i32)],
        "scalekv_window_last": [i32, i32, i32, P(i32), P(i32)],
        "scalekv_policy_budgets": [i32, i32, i32, f64, f64, P(i32)],
        "scalekv_selftest_wait": [ctx_p, i32, P(i32), P(i32)],
        "scalekv_launch_count": [ctx_p, P(i64)],
        "scalekv_profile_enable": [ctx_p, i32],
        "scalekv_profile_read": [ctx_p, i32, P(f64), P(i64)],
        "scalekv_select_static": [C.c_void_p, i32, i32, i32, i32, C.c_void_p, C.c_void_p],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.scalekv_error_string.argtypes = [ctx_p]
    lib.scalekv_error_string.restype = C.c_char_p
    _lib = lib
    return lib


def exported_symbols():
    """Names declared by the header (parsed from its text)."""
    import re

    text = open(HEADER).read()
    return sorted(set(re.findall(r"\b(scalekv_[a-z_]+)\s*\(", text)))


def _i32_array(values):
    arr = (C.c_int32 * len(values))(*[int(v) for v in values])
    return arr


def tensor_arg(t: torch.Tensor) -> scalekv_tensor:
    """[B, H, n, d] tensor -> view with element strides; the last axis must be contiguous."""
    assert t.dim() == 4 and t.stride(3) == 1, "expected [B, H, n, d] with contiguous head_dim"
    return scalekv_tensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


# ---- host-only helpers ----------------------------------------------------------------------
def scalekv_window_centroids(h, w, n_patches=16):
    lib = load_library()
    pos = (C.c_int32 * max(n_patches, 1))()
    cnt = C.c_int32(0)
    st = lib.scalekv_window_centroids(h, w, n_patches, pos, C.byref(cnt))
    if st:
        raise ScaleKVError(st)
    return [pos[i] for i in range(cnt.value)]


def scalekv_assign_roles(asi, n_drafters, mode=0, eps=1e-6):
    import numpy as np

    lib = load_library()
    a = np.ascontiguousarray(asi, dtype=np.float64)
    L, K = a.shape
    out = np.zeros((L, K), dtype=np.uint8)
    st = lib.scalekv_assign_roles(a.ctypes.data_as(C.POINTER(C.c_double)), L, K, n_drafters, mode, eps,
                                  out.ctypes.data_as(C.POINTER(C.c_uint8)))
    if st:
        raise ScaleKVError(st)
    return out.astype(bool)


def scalekv_make_budgets(is_drafter, b_uniform, b_r0, delta):
    import numpy as np

    lib = load_library()
    r = np.ascontiguousarray(is_drafter, dtype=np.uint8)
    L, K = r.shape
    out = np.zeros((L, K), dtype=np.int32)
    st = lib.scalekv_make_budgets(r.ctypes.data_as(C.POINTER(C.c_uint8)), L, K, b_uniform, b_r0, delta,
                                  out.ctypes.data_as(C.POINTER(C.c_int32)))
    if st:
        raise ScaleKVError(st)
    return out


def scalekv_window_last(h, w, n_obs=16):
    lib = load_library()
    pos = (C.c_int32 * max(n_obs, 1))()
    cnt = C.c_int32(0)
    st = lib.scalekv_window_last(h, w, n_obs, pos, C.byref(cnt))
    if st:
        raise ScaleKVError(st)
    return [pos[i] for i in range(cnt.value)]


def scalekv_policy_budgets(shape, n_layers, n_scales, b_mean, beta=20.0):
    """Budget table [L][K] of a comparison policy: shape "uniform" or "pyramid" (see include/scalekv.h)."""
    import numpy as np

    lib = load_library()
    out = np.zeros((n_layers, n_scales), dtype=np.int32)
    st = lib.scalekv_policy_budgets({"uniform": 0, "pyramid": 1}[shape], n_layers, n_scales, float(b_mean), float(beta),
                                    out.ctypes.data_as(C.POINTER(C.c_int32)))
    if st:
        raise ScaleKVError(st)
    return out


def scalekv_budget_tokens(fraction, sides_h, sides_w=None):
    """Tokens that a budget quoted as a fraction of the cached tokens T_c = N_{K-1} stands for (rounded half up)."""
    lib = load_library()
    sides_w = sides_h if sides_w is None else sides_w
    out = C.c_int32(0)
    st = lib.scalekv_budget_tokens(float(fraction), _i32_array(sides_h), _i32_array(sides_w), len(sides_h), C.byref(out))
    if st:
        raise ScaleKVError(st, "scalekv_budget_tokens")
    return out.value


def scalekv_select_static(scores: torch.Tensor, k: int, idx_out: torch.Tensor = None, stream=None):
    """Allocation-free top-k: scores [n_rows, len] float32 on the current CUDA device (row stride
    = scores.stride(0)); returns idx_out [n_rows, k] int32, the ascending indices of each row's k
    largest scores.  The library call itself allocates nothing; pass idx_out to avoid the torch
    allocation made here for convenience."""
    lib = load_library()
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.dim() == 2 and scores.stride(1) == 1
    n_rows, length = scores.shape
    if idx_out is None:
        idx_out = torch.empty(n_rows, k, dtype=torch.int32, device=scores.device)
    st = stream if stream is not None else torch.cuda.current_stream(scores.device)
    rc = lib.scalekv_select_static(scores.data_ptr(), n_rows, length, scores.stride(0), k, idx_out.data_ptr(), st.cuda_stream)
    if rc:
        raise ScaleKVError(rc, "scalekv_select_static")
    return idx_out


# ---- the context ---------------------------------------------------------------------------
class ScaleKV:
    """Owns the device pool / workspace (torch tensors) and one library context."""

    def __init__(self, n_layers, batch, n_heads, head_dim, dtype, sides_h, sides_w, budgets, max_window=16,
                 softmax_scale=0.0, page_tokens=0, device=0, side_stream=True, window_patches=16, window_kind="centroids"):
        if not torch.cuda.is_available():
            raise RuntimeError("ScaleKV needs a CUDA device (sm_100a); there is no CPU path")
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        self.n_layers, self.batch, self.n_heads, self.head_dim = n_layers, batch, n_heads, head_dim
        self.dtype = {"bf16": BF16, "f32": F32, BF16: BF16, F32: F32}[dtype]
        self.torch_dtype = torch.bfloat16 if self.dtype == BF16 else torch.float32
        self.sides_h, self.sides_w = list(sides_h), list(sides_w)
        self.n = [h * w for h, w in zip(self.sides_h, self.sides_w)]
        self.n_scales = len(self.n)
        flat = [int(x) for row in budgets for x in row]
        assert len(flat) == n_layers * self.n_scales
        self._h, self._w, self._b = _i32_array(self.sides_h), _i32_array(self.sides_w), _i32_array(flat)
        cfg = scalekv_config()
        cfg.n_layers, cfg.batch, cfg.n_heads, cfg.head_dim = n_layers, batch, n_heads, head_dim
        cfg.dtype, cfg.n_scales = self.dtype, self.n_scales
        cfg.scale_h, cfg.scale_w, cfg.budgets = self._h, self._w, self._b
        cfg.max_window, cfg.softmax_scale, cfg.page_tokens, cfg.device = max_window, softmax_scale, page_tokens, device
        cfg.window_patches = window_patches if window_patches <= max_window else 0
        cfg.window_kind = {"centroids": 0, "last": 1}[window_kind]
        pb, wb = C.c_size_t(0), C.c_size_t(0)
        st = self.lib.scalekv_query_sizes(C.byref(cfg), C.byref(pb), C.byref(wb))
        if st:
            raise ScaleKVError(st, "scalekv_query_sizes")
        self.pool_bytes, self.workspace_bytes = pb.value, wb.value
        with torch.cuda.device(self.device):
            # the library wants the pool 1024-byte and the workspace 256-byte aligned; the allocator only
            # promises 512 bytes, so allocate a little more and start at the next boundary
            self._pool_raw = torch.empty(pb.value + 1024, dtype=torch.uint8, device=self.device)
            self.pool = self._pool_raw[(-self._pool_raw.data_ptr()) % 1024:][:pb.value]
            self.workspace = torch.empty(wb.value, dtype=torch.uint8, device=self.device)
            self.stream_main = torch.cuda.Stream(device=self.device)
            self.stream_side = torch.cuda.Stream(device=self.device) if side_stream else self.stream_main
        cfg.pool, cfg.pool_bytes = self.pool.data_ptr(), pb.value
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), wb.value
        cfg.stream_main, cfg.stream_side = self.stream_main.cuda_stream, self.stream_side.cuda_stream
        self.ctx = C.c_void_p(None)
        torch.cuda.synchronize(self.device)
        st = self.lib.scalekv_init(C.byref(cfg), C.byref(self.ctx))
        if st:
            raise ScaleKVError(st, "scalekv_init")
        self.cfg = cfg

    # -- plumbing
    def _check(self, st):
        if st:
            raise ScaleKVError(st, self.lib.scalekv_error_string(self.ctx).decode())

    def close(self):
        if getattr(self, "ctx", None) and self.ctx.value:
            self.lib.scalekv_destroy(self.ctx)
            self.ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI, same names
    def scalekv_reset(self):
        self._check(self.lib.scalekv_reset(self.ctx))

    def scalekv_append(self, layer, scale, K, V):
        self._check(self.lib.scalekv_append(self.ctx, layer, scale, tensor_arg(K), tensor_arg(V)))

    def scalekv_attend(self, layer, Q, O=None, lse=None):
        if O is None:
            O = torch.empty_like(Q)
        self._check(self.lib.scalekv_attend(self.ctx, layer, tensor_arg(Q), tensor_arg(O),
                                            None if lse is None else lse.data_ptr()))
        return O

    def scalekv_compress(self, layer, Qw, window_pos=None, qw_is_full_map=False):
        if window_pos is None:
            self._check(self.lib.scalekv_compress(self.ctx, layer, tensor_arg(Qw), 0, None, int(qw_is_full_map)))
        else:
            wp = _i32_array(window_pos)
            self._check(self.lib.scalekv_compress(self.ctx, layer, tensor_arg(Qw), len(window_pos), wp, int(qw_is_full_map)))

    def scalekv_compress_ex(self, layer, Qw=None, window_pos=None, qw_is_full_map=False, policy="score", pool_kernel=1,
                            n_sink=0, head_shared=False, head_budgets=None, separate_kernels=False):
        """scalekv_compress with a selection variant: policy "score" (optionally pooled) or "recent"."""
        hb = _i32_array(head_budgets) if head_budgets is not None else None
        opts = scalekv_select_opts({"score": 0, "recent": 1}[policy], pool_kernel, n_sink, int(head_shared), hb,
                                   int(separate_kernels))
        q = tensor_arg(Qw) if Qw is not None else scalekv_tensor(None, 0, 0, 0)
        if window_pos is None:
            wp, w = None, 0
        else:
            wp, w = _i32_array(window_pos), len(window_pos)
        self._check(self.lib.scalekv_compress_ex(self.ctx, layer, q, w, wp, int(qw_is_full_map), C.byref(opts)))

    def scalekv_step(self, layer, scale, Q, K, V, O, window_pos=None, whole_map=False, lse=None):
        """append + attend + compress (window rows taken from Q) in one call; window_pos None and not whole_map: no compress.
        window_pos may be a prepared ctypes int32 array (see window_array)."""
        if whole_map:
            w, wp = -1, None
        elif window_pos is None:
            w, wp = 0, None
        else:
            wp = window_pos if isinstance(window_pos, C.Array) else _i32_array(window_pos)
            w = len(wp)
        lp = C.cast(lse.data_ptr(), C.POINTER(C.c_float)) if lse is not None else None
        self._check(self.lib.scalekv_step(self.ctx, layer, scale, tensor_arg(Q), tensor_arg(K), tensor_arg(V), tensor_arg(O),
                                          lp, w, wp))

    @staticmethod
    def window_array(window_pos):
        """The window as the ctypes array the calls take, so that a loop need not rebuild it."""
        return _i32_array(window_pos)

    def scalekv_step_ex(self, layer, scale, Q, K, V, O, compress=True, window_pos=None, lse=None, policy="score", pool_kernel=1,
                        n_sink=0, head_shared=False, head_budgets=None, separate_kernels=False):
        """append + attend + scalekv_compress_ex (Q as the full current map) in one call; compress=False: no compress."""
        hb = _i32_array(head_budgets) if head_budgets is not None else None
        opts = scalekv_select_opts({"score": 0, "recent": 1}[policy], pool_kernel, n_sink, int(head_shared), hb,
                                   int(separate_kernels))
        if window_pos is None:
            wp, w = None, 0
        else:
            wp = window_pos if isinstance(window_pos, C.Array) else _i32_array(window_pos)
            w = len(wp)
        lp = C.cast(lse.data_ptr(), C.POINTER(C.c_float)) if lse is not None else None
        self._check(self.lib.scalekv_step_ex(self.ctx, layer, scale, tensor_arg(Q), tensor_arg(K), tensor_arg(V), tensor_arg(O),
                                             lp, int(bool(compress)), w, wp, C.byref(opts)))

    def scalekv_step_host(self, layer, scale, Qh, Kh, Vh, Oh, staging, window_pos=None, whole_map=False):
        if whole_map:
            w, wp = -1, None
        elif window_pos is None:
            w, wp = 0, None
        else:
            w, wp = len(window_pos), _i32_array(window_pos)
        self._check(self.lib.scalekv_step_host(self.ctx, layer, scale, Qh.data_ptr(), Kh.data_ptr(), Vh.data_ptr(),
                                               Oh.data_ptr(), staging.data_ptr(), staging.numel() * staging.element_size(),
                                               w, wp))

    def scalekv_layer_stats(self, layer, Q, topk_prime=16, query_stride=1):
        car, htk = C.c_double(0), C.c_double(0)
        self._check(self.lib.scalekv_layer_stats(self.ctx, layer, tensor_arg(Q), topk_prime, query_stride,
                                                 C.byref(car), C.byref(htk)))
        return car.value, htk.value

    def scalekv_layer_stats_ex(self, layer, Q, topk_prime=16, query_stride=1):
        """(car, htk, car per slice, htk per slice, normalized current attention per slice); lists are [B][H]."""
        car, htk = C.c_double(0), C.c_double(0)
        n = self.batch * self.n_heads
        cs, ts, ns = (C.c_double * n)(), (C.c_double * n)(), (C.c_double * n)()
        self._check(self.lib.scalekv_layer_stats_ex(self.ctx, layer, tensor_arg(Q), topk_prime, query_stride,
                                                    C.byref(car), C.byref(htk), cs, ts, ns))
        shape = lambda a: [[a[b * self.n_heads + h] for h in range(self.n_heads)] for b in range(self.batch)]
        return car.value, htk.value, shape(cs), shape(ts), shape(ns)

    def scalekv_lengths(self, layer):
        out = (C.c_int32 * (self.batch * self.n_heads))()
        self._check(self.lib.scalekv_lengths(self.ctx, layer, out))
        return [[out[b * self.n_heads + h] for h in range(self.n_heads)] for b in range(self.batch)]

    def scalekv_export_slice(self, layer, b, h, with_kv=False, cap=None):
        cap = cap or (sum(self.n) + 8)
        pos = torch.empty(cap, dtype=torch.int32)
        n = C.c_int32(0)
        Kh = Vh = None
        if with_kv:
            Kh = torch.empty(cap, self.head_dim, dtype=self.torch_dtype)
            Vh = torch.empty(cap, self.head_dim, dtype=self.torch_dtype)
        self._check(self.lib.scalekv_export_slice(self.ctx, layer, b, h, C.cast(pos.data_ptr(), C.POINTER(C.c_int32)),
                                                  Kh.data_ptr() if with_kv else None, Vh.data_ptr() if with_kv else None,
                                                  cap, C.byref(n)))
        if with_kv:
            return pos[: n.value], Kh[: n.value], Vh[: n.value]
        return pos[: n.value]

    def scalekv_export_scores(self, b, h, cap=None):
        cap = cap or (sum(self.n) + 8)
        s = torch.empty(cap, dtype=torch.float32)
        n = C.c_int32(0)
        self._check(self.lib.scalekv_export_scores(self.ctx, b, h, C.cast(s.data_ptr(), C.POINTER(C.c_float)), cap, C.byref(n)))
        return s[: n.value]

    def scalekv_sync(self):
        self._check(self.lib.scalekv_sync(self.ctx))

    def scalekv_join(self):
        self._check(self.lib.scalekv_join(self.ctx))

    def scalekv_selftest_wait(self, limit_ms=50):
        """(gave_up, seen_by_peer) of the bounded-wait self-test; leaves the context's device status at TIMEOUT."""
        a, b = C.c_int32(0), C.c_int32(0)
        self._check(self.lib.scalekv_selftest_wait(self.ctx, int(limit_ms), C.byref(a), C.byref(b)))
        return a.value, b.value

    def scalekv_launch_count(self):
        n = C.c_int64(0)
        self._check(self.lib.scalekv_launch_count(self.ctx, C.byref(n)))
        return n.value

    def scalekv_profile_enable(self, on=1):
        """0 off, 1 events on the launching streams, 2 events with compress serialised onto stream_main."""
        self._check(self.lib.scalekv_profile_enable(self.ctx, int(on)))

    def scalekv_profile_read(self):
        out = {}
        for i, name in enumerate(KERNEL_CLASSES):
            ms, n = C.c_double(0), C.c_int64(0)
            self._check(self.lib.scalekv_profile_read(self.ctx, i, C.byref(ms), C.byref(n)))
            out[name] = (ms.value, n.value)
        return out
