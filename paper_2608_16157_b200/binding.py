"""ctypes binding of the C ABI in ``include/ftmoe.h`` (argument marshalling only).

Every step of the layer runs in the CUDA library; nothing here computes.  There is no CPU
fallback: if the shared library is missing the import of :func:`load` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

FT_OK = 0
FT_ERR_INVALID_ARG, FT_ERR_NOT_PINNED, FT_ERR_OOM, FT_ERR_CUDA = 1, 2, 3, 4
FT_ERR_STATE, FT_ERR_TIMEOUT, FT_ERR_NONFINITE, FT_ERR_UNSUPPORTED = 5, 6, 7, 8
FT_W_BF16, FT_W_INT4_G128, FT_W_MXFP4, FT_W_NVFP4, FT_W_MXFP4_TC = 0, 1, 2, 3, 4
FT_FILL_COPY_ENGINE, FT_FILL_SM = 0, 1
STAT_NAMES = ("steps", "routed", "hits", "misses", "fills", "zc", "evictions", "pairs", "pairs_resident",
              "pairs_gemm")

# every symbol include/ftmoe.h declares
SYMBOLS = (
    "ft_moe_expert_bytes", "ft_moe_host_alloc", "ft_moe_host_free", "ft_moe_create", "ft_moe_destroy",
    "ft_moe_calibrate", "ft_moe_route", "ft_moe_plan", "ft_moe_fill", "ft_moe_forward", "ft_moe_layer",
    "ft_moe_layer_host", "ft_moe_get_routing", "ft_moe_get_slot_table", "ft_moe_read_slot",
    "ft_moe_get_stats", "ft_moe_reset", "ft_moe_sync_status", "ft_moe_last_fill", "ft_moe_launch_count",
    "ft_moe_status_string", "ft_moe_timing_enable", "ft_moe_timing_read", "ft_moe_ffn_noalloc",
    "ft_moe_last_cuda_error", "ft_moe_host_register", "ft_moe_host_unregister",
    "ft_moe_get_cta_trace", "ft_moe_set_split_min_pairs", "ft_moe_resize", "ft_moe_ffn_noalloc_status",
    "ft_moe_set_launch_overlap", "ft_moe_debug_inject", "ft_moe_prefetch_layer",
)
NOALLOC_MAX_TOKENS, NOALLOC_MAX_HIDDEN = 64, 2048
TIME_NAMES = ("route", "plan", "ffn_zc", "ffn_res", "finalize", "fill", "gather", "gemm1", "gemm2", "combine")


class Config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("device", C.c_int32), ("n_layers", C.c_int32), ("hidden", C.c_int32),
        ("inter", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32), ("n_shared", C.c_int32),
        ("wdtype", C.c_int32), ("slots_per_layer", C.c_int32), ("max_tokens", C.c_int32),
        ("fill_mode", C.c_int32),
        ("host_pool", C.c_void_p), ("host_pool_bytes", C.c_size_t), ("shared_weights", C.c_void_p),
        ("bw_fill_MBps", C.c_uint32), ("bw_zc_MBps", C.c_uint32), ("bw_zc_residual_MBps", C.c_uint32),
        ("bw_hbm_MBps", C.c_uint32), ("reuse_credit", C.c_int32), ("zc_tokens_per_pass", C.c_int32),
        ("hbm_tokens_per_pass", C.c_int32), ("gemm_min_tokens", C.c_int32), ("split_min_pairs", C.c_int32),
        ("global_pool", C.c_int32),
    ]


class PlanOut(C.Structure):
    _fields_ = [
        ("step", C.c_int64), ("n_routed", C.c_int32), ("n_hit", C.c_int32), ("n_miss", C.c_int32),
        ("n_fill", C.c_int32), ("n_zc", C.c_int32),
        ("hit", C.c_void_p), ("miss", C.c_void_p), ("fill", C.c_void_p), ("zc", C.c_void_p),
        ("fill_order", C.c_void_p), ("fill_slot", C.c_void_p), ("fill_evicted", C.c_void_p),
        ("loc", C.c_void_p),
    ]


class FtMoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code in (FT_ERR_CUDA, FT_ERR_OOM):
            detail = " [" + load().ft_moe_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {status_string(code)} ({code}){detail}")


_lib = None


def load(rebuild: bool = False):
    """Loads (building first if the sources are newer) ``lib/libftmoe.so``.  Raises if that fails."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = _build.LIB_PATH
    if rebuild or not os.path.exists(path):
        path = _build.build(force=rebuild)
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    sig = {
        "ft_moe_expert_bytes": (sz, [C.POINTER(Config)]),
        "ft_moe_host_alloc": (i32, [sz, C.POINTER(vp)]),
        "ft_moe_host_free": (i32, [vp]),
        "ft_moe_host_register": (i32, [vp, sz]),
        "ft_moe_get_cta_trace": (i32, [vp, vp, i32]),
        "ft_moe_set_split_min_pairs": (i32, [vp, i32]),
        "ft_moe_resize": (i32, [vp, i32]),
        "ft_moe_host_unregister": (i32, [vp]),
        "ft_moe_create": (i32, [C.POINTER(Config), C.POINTER(vp)]),
        "ft_moe_destroy": (i32, [vp]),
        "ft_moe_calibrate": (i32, [vp, C.POINTER(C.c_uint32)]),
        "ft_moe_route": (i32, [vp, i32, vp, i32, vp]),
        "ft_moe_plan": (i32, [vp, i32, C.POINTER(PlanOut), vp]),
        "ft_moe_fill": (i32, [vp, i32, vp]),
        "ft_moe_forward": (i32, [vp, i32, vp, vp, vp]),
        "ft_moe_layer": (i32, [vp, i32, vp, vp, vp, i32, vp]),
        "ft_moe_layer_host": (i32, [vp, i32, vp, vp, vp, i32, vp]),
        "ft_moe_get_routing": (i32, [vp, i32, vp, vp, vp, vp, vp, vp]),
        "ft_moe_get_slot_table": (i32, [vp, i32, vp, vp, vp]),
        "ft_moe_read_slot": (i32, [vp, i32, i32, vp]),
        "ft_moe_get_stats": (i32, [vp, i32, vp, i32]),
        "ft_moe_reset": (i32, [vp, i32]),
        "ft_moe_sync_status": (i32, [vp]),
        "ft_moe_last_fill": (i32, [vp, C.POINTER(C.c_float), C.POINTER(C.c_uint64)]),
        "ft_moe_launch_count": (i32, [vp, C.POINTER(C.c_uint64)]),
        "ft_moe_status_string": (C.c_char_p, [i32]),
        "ft_moe_timing_enable": (i32, [vp, i32]),
        "ft_moe_timing_read": (i32, [vp, vp, vp, i32]),
        "ft_moe_ffn_noalloc": (i32, [i32, vp, i32, i32, vp, vp, i32, vp]),
        "ft_moe_last_cuda_error": (C.c_char_p, []),
        "ft_moe_ffn_noalloc_status": (i32, [i32]),
        "ft_moe_set_launch_overlap": (i32, [vp, i32]),
        "ft_moe_debug_inject": (i32, [vp, C.c_uint32, C.c_uint32]),
        "ft_moe_prefetch_layer": (i32, [vp, i32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().ft_moe_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != FT_OK:
        raise FtMoeError(code, where)


def make_config(*, hidden, inter, n_experts, top_k, n_layers=1, slots_per_layer, max_tokens,
                host_pool_ptr, host_pool_bytes, wdtype=FT_W_BF16, n_shared=0, shared_ptr=None,
                fill_mode=FT_FILL_COPY_ENGINE, device=0, bw_fill=50000, bw_zc=50000, bw_zc_residual=0,
                bw_hbm=6000000, reuse_credit=1, zc_tokens_per_pass=64, hbm_tokens_per_pass=128,
                gemm_min_tokens=0, split_min_pairs=32, global_pool=0) -> Config:
    c = Config()
    c.struct_size = C.sizeof(Config)
    c.device, c.n_layers, c.hidden, c.inter = device, n_layers, hidden, inter
    c.n_experts, c.top_k, c.n_shared, c.wdtype = n_experts, top_k, n_shared, wdtype
    c.slots_per_layer, c.max_tokens, c.fill_mode = slots_per_layer, max_tokens, fill_mode
    c.host_pool, c.host_pool_bytes, c.shared_weights = host_pool_ptr, host_pool_bytes, shared_ptr
    c.bw_fill_MBps, c.bw_zc_MBps, c.bw_zc_residual_MBps, c.bw_hbm_MBps = bw_fill, bw_zc, bw_zc_residual, bw_hbm
    c.reuse_credit, c.zc_tokens_per_pass, c.hbm_tokens_per_pass = reuse_credit, zc_tokens_per_pass, hbm_tokens_per_pass
    c.gemm_min_tokens = gemm_min_tokens
    c.split_min_pairs = split_min_pairs
    c.global_pool = global_pool
    return c


def ft_moe_expert_bytes(cfg: Config) -> int:
    return int(load().ft_moe_expert_bytes(C.byref(cfg)))


def ft_moe_ffn_noalloc(device, record_dev, hidden, inter, x_dev, y_dev, T, stream=None) -> int:
    """One expert FFN on caller-held device memory without any allocation (scratch is a fixed array
    inside the library).  Returns the status code; see ``include/ftmoe.h`` for the limits."""
    return int(load().ft_moe_ffn_noalloc(device, _ptr(record_dev), hidden, inter, _ptr(x_dev), _ptr(y_dev), T,
                                         _stream(stream)))


def ft_moe_ffn_noalloc_status(device) -> int:
    """Waits for the device; returns and clears the status the allocation-free kernels latched there."""
    return int(load().ft_moe_ffn_noalloc_status(device))


class HostPool:
    """Pinned + mapped host memory from ``ft_moe_host_alloc`` viewed as a uint8 torch tensor."""

    def __init__(self, n_bytes: int):
        import torch
        self.ptr = C.c_void_p()
        _check(load().ft_moe_host_alloc(n_bytes, C.byref(self.ptr)), "ft_moe_host_alloc")
        self.n_bytes = n_bytes
        buf = (C.c_uint8 * n_bytes).from_address(self.ptr.value)
        self.tensor = torch.frombuffer(buf, dtype=torch.uint8)

    def free(self):
        if self.ptr is not None and self.ptr.value:
            self.tensor = None
            _check(load().ft_moe_host_free(self.ptr), "ft_moe_host_free")
            self.ptr = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class RegisteredPool:
    """Caller-owned host memory (a numpy array, e.g. a shared file mapping) pinned and mapped in place
    with ``ft_moe_host_register``; same interface as :class:`HostPool`."""

    def __init__(self, array: np.ndarray):
        import torch
        assert array.dtype == np.uint8 and array.flags["C_CONTIGUOUS"]
        self.array = array
        self.n_bytes = array.size
        self.ptr = C.c_void_p(array.ctypes.data)
        _check(load().ft_moe_host_register(self.ptr, self.n_bytes), "ft_moe_host_register")
        self.tensor = torch.from_numpy(array)

    def free(self):
        if self.ptr is not None and self.ptr.value:
            _check(load().ft_moe_host_unregister(self.ptr), "ft_moe_host_unregister")
            self.ptr = None
            self.tensor = None


def _ptr(t) -> int:
    """Device or host address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(s) -> int:
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


class FtMoe:
    """Handle of one stack of expert-cached MoE layers.  Methods mirror the C entry points."""

    def __init__(self, cfg: Config):
        self._lib = load()
        self.cfg = cfg
        self.E, self.k, self.Ns = cfg.n_experts, cfg.top_k, cfg.slots_per_layer
        self.L, self.global_pool = cfg.n_layers, bool(cfg.global_pool)
        self.expert_bytes = ft_moe_expert_bytes(cfg)
        self._h = C.c_void_p()
        _check(self._lib.ft_moe_create(C.byref(cfg), C.byref(self._h)), "ft_moe_create")

    def destroy(self):
        if self._h is not None and self._h.value:
            _check(self._lib.ft_moe_destroy(self._h), "ft_moe_destroy")
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- the hot path -------------------------------------------------------------
    def route(self, layer, logits_dev, T, stream=None):
        _check(self._lib.ft_moe_route(self._h, layer, _ptr(logits_dev), T, _stream(stream)), "ft_moe_route")

    def plan(self, layer, stream=None, want=True):
        """Runs the plan kernel; with ``want`` returns the host-visible plan as a dict."""
        if not want:
            _check(self._lib.ft_moe_plan(self._h, layer, None, _stream(stream)), "ft_moe_plan")
            return None
        E = self.E
        arrs = {n: np.full(E, -9, dtype=np.int32) for n in
                ("hit", "miss", "fill", "zc", "fill_order", "fill_slot", "fill_evicted", "loc")}
        out = PlanOut()
        for n, a in arrs.items():
            setattr(out, n, a.ctypes.data)
        _check(self._lib.ft_moe_plan(self._h, layer, C.byref(out), _stream(stream)), "ft_moe_plan")
        res = {"step": int(out.step), "n_routed": out.n_routed}
        for n, cnt in (("hit", out.n_hit), ("miss", out.n_miss), ("fill", out.n_fill), ("zc", out.n_zc),
                       ("fill_order", out.n_fill), ("fill_slot", out.n_fill), ("fill_evicted", out.n_fill)):
            res[n] = arrs[n][:cnt].tolist()
        res["loc"] = arrs["loc"]
        return res

    def fill(self, layer, copy_stream=None):
        _check(self._lib.ft_moe_fill(self._h, layer, _stream(copy_stream)), "ft_moe_fill")

    def prefetch_layer(self, layer, stream=None, copy_stream=None):
        _check(self._lib.ft_moe_prefetch_layer(self._h, layer, _stream(stream), _stream(copy_stream)),
               "ft_moe_prefetch_layer")

    def forward(self, layer, x_dev, y_dev, stream=None):
        _check(self._lib.ft_moe_forward(self._h, layer, _ptr(x_dev), _ptr(y_dev), _stream(stream)), "ft_moe_forward")

    def layer(self, layer, logits_dev, x_dev, y_dev, T, stream=None):
        _check(self._lib.ft_moe_layer(self._h, layer, _ptr(logits_dev), _ptr(x_dev), _ptr(y_dev), T,
                                      _stream(stream)), "ft_moe_layer")

    def layer_host(self, layer, logits_host, x_host, y_host, T, stream=None):
        _check(self._lib.ft_moe_layer_host(self._h, layer, _ptr(logits_host), _ptr(x_host), _ptr(y_host), T,
                                           _stream(stream)), "ft_moe_layer_host")

    # ---- calibration and introspection ----------------------------------------------
    def calibrate(self):
        out = (C.c_uint32 * 4)()
        _check(self._lib.ft_moe_calibrate(self._h, out), "ft_moe_calibrate")
        return {"fill_MBps": out[0], "zc_MBps": out[1], "zc_residual_MBps": out[2], "hbm_MBps": out[3]}

    def get_routing(self, layer, T):
        P, E = T * self.k, self.E
        ids = np.zeros(P, dtype=np.int32)
        w = np.zeros(P, dtype=np.float32)
        count = np.zeros(E, dtype=np.int32)
        offset = np.zeros(E + 1, dtype=np.int32)
        perm = np.zeros(P, dtype=np.int32)
        inv = np.zeros(P, dtype=np.int32)
        _check(self._lib.ft_moe_get_routing(self._h, layer, _ptr(ids), _ptr(w), _ptr(count), _ptr(offset),
                                            _ptr(perm), _ptr(inv)), "ft_moe_get_routing")
        return ids.reshape(T, self.k), w.reshape(T, self.k), count, offset, perm, inv

    def get_slot_table(self, layer):
        """(slot_expert, slot_stamp, expert_slot of `layer`); with a global pool the first two cover the shared
        pool and hold flattened ids layer*E + expert."""
        n = self.Ns * self.L if self.global_pool else self.Ns
        se = np.zeros(max(n, 1), dtype=np.int32)
        ss = np.zeros(max(n, 1), dtype=np.int64)
        es = np.zeros(self.E, dtype=np.int32)
        _check(self._lib.ft_moe_get_slot_table(self._h, layer, _ptr(se), _ptr(ss), _ptr(es)), "ft_moe_get_slot_table")
        return se[:n], ss[:n], es

    def resize(self, slots_per_layer):
        _check(self._lib.ft_moe_resize(self._h, int(slots_per_layer)), "ft_moe_resize")
        self.Ns = int(slots_per_layer)
        self.cfg.slots_per_layer = int(slots_per_layer)

    def read_slot(self, layer, slot):
        buf = np.empty(self.expert_bytes, dtype=np.uint8)
        _check(self._lib.ft_moe_read_slot(self._h, layer, slot, _ptr(buf)), "ft_moe_read_slot")
        return buf

    def get_stats(self, layer):
        a = np.zeros(len(STAT_NAMES), dtype=np.uint64)
        _check(self._lib.ft_moe_get_stats(self._h, layer, _ptr(a), len(STAT_NAMES)), "ft_moe_get_stats")
        return dict(zip(STAT_NAMES, (int(v) for v in a)))

    def reset(self, layer=-1):
        _check(self._lib.ft_moe_reset(self._h, layer), "ft_moe_reset")

    def sync_status(self):
        return int(self._lib.ft_moe_sync_status(self._h))

    def last_fill(self):
        us, b = C.c_float(), C.c_uint64()
        _check(self._lib.ft_moe_last_fill(self._h, C.byref(us), C.byref(b)), "ft_moe_last_fill")
        return float(us.value), int(b.value)

    def timing_enable(self, on=True):
        _check(self._lib.ft_moe_timing_enable(self._h, 1 if on else 0), "ft_moe_timing_enable")

    def timing_read(self):
        """{kind: (total microseconds, timed launches)} since timing was enabled."""
        us = np.zeros(len(TIME_NAMES), dtype=np.float64)
        n = np.zeros(len(TIME_NAMES), dtype=np.uint64)
        _check(self._lib.ft_moe_timing_read(self._h, _ptr(us), _ptr(n), len(TIME_NAMES)), "ft_moe_timing_read")
        return {k: (float(a), int(b)) for k, a, b in zip(TIME_NAMES, us, n)}

    def cta_trace(self, n_ctas=148):
        """int64 [n_ctas, 4]: start clock, end clock, blocks, segments of the latest streaming-kernel launch."""
        a = np.zeros((n_ctas, 4), dtype=np.int64)
        _check(self._lib.ft_moe_get_cta_trace(self._h, _ptr(a), n_ctas), "ft_moe_get_cta_trace")
        return a

    def set_split_min_pairs(self, pairs):
        _check(self._lib.ft_moe_set_split_min_pairs(self._h, int(pairs)), "ft_moe_set_split_min_pairs")

    def set_launch_overlap(self, mode):
        _check(self._lib.ft_moe_set_launch_overlap(self._h, int(mode)), "ft_moe_set_launch_overlap")

    def debug_inject(self, withhold_mask, wait_polls):
        _check(self._lib.ft_moe_debug_inject(self._h, int(withhold_mask), int(wait_polls)), "ft_moe_debug_inject")

    def launch_count(self):
        n = C.c_uint64()
        _check(self._lib.ft_moe_launch_count(self._h, C.byref(n)), "ft_moe_launch_count")
        return int(n.value)
