"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ftmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ft_moe_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build_mod.build()
    lib = ctypes.CDLL(path)
    declared = _declared_symbols()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(B.SYMBOLS) == declared


def test_config_struct_matches_header_size_and_expert_bytes():
    # 12 int32 + (ptr, size_t, ptr) + 4 uint32 + 6 int32 on LP64
    assert ctypes.sizeof(B.Config) == 12 * 4 + 3 * 8 + 10 * 4
    cfg = B.make_config(hidden=2048, inter=768, n_experts=128, top_k=8, slots_per_layer=64, max_tokens=8,
                        host_pool_ptr=None, host_pool_bytes=0)
    assert B.ft_moe_expert_bytes(cfg) == 9437184
    cfg = B.make_config(hidden=7168, inter=2048, n_experts=256, top_k=8, slots_per_layer=64, max_tokens=8,
                        host_pool_ptr=None, host_pool_bytes=0, wdtype=B.FT_W_INT4_G128)
    assert B.ft_moe_expert_bytes(cfg) == 22708224
    # the library's record sizes and the generator's agree for every weight format
    from paper_2608_16157_b200 import workload as W
    for wd, name in ((B.FT_W_MXFP4, "mxfp4"), (B.FT_W_MXFP4_TC, "mxfp4tc"), (B.FT_W_NVFP4, "nvfp4"), (B.FT_W_INT4_G128, "int4")):
        for d, inter in ((7168, 2048), (512, 256)):
            cfg = B.make_config(hidden=d, inter=inter, n_experts=8, top_k=2, slots_per_layer=4, max_tokens=8,
                                host_pool_ptr=None, host_pool_bytes=0, wdtype=wd)
            assert B.ft_moe_expert_bytes(cfg) == W.LayerShape(d, inter, 8, 2, name).expert_bytes
    cfg = B.make_config(hidden=100, inter=768, n_experts=128, top_k=8, slots_per_layer=64, max_tokens=8,
                        host_pool_ptr=None, host_pool_bytes=0)
    assert B.ft_moe_expert_bytes(cfg) == 0


def test_status_strings():
    assert B.status_string(0) == "ok"
    assert "pinned" in B.status_string(B.FT_ERR_NOT_PINNED)
    assert B.status_string(99) == "unknown status"


def test_create_rejects_bad_arguments_without_a_gpu_call():
    lib = B.load()
    h = ctypes.c_void_p()
    assert lib.ft_moe_create(None, ctypes.byref(h)) == B.FT_ERR_INVALID_ARG
    cfg = B.make_config(hidden=256, inter=128, n_experts=8, top_k=2, slots_per_layer=4, max_tokens=8,
                        host_pool_ptr=None, host_pool_bytes=0)
    cfg.struct_size = 7
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_INVALID_ARG
    cfg.struct_size = ctypes.sizeof(B.Config)
    cfg.top_k = 9
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_INVALID_ARG
    cfg.top_k = 2
    cfg.bw_fill_MBps = 0
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_INVALID_ARG
    cfg.bw_fill_MBps = 50000
    cfg.hidden = 300
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_UNSUPPORTED
    cfg.hidden = 256
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_INVALID_ARG   # null pool
    assert not h.value


def test_noalloc_entry_point_checks_its_arguments_before_any_device_work():
    """Size limits and pointer alignment are checked on the host: a view with an odd element offset is refused with
    FT_ERR_INVALID_ARG instead of faulting on the device (no GPU needed: nothing is launched)."""
    lib = B.load()
    base = 0x7f0000001000                    # never dereferenced
    f = lib.ft_moe_ffn_noalloc
    assert f(0, base + 2, 256, 128, base, base, 4, None) == B.FT_ERR_INVALID_ARG
    assert f(0, base, 256, 128, base + 6, base, 4, None) == B.FT_ERR_INVALID_ARG
    assert f(0, base, 256, 128, base, base + 8, 4, None) == B.FT_ERR_INVALID_ARG
    assert f(0, base, 256, 128, base, base, 0, None) == B.FT_ERR_INVALID_ARG
    assert f(0, base, 256, 128, base, base, B.NOALLOC_MAX_TOKENS + 1, None) == B.FT_ERR_INVALID_ARG
    assert f(0, None, 256, 128, base, base, 4, None) == B.FT_ERR_INVALID_ARG
    assert f(0, base, 300, 128, base, base, 4, None) == B.FT_ERR_UNSUPPORTED
