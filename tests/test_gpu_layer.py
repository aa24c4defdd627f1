"""GPU parity of the whole layer path against the CPU oracle, through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair, check_output

pytestmark = pytest.mark.gpu

LAPTOP = dict(bw_fill=11800, bw_zc_residual=35700, bw_zc=11800)     # Table 1, 4060-laptop row


@pytest.mark.parametrize("fill_mode", [B.FT_FILL_COPY_ENGINE, B.FT_FILL_SM])
@pytest.mark.parametrize("cost", [dict(), LAPTOP])
def test_tiny_config_all_steps_every_array(fill_mode, cost):
    """d=256, 8 experts, top-2, 4 slots, 4 steps x 8 tokens, cold start: H, F and Z all occur."""
    pr = Pair(W.TINY, n_slots=4, max_tokens=8, fill_mode=fill_mode, **cost)
    seen = set()
    for step in range(4):
        logits = W.normal_logits(8, 8, 0, step)
        x = W.noise_x(8, 256, 0, step, 0)
        _, r = pr.step(0, logits, x, check_slots=True)
        seen |= {"H"} if r.plan.hit else set()
        seen |= {"F"} if r.plan.fill else set()
        seen |= {"Z"} if r.plan.zc else set()
    assert seen == {"H", "F", "Z"}
    st = pr.moe.get_stats(0)
    assert st["steps"] == 4 and st["pairs"] == 4 * 16
    assert st["routed"] == st["hits"] + st["misses"] and st["misses"] == st["fills"] + st["zc"]
    pr.close()


@pytest.mark.parametrize("T", [1, 2, 3, 5, 8, 13, 37, 128, 129, 300])
def test_token_counts_span_tiles_and_both_route_paths(T):
    shape = W.LayerShape(d=512, inter=192, n_experts=16, top_k=4)
    pr = Pair(shape, n_slots=6, max_tokens=300, seed=T)
    rng = np.random.default_rng(T)
    for step in range(3):
        logits = (rng.standard_normal((T, 16)) * 2).astype(np.float32)
        x = W.noise_x(T, 512, T, step, 0)
        pr.step(0, logits, x, check_slots=(step == 2))
    pr.close()


def test_empty_call_is_a_noop_and_does_not_advance():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8)
    pr.step(0, W.normal_logits(8, 8, 0, 0), W.noise_x(8, 256, 0, 0, 0))
    pr.step(0, np.zeros((0, 8), dtype=np.float32), torch.zeros((0, 256), dtype=torch.bfloat16))
    _, r = pr.step(0, W.normal_logits(8, 8, 0, 1), W.noise_x(8, 256, 0, 1, 0))
    assert r.plan.step == 1
    pr.close()


def test_ties_signed_zero_and_nonfinite_logits():
    pr = Pair(W.TINY, n_slots=8, max_tokens=8)
    z = np.zeros((8, 8), dtype=np.float32)
    z[0] = [1, 2, 2, -0.0, 0.0, 2, 2, 1]
    z[1] = [0.0, -0.0, 0.0, -0.0, -1, -1, -1, -1]
    z[2] = 3.0
    z[3] = [5, 4, 3, 2, 1, 0, -1, -2]
    z[4] = z[3][::-1]
    z[5] = [-1e30, 1e30, 0, 0, 0, 0, 0, 0]
    z[6] = [1e-40, -1e-40, 0, 0, 0, 0, 0, 0]       # subnormals
    z[7] = [7, 7, 7, 7, 8, 8, 8, 8]
    x = W.noise_x(8, 256, 1, 0, 0)
    pr.step(0, z, x)
    bad = z.copy()
    bad[3, 2] = np.nan
    lg = torch.from_numpy(bad).cuda()
    pr.moe.route(0, lg, 8)
    assert pr.moe.sync_status() == B.FT_ERR_NONFINITE
    assert pr.moe.sync_status() == 0          # latched once
    bad[3, 2] = np.inf
    pr.moe.route(0, torch.from_numpy(bad).cuda(), 8)
    with pytest.raises(B.FtMoeError) as ei:
        pr.moe.plan(0)
    assert ei.value.code == B.FT_ERR_NONFINITE
    pr.close()


def test_results_do_not_depend_on_residency():
    """All-zero-copy, cold all-fill and warm all-hit runs give the same y (the host pool is the
    source of truth; the cache affects only performance)."""
    shape = W.LayerShape(d=512, inter=128, n_experts=8, top_k=2)
    logits = W.normal_logits(12, 8, 3, 0)
    x = W.noise_x(12, 512, 3, 0, 0)
    ys = {}
    for name, n_slots in (("zc", 0), ("full", 8)):
        pr = Pair(shape, n_slots=n_slots, max_tokens=12, seed=3)
        y, r = pr.step(0, logits, x)
        if name == "zc":
            assert r.plan.zc == r.plan.routed
            ys["zc"] = y.float().cpu()
        else:
            assert r.plan.fill == r.plan.routed
            ys["fill"] = y.float().cpu()
            y2, r2 = pr.step(0, logits, x)
            assert r2.plan.hit == r2.plan.routed
            ys["hit"] = y2.float().cpu()
        pr.close()
    scale = ys["hit"].abs().max()
    assert (ys["zc"] - ys["hit"]).abs().max() <= 1e-2 * scale
    assert torch.equal(ys["fill"], ys["hit"]) or (ys["fill"] - ys["hit"]).abs().max() <= 1e-2 * scale


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4"])
@pytest.mark.parametrize("n_shared", [0, 1])
@pytest.mark.parametrize("T", [1, 4, 7])
def test_int4_group_dequant_and_shared_expert(n_shared, T, wdtype):
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype, n_shared=n_shared)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=5)
    for step in range(3):
        pr.step(0, W.normal_logits(T, 8, 5, step), W.noise_x(T, 512, 5, step, 0), check_slots=True)
    pr.close()


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4", "mxfp4tc"])
@pytest.mark.parametrize("T", [9, 24, 40])
def test_int4_resident_experts_with_many_tokens_and_shared_expert(T, wdtype):
    """More than 8 tokens per slot-resident 4-bit expert (several weight passes) and the shared expert at T > 8."""
    shape = W.LayerShape(d=512, inter=256, n_experts=4, top_k=2, wdtype=wdtype, n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=40, seed=6)
    for step in range(3):
        _, r = pr.step(0, W.normal_logits(T, 4, 6, step), W.noise_x(T, 512, 6, step, 0))
        if step > 0:
            assert r.plan.zc == []                       # every routed expert is resident ...
            assert T < 24 or max(r.count) >= 9           # ... some with more than 8 tokens (at T = 9 the shared one)
    pr.close()


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4"])
@pytest.mark.parametrize("scale_log2", [-10, 10])
def test_int4_activation_range(scale_log2, wdtype):
    """The 4-bit kernels re-express activations and h per (token, group of 128) against the group's largest magnitude,
    so their range is that of fp32: inputs scaled by 2^-10 and 2^10 still meet the tolerance (the output scales
    roughly by the square)."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype, n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=8)
    for step in range(2):
        x = (W.noise_x(6, 512, 8, step, 0).float() * (2.0 ** scale_log2)).to(torch.bfloat16)
        pr.step(0, W.normal_logits(6, 8, 8, step), x)
    pr.close()


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4"])
def test_int4_activation_outlier_in_a_group(wdtype):
    """One element 1000 x larger than the rest of its quantisation group: the group's re-expressed form (15-bit fixed
    point, or two fp8 numbers, against the group's largest magnitude) keeps the result within the tolerance."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype, n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=12)
    for step in range(2):
        x = W.noise_x(6, 512, 12, step, 0).float()
        x[:, 5::128] *= 1000.0                       # one outlier per group of 128, every token
        x[2, :] = 0.0                                # and an all-zero token
        pr.step(0, W.normal_logits(6, 8, 12, step), x.to(torch.bfloat16))
    pr.close()


@pytest.mark.parametrize("n_shared", [0, 1])
@pytest.mark.parametrize("T", [1, 4, 8])
def test_mxfp4_tensor_core_images_decode(n_shared, T):
    """MXFP4 experts stored as operand images of the block-scaled tensor-core instruction: slot-resident, filled and
    zero-copy experts (4 slots for 8 experts) and the shared expert, 1 to 8 tokens."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype="mxfp4tc", n_shared=n_shared)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=5)
    for step in range(3):
        pr.step(0, W.normal_logits(T, 8, 5, step), W.noise_x(T, 512, 5, step, 0), check_slots=True)
    pr.close()


@pytest.mark.parametrize("scale_log2", [-10, 10])
def test_mxfp4_tensor_core_images_activation_range(scale_log2):
    """The bit-sliced activations carry a power-of-two scale per (token, term, block of 32), so inputs scaled by
    2^-10 and 2^10 meet the same tolerance."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype="mxfp4tc", n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=8)
    for step in range(2):
        x = (W.noise_x(6, 512, 8, step, 0).float() * (2.0 ** scale_log2)).to(torch.bfloat16)
        pr.step(0, W.normal_logits(6, 8, 8, step), x)
    pr.close()


def test_mxfp4_tensor_core_images_activation_outlier_in_a_block():
    """One element 1000 x larger than the rest of its block, every token, and an all-zero token."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype="mxfp4tc", n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=12)
    for step in range(2):
        x = W.noise_x(6, 512, 12, step, 0).float()
        x[:, 5::128] *= 1000.0
        x[2, :] = 0.0
        pr.step(0, W.normal_logits(6, 8, 12, step), x.to(torch.bfloat16))
    pr.close()


def test_mxfp4_tensor_core_images_many_steps_device_fills_and_wide_shape():
    """d=2048, I=768 (6 neuron groups, 16 stages per tile), 32 experts, top-4, 12 slots, device-driven fills, 12
    steps of 8 tokens: evictions, zero-copy experts and tiles split between CTAs."""
    shape = W.LayerShape(d=2048, inter=768, n_experts=32, top_k=4, wdtype="mxfp4tc")
    pr = Pair(shape, n_slots=12, max_tokens=8, seed=14, fill_mode=B.FT_FILL_SM, gen_device="cuda")
    ev = 0
    for step in range(12):
        _, r = pr.step(0, W.normal_logits(8, 32, 14, step), W.noise_x(8, 2048, 14, step, 0), fused=(step % 2 == 1))
        ev += sum(1 for e in r.plan.fill_evicted if e >= 0)
    assert ev > 0
    pr.close()


def test_mxfp4_tensor_core_images_many_tokens_then_few_on_one_handle():
    """A handle for up to 64 tokens: calls with 64, 20 and 3 tokens (one activation image per pass of 8 tokens of an
    expert, or the single image of a call with at most 8 tokens), slots, fills and zero-copy experts."""
    shape = W.LayerShape(d=1024, inter=256, n_experts=8, top_k=2, wdtype="mxfp4tc", n_shared=1)
    pr = Pair(shape, n_slots=5, max_tokens=64, seed=16, fill_mode=B.FT_FILL_SM)
    for step, T in enumerate((64, 20, 3, 64)):
        _, r = pr.step(0, W.normal_logits(T, 8, 16, step), W.noise_x(T, 1024, 16, step, 0), fused=(step == 1))
        if T == 64:
            assert max(r.count) > 8
    pr.close()


def test_nvfp4_small_and_subnormal_block_scales():
    """NVFP4 records written by definition whose gate and down block scales are the 15 smallest e4m3 numbers (exponent
    field 0 or 1: the subnormal bytes included) under a matrix scale of 2^9, so that an error in the decoding of
    those bytes would show in y."""
    from tests.test_oracle_ffn import _record_nvfp4_by_definition
    d, I, E = 512, 128, 4
    shape = W.LayerShape(d=d, inter=I, n_experts=E, top_k=2, wdtype="nvfp4")
    rng = np.random.default_rng(21)
    pool = B.HostPool(E * shape.expert_bytes)
    recs = pool.tensor.view(E, shape.expert_bytes).numpy()
    for e in range(E):
        cg, cu, cd = (rng.integers(0, 16, size=(I, d)) for _ in range(3))
        bg = rng.integers(1, 16, size=(I, d // 16))
        bu = rng.integers(0x2C, 0x3C, size=(I, d // 16))
        bd = rng.integers(1, 16, size=(I // 16, d))
        recs[e] = _record_nvfp4_by_definition(cg, cu, cd, bg, bu, bd, (512.0 * 0.05, 0.02, 512.0 * 0.05))
    pr = Pair(shape, n_slots=2, max_tokens=8, seed=21, pool=pool)
    for step in range(2):
        pr.step(0, W.normal_logits(5, E, 21, step), W.noise_x(5, d, 21, step, 0), check_slots=True)
    pr.close()
    pool.free()


def test_plan_and_permutation_are_deterministic():
    shape = W.LayerShape(d=256, inter=64, n_experts=32, top_k=4)
    runs = []
    for rep in range(3):
        pr = Pair(shape, n_slots=10, max_tokens=64, seed=9, **LAPTOP)
        out = []
        for step in range(5):
            logits = W.normal_logits(64, 32, 9, step)
            lg = torch.from_numpy(logits).cuda()
            pr.moe.route(0, lg, 64)
            plan = pr.moe.plan(0)
            pr.moe.fill(0, None)
            x = W.noise_x(64, 256, 9, step, 0).cuda()
            pr.moe.forward(0, x, torch.empty_like(x))
            ids, w, count, offset, perm, inv = pr.moe.get_routing(0, 64)
            out.append((ids.tobytes(), perm.tobytes(), inv.tobytes(), str(plan["fill_order"]), str(plan["fill_slot"]),
                        str(plan["zc"]), plan["loc"].tobytes()))
        runs.append(out)
        pr.close()
    assert runs[0] == runs[1] == runs[2]


def test_multi_layer_stack_keeps_per_layer_state():
    shape = W.LayerShape(d=256, inter=64, n_experts=16, top_k=2)
    pr = Pair(shape, n_slots=5, max_tokens=4, n_layers=3, seed=11)
    for step in range(4):
        for l in range(3):
            logits = W.normal_logits(4, 16, 11 + l, step)
            pr.step(l, logits, W.noise_x(4, 256, 11, step, l), check_slots=True, fused=(step % 2 == 1))
    pr.close()


def test_error_paths():
    lib = B.load()
    shape = W.TINY
    S = shape.expert_bytes
    # pageable pool -> FT_ERR_NOT_PINNED (there is no CPU fallback)
    pageable = torch.zeros(shape.n_experts * S, dtype=torch.uint8)
    cfg = B.make_config(hidden=256, inter=128, n_experts=8, top_k=2, slots_per_layer=4, max_tokens=8,
                        host_pool_ptr=pageable.data_ptr(), host_pool_bytes=pageable.numel())
    h = ctypes.c_void_p()
    assert lib.ft_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == B.FT_ERR_NOT_PINNED
    # pool too small
    pr = Pair(shape, n_slots=4, max_tokens=8)
    cfg2 = B.make_config(hidden=256, inter=128, n_experts=8, top_k=2, slots_per_layer=4, max_tokens=8,
                         host_pool_ptr=pr.pool.ptr.value, host_pool_bytes=S)
    assert lib.ft_moe_create(ctypes.byref(cfg2), ctypes.byref(h)) == B.FT_ERR_INVALID_ARG
    # call order
    lg = torch.from_numpy(W.normal_logits(8, 8, 0, 0)).cuda()
    x = W.noise_x(8, 256, 0, 0, 0).cuda()
    y = torch.empty_like(x)
    for call in (lambda: pr.moe.plan(0), lambda: pr.moe.fill(0, None), lambda: pr.moe.forward(0, x, y)):
        with pytest.raises(B.FtMoeError) as ei:
            call()
        assert ei.value.code == B.FT_ERR_STATE
    pr.moe.route(0, lg, 8)
    with pytest.raises(B.FtMoeError) as ei:
        pr.moe.forward(0, x, y)
    assert ei.value.code == B.FT_ERR_STATE
    with pytest.raises(B.FtMoeError) as ei:
        pr.moe.route(0, lg, 9)        # T > max_tokens
    assert ei.value.code == B.FT_ERR_INVALID_ARG
    with pytest.raises(B.FtMoeError):
        pr.moe.route(1, lg, 8)        # no such layer
    # the handle still works after the errors
    pr.moe.reset()
    pr.step(0, W.normal_logits(8, 8, 0, 0), W.noise_x(8, 256, 0, 0, 0))
    pr.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8)
    logits = W.normal_logits(8, 8, 0, 0)
    x = W.noise_x(8, 256, 0, 0, 0)
    y_dev, r = pr.step(0, logits, x)
    pr.moe.reset()
    y_host = torch.empty_like(x)
    pr.moe.layer_host(0, logits, x, y_host, 8)
    assert torch.equal(y_host, y_dev.cpu()) or (y_host.float() - y_dev.cpu().float()).abs().max() < 1e-3
    check_output(y_host, r.y)
    pr.close()


@pytest.mark.parametrize("batch", [1, 8])
def test_qwen3_shaped_decode_two_layers(batch):
    """d=2048, 128 experts, I=768, top-8, 64 slots per layer; AR(1) + Zipf logits; teacher-forced layers."""
    shape = W.QWEN3_30B
    L, steps = 2, 6
    pr = Pair(shape, n_slots=64, max_tokens=8, n_layers=L, seed=0, gen_device="cuda")
    logits = W.ar1_logits(L, steps, batch, 128, rho=0.8, alpha=1.1, seed=0)
    for t in range(steps):
        y_prev = None
        for l in range(L):
            n = W.noise_x(batch, 2048, 0, t, l)
            x = n if y_prev is None else (n.float() + y_prev.float().cpu()).to(torch.bfloat16)
            y_prev, _ = pr.step(l, logits[t, l], x, check_y=(t in (0, steps - 1)), check_slots=(t == 0 and l == 0))
    st = pr.moe.get_stats(0)
    assert st["hits"] > 0 and st["fills"] > 0
    pr.close()


@pytest.mark.parametrize("shape", [W.DSV3_INT4, W.DSV3_MXFP4, W.DSV3_NVFP4, W.DSV3_MXFP4TC],
                         ids=["int4", "mxfp4", "nvfp4", "mxfp4tc"])
def test_dsv3_shaped_int4_decode_one_layer(shape):
    """d=7168, 256 routed experts (int4 group 128, mxfp4 or nvfp4) + 1 shared expert, I=2048, top-8, 64 slots, batch 4."""
    steps = 3
    pr = Pair(shape, n_slots=64, max_tokens=8, n_layers=1, seed=0, gen_device="cuda")
    logits = W.ar1_logits(1, steps, 4, 256, rho=0.9, alpha=1.2, seed=0)
    for t in range(steps):
        x = W.noise_x(4, 7168, 0, t, 0)
        pr.step(0, logits[t, 0], x, check_y=(t != 1), check_slots=(t == 0), fused=(t == 2))
    pr.close()


def test_pool_pinned_in_place_with_host_register():
    """A pool in ordinary (here: anonymously mapped) memory, pinned afterwards with ft_moe_host_register."""
    import mmap
    shape = W.TINY
    S = shape.expert_bytes
    buf = mmap.mmap(-1, shape.n_experts * S)
    arr = np.frombuffer(buf, dtype=np.uint8)
    W.fill_pool(torch.from_numpy(arr), shape, 1, seed=0)
    pool = B.RegisteredPool(arr)
    pr = Pair(shape, n_slots=4, max_tokens=8, pool=pool)
    for step in range(2):
        pr.step(0, W.normal_logits(8, 8, 0, step), W.noise_x(8, 256, 0, step, 0), check_slots=True)
    pr.close()
    pool.free()
