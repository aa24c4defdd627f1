"""GPU edge cases of the layer path: extreme shapes, zero-copy-only handles, reset, calibration, timing."""
import numpy as np
import pytest
import torch

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair

pytestmark = pytest.mark.gpu


def test_max_experts_and_max_top_k():
    """1024 experts (one per plan thread, 32 logits per lane) and top-32."""
    shape = W.LayerShape(d=256, inter=64, n_experts=1024, top_k=32)
    pr = Pair(shape, n_slots=40, max_tokens=4, seed=41)
    rng = np.random.default_rng(41)
    for step in range(3):
        logits = rng.standard_normal((3, 1024)).astype(np.float32)
        pr.step(0, logits, W.noise_x(3, 256, 41, step, 0), check_slots=(step == 0))
    pr.close()


def test_256_experts_more_slots_than_experts_used():
    shape = W.LayerShape(d=256, inter=64, n_experts=256, top_k=8)
    pr = Pair(shape, n_slots=300, max_tokens=16, seed=42)
    for step in range(3):
        pr.step(0, W.normal_logits(16, 256, 42, step), W.noise_x(16, 256, 42, step, 0))
    pr.close()


@pytest.mark.parametrize("wdtype", ["bf16", "int4", "mxfp4", "nvfp4", "mxfp4tc"])
def test_zero_slots_everything_zero_copy_many_tokens(wdtype):
    """No cache at all: every expert is computed from the mapped host pool, more than 8 tokens per expert."""
    shape = W.LayerShape(d=512, inter=128, n_experts=4, top_k=2, wdtype=wdtype)
    pr = Pair(shape, n_slots=0, max_tokens=40, seed=43)
    for step in range(2):
        _, r = pr.step(0, W.normal_logits(40, 4, 43, step), W.noise_x(40, 512, 43, step, 0))
        assert r.plan.zc == r.plan.routed and max(r.count) > 8
    pr.close()


def test_reset_restores_a_cold_cache():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8)
    logits, x = W.normal_logits(8, 8, 0, 0), W.noise_x(8, 256, 0, 0, 0)
    _, r0 = pr.step(0, logits, x)
    pr.moe.reset(0)
    pr.oracles[0].state.reset()
    pr.oracles[0].slots = [None] * 4
    _, r1 = pr.step(0, logits, x)
    assert r1.plan.step == 0 and r1.plan.fill_order == r0.plan.fill_order and r1.plan.hit == []
    assert pr.moe.get_stats(0)["steps"] == 1
    pr.close()


def test_calibrate_and_timing_do_not_disturb_the_layer():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8)
    pr.step(0, W.normal_logits(8, 8, 0, 0), W.noise_x(8, 256, 0, 0, 0))
    cal = pr.moe.calibrate()
    assert all(v > 0 for v in cal.values())
    pr.moe.timing_enable(True)
    pr.step(0, W.normal_logits(8, 8, 0, 1), W.noise_x(8, 256, 0, 1, 0), check_slots=True)
    tim = pr.moe.timing_read()
    assert tim["route"][1] == 1 and tim["plan"][1] == 1 and tim["ffn_res"][1] >= 1 and tim["ffn_res"][0] > 0
    pr.moe.timing_enable(False)
    pr.step(0, W.normal_logits(8, 8, 0, 2), W.noise_x(8, 256, 0, 2, 0), fused=True)
    assert pr.moe.launch_count() > 0
    pr.close()


def test_split_launch_gives_the_same_output_as_one_launch():
    """Hits evaluated while the fills are in flight vs everything after the fills."""
    shape = W.LayerShape(d=512, inter=128, n_experts=16, top_k=4)
    outs = []
    for split in (0, 8):
        pr = Pair(shape, n_slots=8, max_tokens=16, seed=44, fill_mode=B.FT_FILL_SM, split_min_pairs=split)
        ys = []
        for step in range(4):
            y, _ = pr.step(0, W.normal_logits(16, 16, 44, step), W.noise_x(16, 512, 44, step, 0), fused=(step % 2 == 1))
            ys.append(y.float().cpu())
        outs.append(ys)
        pr.close()
    for a, b in zip(*outs):
        assert (a - b).abs().max() <= 1e-2 * b.abs().max()
