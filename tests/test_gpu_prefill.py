"""GPU parity of the prefill path (grouped tcgen05 GEMM + gather / combine) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair

pytestmark = pytest.mark.gpu


def _zipf_logits(T, E, seed, step, alpha=1.1):
    b = W.zipf_bias(E, alpha, seed, 0)
    rng = np.random.default_rng(W.mix64(seed, 99, step))
    return (rng.standard_normal((T, E)) + b).astype(np.float32)


@pytest.mark.parametrize("wdtype", ["bf16", "int4", "mxfp4", "nvfp4", "mxfp4tc"])
@pytest.mark.parametrize("T,n_slots", [(300, 8), (1000, 6), (129, 3)])
def test_prefill_grouped_gemm_matches_oracle(T, n_slots, wdtype):
    """Experts with >= 32 tokens and a slot go through the tensor-core GEMMs (4-bit experts after their expansion to
    bf16 records in the scratch pool), the rest through the streaming kernels (slots or zero-copy); row tiles are
    ragged (token counts are Zipf-skewed)."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype)
    pr = Pair(shape, n_slots=n_slots, max_tokens=1000, seed=31, gemm_min_tokens=32)
    for step in range(2):
        logits = _zipf_logits(T, 8, 31, step)
        x = W.noise_x(T, 512, 31, step, 0)
        _, r = pr.step(0, logits, x, check_slots=(step == 0))
        if T >= 300:
            assert max(r.count) >= 128      # at least one expert spans more than one 128-row tile
    assert pr.moe.get_stats(0)["pairs_gemm"] > 0   # the tensor-core path was taken
    pr.close()


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4", "mxfp4tc"])
def test_prefill_4bit_wide_hidden_size(wdtype):
    """d=7168, I=2048 (the 4-bit decode configuration's layer shape), 8 experts, 256 tokens: K = 7168 in the gate/up
    GEMM, 56 column tiles in the down GEMM, weights from the bf16 scratch records."""
    shape = W.LayerShape(d=7168, inter=2048, n_experts=8, top_k=2, wdtype=wdtype)
    pr = Pair(shape, n_slots=8, max_tokens=256, n_layers=1, seed=35, gen_device="cuda", gemm_min_tokens=32)
    for step in range(2):
        pr.step(0, _zipf_logits(256, 8, 35, step), W.noise_x(256, 7168, 35, step, 0), check_slots=(step == 0))
    assert pr.moe.get_stats(0)["pairs_gemm"] > 0
    pr.close()


@pytest.mark.parametrize("wdtype", ["bf16", "mxfp4", "mxfp4tc"])
def test_prefill_then_decode_on_the_same_handle(wdtype):
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype)
    pr = Pair(shape, n_slots=8, max_tokens=512, seed=33, gemm_min_tokens=32)
    pr.step(0, _zipf_logits(512, 8, 33, 0), W.noise_x(512, 512, 33, 0, 0))
    for step in range(1, 4):
        _, r = pr.step(0, _zipf_logits(4, 8, 33, step), W.noise_x(4, 512, 33, step, 0), fused=(step == 2))
        assert r.plan.miss == []            # the prefill left every routed expert resident
    pr.close()


@pytest.mark.parametrize("wdtype", ["int4", "mxfp4", "nvfp4", "mxfp4tc"])
def test_prefill_4bit_after_resize(wdtype):
    """The bf16 scratch pool the GEMMs read 4-bit experts from holds one record per slot of a layer, so a resize to
    more slots must grow it (and rebind the weight tensor maps): 3 slots -> 8 slots -> 2 slots."""
    from oracle import ftmoe_oracle as O
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype=wdtype)
    pr = Pair(shape, n_slots=3, max_tokens=512, seed=37, gemm_min_tokens=32)
    step = 0
    for new_slots in (None, 8, 2):
        if new_slots is not None:
            pr.moe.resize(new_slots)
            ora = pr.oracles[0]
            step_now = ora.state.step
            ora.state = O.CacheState(8, new_slots)
            ora.state.step = step_now
            ora.slots = [None] * new_slots
        for _ in range(2):
            pr.step(0, _zipf_logits(400, 8, 37, step), W.noise_x(400, 512, 37, step, 0), check_slots=True)
            step += 1
    assert pr.moe.get_stats(0)["pairs_gemm"] > 0
    pr.close()


def test_prefill_qwen3_shape_one_layer():
    """d=2048, 128 experts, I=768, top-8, 64 slots, 1024 tokens, cold then warm."""
    shape = W.QWEN3_30B
    pr = Pair(shape, n_slots=64, max_tokens=1024, n_layers=1, seed=0, gen_device="cuda", gemm_min_tokens=32)
    for step in range(2):
        logits = W.prefill_logits(1, 1024, 128, 1.1, 0, step)[0]
        x = W.noise_x(1024, 2048, 0, step, 0)
        _, r = pr.step(0, logits, x, check_slots=(step == 0))
        if step == 0:
            assert len(r.plan.fill) == 64 and len(r.plan.zc) > 0
    pr.close()
