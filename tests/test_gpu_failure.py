"""The failure path of the bounded device-side waits, exercised without faulting or hanging anything: a test hook
makes one producer withhold a single copy, the consumer's wait (limited to a few thousand polls) runs out, the
kernel returns, the status word reports FT_ERR_TIMEOUT once, and after a reset the handle gives correct results."""
import numpy as np
import pytest
import torch

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair

pytestmark = pytest.mark.gpu

FT_DEBUG_WITHHOLD_FILL, FT_DEBUG_WITHHOLD_GEMM, FT_DEBUG_WITHHOLD_TC = 1, 4, 8


def _reset_both(pr):
    pr.moe.reset()
    for o in pr.oracles:
        o.state.reset()
        o.slots = [None] * len(o.slots)


def _run_expect_timeout(pr, mask, T, logits, x):
    pr.moe.debug_inject(mask, 4000)
    try:
        lg, xd = torch.from_numpy(logits).cuda(), x.cuda()
        y = torch.zeros_like(xd)
        pr.moe.route(0, lg, T)
        pr.moe.plan(0, want=False)
        pr.moe.fill(0, None)
        pr.moe.forward(0, xd, y)
        assert pr.moe.sync_status() == B.FT_ERR_TIMEOUT      # the kernel came back and said why
        assert pr.moe.sync_status() == 0                     # latched once
    finally:
        pr.moe.debug_inject(0, 0)


def test_fill_kernel_wait_runs_out_and_the_handle_recovers():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8, fill_mode=B.FT_FILL_SM)
    pr.step(0, W.normal_logits(8, 8, 0, 0), W.noise_x(8, 256, 0, 0, 0), check_slots=True)
    _reset_both(pr)                                          # cold cache: the next step has fills
    _run_expect_timeout(pr, FT_DEBUG_WITHHOLD_FILL, 8, W.normal_logits(8, 8, 0, 1), W.noise_x(8, 256, 0, 1, 0))
    _reset_both(pr)
    for step in range(2):
        pr.step(0, W.normal_logits(8, 8, 0, step), W.noise_x(8, 256, 0, step, 0), check_slots=True)
    pr.close()


def test_prefill_gemm_wait_runs_out_and_the_handle_recovers():
    shape = W.LayerShape(d=256, inter=256, n_experts=4, top_k=2)
    pr = Pair(shape, n_slots=4, max_tokens=128, seed=7, gemm_min_tokens=16)
    rng = np.random.default_rng(7)
    logits = (rng.standard_normal((128, 4)) * 2).astype(np.float32)
    x = W.noise_x(128, 256, 7, 0, 0)
    pr.step(0, logits, x)
    assert pr.moe.get_stats(0)["pairs_gemm"] > 0
    _run_expect_timeout(pr, FT_DEBUG_WITHHOLD_GEMM, 128, logits, x)
    _reset_both(pr)
    pr.step(0, logits, x)
    pr.close()


def test_tensor_core_decode_waits_run_out_and_the_handle_recovers():
    """FT_W_MXFP4_TC: one stage of the gate/up kernel's ring never arrives: its MMA issuers and epilogue give up, the
    down kernel gives up waiting for h, both kernels return, the status says so, and after a reset (which also clears
    the partial sums of the hand-over buffers) the handle is correct again."""
    shape = W.LayerShape(d=512, inter=256, n_experts=8, top_k=2, wdtype="mxfp4tc", n_shared=1)
    pr = Pair(shape, n_slots=4, max_tokens=8, seed=9)
    pr.step(0, W.normal_logits(6, 8, 9, 0), W.noise_x(6, 512, 9, 0, 0))
    _run_expect_timeout(pr, FT_DEBUG_WITHHOLD_TC, 6, W.normal_logits(6, 8, 9, 1), W.noise_x(6, 512, 9, 1, 0))
    _reset_both(pr)
    for step in range(2):
        pr.step(0, W.normal_logits(6, 8, 9, step), W.noise_x(6, 512, 9, step, 0), check_slots=True)
    pr.close()
