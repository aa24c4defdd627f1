"""Launch-overlap modes of the streaming kernel, batched forward calls over already planned layers, handles of
different shapes side by side: the results are those of the plain path (and of the oracle)."""
import numpy as np
import pytest
import torch

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair, bits, check_output

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wdtype", ["bf16", "mxfp4tc"])
@pytest.mark.parametrize("T", [3, 8, 21])
def test_forward_calls_of_planned_layers_back_to_back_in_every_overlap_mode(T, wdtype):
    """(For the tensor-core MXFP4 path mode 2 lets a call's activation slicing and gate/up kernel start while the call
    before is still in its down kernel; completion counts order what the calls share.)"""
    shape = W.LayerShape(d=1024, inter=256, n_experts=16, top_k=4, wdtype=wdtype)
    L = 4
    pr = Pair(shape, n_slots=8, max_tokens=32, n_layers=L, seed=13, fill_mode=B.FT_FILL_SM)
    dev = pr.dev
    for step in range(3):
        for mode in (0, 1, 2):
            pr.moe.set_launch_overlap(mode)
            logits = [W.normal_logits(T, 16, 13 + l, 10 * step + mode) for l in range(L)]
            xs = [W.noise_x(T, 1024, 13, 10 * step + mode, l) for l in range(L)]
            refs = [pr.oracles[l].step(logits[l], bits(xs[l])) for l in range(L)]
            xd = [x.to(dev) for x in xs]
            ys = [torch.full_like(x, float("nan")) for x in xd]
            for l in range(L):                      # route, plan and fill every layer first ...
                pr.moe.route(l, torch.from_numpy(logits[l]).to(dev), T)
                pr.moe.plan(l, want=False)
                pr.moe.fill(l, None)
            for l in range(L):                      # ... then the expert FFNs back to back
                pr.moe.forward(l, xd[l], ys[l])
            assert pr.moe.sync_status() == 0
            for l in range(L):
                ids, w, count, offset, perm, inv = pr.moe.get_routing(l, T)    # every layer keeps its own arrays
                assert np.array_equal(ids, refs[l].ids) and np.array_equal(perm, refs[l].perm)
                se, ss, es = pr.moe.get_slot_table(l)
                assert np.array_equal(se, pr.oracles[l].state.slot_expert)
                check_output(ys[l], refs[l].y)
    pr.moe.set_launch_overlap(0)
    pr.close()


def test_two_handles_of_different_width_interleaved():
    """Kernel attributes (shared-memory limits) belong to the function, not the handle: a narrow handle created
    after a wide one must not break the wide one's launches."""
    wide = Pair(W.LayerShape(d=2048, inter=128, n_experts=8, top_k=2), n_slots=4, max_tokens=8, seed=1)
    narrow = Pair(W.LayerShape(d=256, inter=64, n_experts=8, top_k=2), n_slots=4, max_tokens=8, seed=2)
    q4 = Pair(W.LayerShape(d=1024, inter=128, n_experts=8, top_k=2, wdtype="int4"), n_slots=4, max_tokens=8, seed=3)
    for step in range(3):
        wide.step(0, W.normal_logits(8, 8, 1, step), W.noise_x(8, 2048, 1, step, 0))
        narrow.step(0, W.normal_logits(8, 8, 2, step), W.noise_x(8, 256, 2, step, 0))
        q4.step(0, W.normal_logits(5, 8, 3, step), W.noise_x(5, 1024, 3, step, 0))
    narrow.moe.resize(2)
    wide.step(0, W.normal_logits(8, 8, 1, 9), W.noise_x(8, 2048, 1, 9, 0))
    q4.close()
    narrow.close()
    wide.close()


def test_misaligned_activations_are_refused_not_faulted():
    pr = Pair(W.TINY, n_slots=4, max_tokens=8)
    lg = torch.from_numpy(W.normal_logits(8, 8, 0, 0)).cuda()
    flat = torch.zeros(8 * 256 + 8, dtype=torch.bfloat16, device="cuda")
    odd = flat[1:1 + 8 * 256].view(8, 256)          # starts 2 bytes past a 16-byte boundary
    good = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    pr.moe.route(0, lg, 8)
    pr.moe.plan(0, want=False)
    pr.moe.fill(0, None)
    with pytest.raises(B.FtMoeError) as ei:
        pr.moe.forward(0, odd, good)
    assert ei.value.code == B.FT_ERR_INVALID_ARG
    assert pr.moe.sync_status() == 0
    pr.close()
