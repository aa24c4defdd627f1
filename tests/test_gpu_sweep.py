"""Cache-pressure sweep: routing, plans and slot tables stay bit-exact against the oracle at every point
(cache fraction x temporal locality x batch), cold start, Qwen3-30B-A3B layer shapes."""
import numpy as np
import pytest
import torch

from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import Pair

pytestmark = pytest.mark.gpu


def test_sweep_points_plan_parity_and_monotone_hit_rate():
    shape = W.QWEN3_30B
    L, steps = 2, 12
    pool = B.HostPool(L * shape.n_experts * shape.expert_bytes)
    W.fill_pool(pool.tensor, shape, L, 0, device="cuda", chunk=32)
    hit_rate = {}
    for batch in (1, 16, 64):
        for rho in (0.0, 0.5, 0.9):
            logits = W.ar1_logits(L, steps, batch, 128, rho=rho, alpha=1.1, seed=7)
            for frac in (0.10, 0.25, 0.50, 0.75, 1.00):
                n_slots = W.slots_for_fraction(frac, 128)
                fill_mode = B.FT_FILL_SM if (batch == 16) else B.FT_FILL_COPY_ENGINE
                pr = Pair(shape, n_slots=n_slots, max_tokens=64, n_layers=L, pool=pool, fill_mode=fill_mode)
                for t in range(steps):
                    for l in range(L):
                        x = W.noise_x(batch, 2048, 7, t, l)
                        # outputs are checked once per point (last step, first layer); plans at every step
                        pr.step(l, logits[t, l], x, check_y=(t == steps - 1 and l == 0 and frac in (0.10, 0.50)))
                st = pr.moe.get_stats(0)
                assert st["routed"] == st["hits"] + st["fills"] + st["zc"]
                hit_rate[(batch, rho, frac)] = st["hits"] / st["routed"]
                pr.close()
            rates = [hit_rate[(batch, rho, f)] for f in (0.10, 0.25, 0.50, 0.75, 1.00)]
            assert rates[-1] >= rates[0]
    assert W.slots_for_fraction(0.10, 128) == 13 and W.slots_for_fraction(0.75, 128) == 96
    pool.free()
