"""The shared (global) slot pool with one LRU clock over (layer, expert) ids, and runtime resizing."""
import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import bits, check_output

pytestmark = pytest.mark.gpu


class SharedPoolOracle:
    """The oracle's state machine applied to flattened ids l*E + e: one table, one clock for all layers."""

    def __init__(self, shape, L, total_slots, recs, cm):
        self.shape, self.L, self.cm = shape, L, cm
        self.state = O.CacheState(L * shape.n_experts, total_slots)
        self.recs = recs

    def step(self, l, logits, x_bits, compute_y):
        E, k = self.shape.n_experts, self.shape.top_k
        ids, w = O.route(logits, k)
        count, offset, perm, inv = O.permute(ids, E)
        flat = np.zeros(self.L * E, dtype=np.int32)
        flat[l * E:(l + 1) * E] = count
        p = O.plan(self.state, flat, self.cm)
        y = None
        if compute_y:
            get = lambda e: O.unpack_record(self.recs[l][e], self.shape.d, self.shape.inter, self.shape.wdtype)
            y = O.moe_layer(O.bf16_to_f64(x_bits), ids, w, get)
        return ids, w, count, offset, perm, inv, p, y


def _run(shape, L, slots_per_layer, steps, T, seed, fused_every=2):
    E, S = shape.n_experts, shape.expert_bytes
    pool = B.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, seed)
    cfg = B.make_config(hidden=shape.d, inter=shape.inter, n_experts=E, top_k=shape.top_k, n_layers=L,
                        slots_per_layer=slots_per_layer, max_tokens=T, host_pool_ptr=pool.ptr.value,
                        host_pool_bytes=pool.n_bytes, fill_mode=B.FT_FILL_SM, global_pool=1)
    moe = B.FtMoe(cfg)
    cm = O.CostModel(S, cfg.bw_fill_MBps, cfg.bw_zc_residual_MBps, cfg.bw_zc_MBps, cfg.bw_hbm_MBps,
                     cfg.reuse_credit, cfg.zc_tokens_per_pass, cfg.hbm_tokens_per_pass)
    recs = pool.tensor.view(L, E, S).numpy()
    ora = SharedPoolOracle(shape, L, L * slots_per_layer, recs, cm)
    dev = torch.device("cuda:0")
    cross_layer_evictions = 0
    for t in range(steps):
        for l in range(L):
            logits = W.normal_logits(T, E, seed + l, t)
            x = W.noise_x(T, shape.d, seed, t, l)
            ids, w, count, offset, perm, inv, p, y_ref = ora.step(l, logits, bits(x), compute_y=(t % 2 == 0))
            lg, xd = torch.from_numpy(logits).to(dev), x.to(dev)
            y = torch.empty_like(xd)
            moe.route(l, lg, T)
            plan = moe.plan(l)
            moe.fill(l, None)
            moe.forward(l, xd, y)
            assert moe.sync_status() == 0
            base = l * E
            assert plan["step"] == p.step
            assert plan["hit"] == [g - base for g in p.hit] and plan["miss"] == [g - base for g in p.miss]
            assert plan["fill_order"] == [g - base for g in p.fill_order] and plan["zc"] == [g - base for g in p.zc]
            assert plan["fill_slot"] == p.fill_slot and plan["fill_evicted"] == p.fill_evicted
            assert np.array_equal(plan["loc"], p.loc[base:base + E])
            cross_layer_evictions += sum(1 for g in p.fill_evicted if g >= 0 and g // E != l)
            se, ss, es = moe.get_slot_table(l)
            assert np.array_equal(se, ora.state.slot_expert) and np.array_equal(ss, ora.state.slot_stamp)
            assert np.array_equal(es, ora.state.expert_slot[base:base + E])
            for i, (g, s) in enumerate(zip(p.fill_order, p.fill_slot)):
                if i < 2:
                    assert np.array_equal(moe.read_slot(l, s), recs[l][g - base])
            if y_ref is not None:
                check_output(y, y_ref)
    moe.destroy()
    pool.free()
    return cross_layer_evictions


@pytest.mark.parametrize("fill_mode", [B.FT_FILL_COPY_ENGINE, B.FT_FILL_SM])
def test_full_layer_prefetch_ahead_of_routing(fill_mode):
    """Double-buffered prefill: while layer l is evaluated the whole expert set of layer l+1 is admitted into the
    shared pool (its routing still unknown); the layer's own plan then finds only hits, the victims are the least
    recently used slots (layers already computed), and the outputs are unchanged."""
    shape = W.LayerShape(d=256, inter=64, n_experts=8, top_k=2)
    L, E, S, T = 4, 8, shape.expert_bytes, 12
    pool = B.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, 61)
    cfg = B.make_config(hidden=shape.d, inter=shape.inter, n_experts=E, top_k=2, n_layers=L, slots_per_layer=5,
                        max_tokens=T, host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                        fill_mode=fill_mode, global_pool=1)          # 20 shared slots >= two layers of 8
    moe = B.FtMoe(cfg)
    cm = O.CostModel(S, cfg.bw_fill_MBps, cfg.bw_zc_residual_MBps, cfg.bw_zc_MBps, cfg.bw_hbm_MBps,
                     cfg.reuse_credit, cfg.zc_tokens_per_pass, cfg.hbm_tokens_per_pass)
    recs = pool.tensor.view(L, E, S).numpy()
    ora = SharedPoolOracle(shape, L, 20, recs, cm)
    dev = torch.device("cuda:0")

    def prefetch(l):
        flat = np.zeros(L * E, dtype=np.int32)
        flat[l * E:(l + 1) * E] = 1                       # every expert of the layer "routed" once
        p = O.plan(ora.state, flat, cm)
        moe.prefetch_layer(l)
        return p

    for t in range(3):
        p0 = prefetch(0)
        assert t > 0 or len(p0.fill) == E
        for l in range(L):
            logits = W.normal_logits(T, E, 61 + l, t)
            x = W.noise_x(T, shape.d, 61, t, l)
            ids, w, count, offset, perm, inv, p, y_ref = ora.step(l, logits, bits(x), compute_y=True)
            assert p.miss == []                           # everything was brought in ahead of the routing
            lg, xd = torch.from_numpy(logits).to(dev), x.to(dev)
            y = torch.empty_like(xd)
            moe.route(l, lg, T)
            plan = moe.plan(l)
            moe.fill(l, None)
            if l + 1 < L:
                pn = prefetch(l + 1)                      # loads while layer l is evaluated
                assert all(g < 0 or g // E != l for g in pn.fill_evicted)     # never the layer in use
            moe.forward(l, xd, y)
            assert moe.sync_status() == 0
            assert plan["miss"] == [] and plan["hit"] == [g - l * E for g in p.hit]
            se, ss, es = moe.get_slot_table(l)
            assert np.array_equal(se, ora.state.slot_expert) and np.array_equal(ss, ora.state.slot_stamp)
            check_output(y, y_ref)
            for s_ in range(20):
                g = int(ora.state.slot_expert[s_])
                if g >= 0 and g // E == min(l + 1, L - 1):
                    assert np.array_equal(moe.read_slot(0, s_), recs[g // E][g % E])
        st = moe.get_stats(1)
        assert st["steps"] == t + 1                       # a prefetch is not a step of the layer
    # a pool that cannot hold two full layers refuses: the caller falls back to on-demand fills
    moe.resize(3)
    with pytest.raises(B.FtMoeError) as ei:
        moe.prefetch_layer(0)
    assert ei.value.code == B.FT_ERR_UNSUPPORTED
    moe.destroy()
    pool.free()


def test_shared_pool_small_table_paths():
    """3 layers sharing 9 slots: layers evict each other's experts by the common clock."""
    ev = _run(W.LayerShape(d=256, inter=64, n_experts=8, top_k=2), L=3, slots_per_layer=3, steps=6, T=4, seed=51)
    assert ev > 0


def test_shared_pool_large_table_block_wide_selection():
    """8 layers x 40 slots = 320 shared slots (more than the single-warp selection handles)."""
    ev = _run(W.LayerShape(d=256, inter=64, n_experts=64, top_k=4), L=8, slots_per_layer=40, steps=5, T=6, seed=52)
    assert ev >= 0


def test_resize_rebuilds_an_empty_cache_and_keeps_the_clock():
    shape = W.TINY
    S = shape.expert_bytes
    pool = B.HostPool(shape.n_experts * S)
    W.fill_pool(pool.tensor, shape, 1, 0)
    cfg = B.make_config(hidden=256, inter=128, n_experts=8, top_k=2, slots_per_layer=6, max_tokens=8,
                        host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes)
    moe = B.FtMoe(cfg)
    cm = O.CostModel(S, cfg.bw_fill_MBps, cfg.bw_zc_residual_MBps, cfg.bw_zc_MBps, cfg.bw_hbm_MBps)
    recs = pool.tensor.view(8, S).numpy()
    ora = O.OracleLayer(256, 128, 8, 2, 6, "bf16", recs, cm)
    dev = torch.device("cuda:0")

    def one(step):
        logits, x = W.normal_logits(8, 8, 0, step), W.noise_x(8, 256, 0, step, 0)
        r = ora.step(logits, bits(x))
        y = torch.empty((8, 256), dtype=torch.bfloat16, device=dev)
        moe.route(0, torch.from_numpy(logits).to(dev), 8)
        plan = moe.plan(0)
        moe.fill(0, None)
        moe.forward(0, x.to(dev), y)
        assert plan["step"] == r.plan.step and plan["hit"] == r.plan.hit and plan["fill_order"] == r.plan.fill_order
        assert plan["fill_slot"] == r.plan.fill_slot and plan["zc"] == r.plan.zc
        se, ss, es = moe.get_slot_table(0)
        assert np.array_equal(se, ora.state.slot_expert) and np.array_equal(ss, ora.state.slot_stamp)
        check_output(y, r.y)

    one(0)
    one(1)
    for new_slots in (2, 8, 0):
        moe.resize(new_slots)
        step_now = ora.state.step
        ora.state = O.CacheState(8, new_slots)
        ora.state.step = step_now
        ora.slots = [None] * new_slots
        one(step_now)
        one(step_now + 1)
    assert moe.get_stats(0)["steps"] == 8
    moe.destroy()
    pool.free()
