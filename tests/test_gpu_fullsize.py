"""Parity at the benchmark's full sizes and in the launch configuration bench.py times (device-driven fills,
split launches, CUDA-graph replay of a whole 48-layer step): plans of every layer at every step, outputs of
sampled layers / sampled tokens against the oracle."""
import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W
from tests.helpers import bits, check_output

pytestmark = pytest.mark.gpu


def _make(shape, L, n_slots, max_tokens, pool, **kw):
    cfg = B.make_config(hidden=shape.d, inter=shape.inter, n_experts=shape.n_experts, top_k=shape.top_k, n_layers=L,
                        slots_per_layer=n_slots, max_tokens=max_tokens, host_pool_ptr=pool.ptr.value,
                        host_pool_bytes=pool.n_bytes, fill_mode=B.FT_FILL_SM, **kw)
    moe = B.FtMoe(cfg)
    cm = O.CostModel(shape.expert_bytes, cfg.bw_fill_MBps, cfg.bw_zc_residual_MBps, cfg.bw_zc_MBps, cfg.bw_hbm_MBps,
                     cfg.reuse_credit, cfg.zc_tokens_per_pass, cfg.hbm_tokens_per_pass)
    return moe, cm


def test_decode_config1_full_stack_graph_replay():
    """48 layers x 128 experts (54 GiB pinned pool, 27 GiB of slots), batch 8, the step replayed as one CUDA graph."""
    shape = W.QWEN3_30B
    L, E, k, d, Bt, steps = 48, 128, 8, 2048, 8, 4
    S = shape.expert_bytes
    dev = torch.device("cuda:0")
    pool = B.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, 0, device=dev, chunk=32)
    moe, cm = _make(shape, L, 64, 8, pool)
    recs = pool.tensor.view(L, E, S).numpy()
    oracles = [O.OracleLayer(d, shape.inter, E, k, 64, "bf16", recs[l], cm) for l in range(L)]
    logits = W.ar1_logits(L, steps, Bt, E, 0.8, 1.1, 0)
    # step 0 routes the 64 pairs of every layer to 64 different experts, so all 64 slots are taken at once and
    # the following steps have to evict
    for l in range(L):
        z = np.full((Bt, E), -20.0, dtype=np.float32)
        for t in range(Bt):
            z[t, (5 * l + 8 * t + np.arange(8)) % E] = np.linspace(2.0, 1.0, 8)
        logits[0, l] = z
    lg_all = torch.from_numpy(logits).to(dev)
    s_lg = torch.empty((L, Bt, E), dtype=torch.float32, device=dev)
    s_noise = torch.empty((L, Bt, d), dtype=torch.bfloat16, device=dev)
    xbuf = torch.empty((L, Bt, d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, Bt, d), dtype=torch.bfloat16, device=dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cs = torch.cuda.current_stream()
        for l in range(L):
            if l == 0:
                xbuf[0].copy_(s_noise[0])
            else:
                torch.add(s_noise[l], ybuf[l - 1], out=xbuf[l])
            moe.layer(l, s_lg[l], xbuf[l], ybuf[l], Bt, cs)
    for t in range(steps):
        noise = torch.stack([W.noise_x(Bt, d, 0, t, l) for l in range(L)]).to(dev)
        s_lg.copy_(lg_all[t])
        s_noise.copy_(noise)
        g.replay()
        torch.cuda.synchronize()
        assert moe.sync_status() == 0
        x_host = xbuf.cpu()
        for l in range(L):
            check = l in (0, 24, 47)
            r = oracles[l].step(logits[t, l], bits(x_host[l]), compute_y=check)
            se, ss, es = moe.get_slot_table(l)          # the plan of every layer, through its effect on the tables
            assert np.array_equal(se, oracles[l].state.slot_expert), (t, l)
            assert np.array_equal(ss, oracles[l].state.slot_stamp), (t, l)
            assert np.array_equal(es, oracles[l].state.expert_slot), (t, l)
            if check:
                check_output(ybuf[l], r.y)
        st = moe.get_stats(17)
        assert st["steps"] == t + 1 and st["routed"] == st["hits"] + st["fills"] + st["zc"]
    assert sum(moe.get_stats(l)["evictions"] for l in range(L)) > L      # the LRU was exercised at full size
    moe.destroy()
    pool.free()


def test_prefill_config2_full_token_count_sampled_outputs():
    """4096 tokens, 128 experts, 64 slots, cold then warm: every routing / plan array, outputs of sampled tokens."""
    shape = W.QWEN3_30B
    E, k, d, T = 128, 8, 2048, 4096
    S = shape.expert_bytes
    dev = torch.device("cuda:0")
    pool = B.HostPool(E * S)
    W.fill_pool(pool.tensor, shape, 1, 0, device=dev, chunk=32)
    moe, cm = _make(shape, 1, 64, T, pool, gemm_min_tokens=32)
    ora = O.OracleLayer(d, shape.inter, E, k, 64, "bf16", pool.tensor.view(E, S).numpy(), cm)
    rng = np.random.default_rng(0)
    for step in range(2):
        logits = W.prefill_logits(1, T, E, 1.1, 0, step)[0]
        x = W.noise_x(T, d, 0, step, 0)
        r = ora.step(logits, None, compute_y=False)
        lg, xd = torch.from_numpy(logits).to(dev), x.to(dev)
        y = torch.empty_like(xd)
        moe.route(0, lg, T)
        plan = moe.plan(0)
        moe.fill(0, None)
        moe.forward(0, xd, y)
        assert moe.sync_status() == 0
        ids, w, count, offset, perm, inv = moe.get_routing(0, T)
        assert np.array_equal(ids, r.ids) and np.abs(w - r.w).max() <= 1e-6
        assert np.array_equal(count, r.count) and np.array_equal(offset, r.offset)
        assert np.array_equal(perm, r.perm) and np.array_equal(inv, r.inv)
        p = r.plan
        assert plan["hit"] == p.hit and plan["fill_order"] == p.fill_order and plan["fill_slot"] == p.fill_slot
        assert plan["zc"] == p.zc and plan["fill_evicted"] == p.fill_evicted and np.array_equal(plan["loc"], p.loc)
        if step == 0:
            assert len(p.fill) == 64 and len(p.zc) > 0
        else:
            assert len(p.hit) == 64 and p.fill == []
        sample = np.sort(rng.choice(T, size=96, replace=False))
        y_ref = O.moe_layer(O.bf16_to_f64(bits(x)[sample]), r.ids[sample], r.w[sample], ora.get_expert)
        check_output(y[torch.from_numpy(sample).to(dev)], y_ref)
    moe.destroy()
    pool.free()
