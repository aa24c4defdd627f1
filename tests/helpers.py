"""Shared harness of the GPU parity tests: one CUDA layer stack and the CPU oracle side by side."""
from __future__ import annotations

import numpy as np
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import binding as B
from paper_2608_16157_b200 import workload as W

REL_L2_TOL = 1e-2          # relative L2 error of y (bf16 / int4 weights)
MAX_ABS_TOL = 3e-2         # max-abs error of y as a fraction of max |y_ref|
GATE_W_TOL = 1e-6          # absolute error of the gate weights


def bits(x_bf16: torch.Tensor) -> np.ndarray:
    return x_bf16.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class Pair:
    """A CUDA handle and per-layer oracles over the same pinned pool."""

    def __init__(self, shape: W.LayerShape, n_slots: int, max_tokens: int, n_layers: int = 1, seed: int = 0,
                 fill_mode: int = B.FT_FILL_COPY_ENGINE, gen_device="cpu", pool=None, **cost):
        self.shape, self.n_slots, self.L = shape, n_slots, n_layers
        S = shape.expert_bytes
        self.S = S
        self.owns_pool = pool is None
        if pool is None:
            pool = B.HostPool(n_layers * shape.n_experts * S)
            W.fill_pool(pool.tensor, shape, n_layers, seed, device=gen_device)
        self.pool = pool
        self.shared = None
        if shape.n_shared:
            self.shared = W.make_shared_records(shape, n_layers, seed, device=gen_device)
        wd = {"bf16": B.FT_W_BF16, "int4": B.FT_W_INT4_G128, "mxfp4": B.FT_W_MXFP4, "nvfp4": B.FT_W_NVFP4, "mxfp4tc": B.FT_W_MXFP4_TC}[shape.wdtype]
        self.cfg = B.make_config(hidden=shape.d, inter=shape.inter, n_experts=shape.n_experts,
                                 top_k=shape.top_k, n_layers=n_layers, slots_per_layer=n_slots,
                                 max_tokens=max_tokens, host_pool_ptr=self.pool.ptr.value,
                                 host_pool_bytes=self.pool.n_bytes, wdtype=wd, n_shared=shape.n_shared,
                                 shared_ptr=None if self.shared is None else self.shared.data_ptr(),
                                 fill_mode=fill_mode, **cost)
        self.moe = B.FtMoe(self.cfg)
        c = self.cfg
        self.cm = O.CostModel(S, c.bw_fill_MBps, c.bw_zc_residual_MBps, c.bw_zc_MBps, c.bw_hbm_MBps,
                              c.reuse_credit, c.zc_tokens_per_pass, c.hbm_tokens_per_pass)
        recs = self.pool.tensor.view(n_layers, shape.n_experts, S).numpy()
        self.oracles = [
            O.OracleLayer(shape.d, shape.inter, shape.n_experts, shape.top_k, n_slots, shape.wdtype, recs[l],
                          self.cm, shared_records=() if self.shared is None else [self.shared[l].numpy()])
            for l in range(n_layers)]
        self.dev = torch.device("cuda:0")

    def close(self):
        self.moe.destroy()
        if self.owns_pool:
            self.pool.free()

    def step(self, layer: int, logits: np.ndarray, x: torch.Tensor, check_y: bool = True,
             check_slots: bool = False, fused: bool = False):
        """Runs one (layer, step) on both sides and asserts parity.  Returns (gpu y, oracle result)."""
        T = logits.shape[0]
        ora = self.oracles[layer]
        r = ora.step(logits, bits(x) if T else None, compute_y=check_y)
        lg = torch.from_numpy(np.ascontiguousarray(logits)).to(self.dev)
        xd = x.to(self.dev)
        y = torch.full_like(xd, float("nan"))
        if fused:
            self.moe.layer(layer, lg, xd, y, T)
            plan = None
        else:
            self.moe.route(layer, lg, T)
            plan = self.moe.plan(layer)
            self.moe.fill(layer, None)
            self.moe.forward(layer, xd, y)
        assert self.moe.sync_status() == 0
        if T == 0:
            return y, r
        ids, w, count, offset, perm, inv = self.moe.get_routing(layer, T)
        assert np.array_equal(ids, r.ids)
        assert np.abs(w - r.w).max() <= GATE_W_TOL
        assert np.array_equal(count, r.count) and np.array_equal(offset, r.offset)
        assert np.array_equal(perm, r.perm) and np.array_equal(inv, r.inv)
        p = r.plan
        if plan is not None:
            assert plan["step"] == p.step
            assert plan["n_routed"] == len(p.routed)
            assert plan["hit"] == p.hit and plan["miss"] == p.miss
            assert plan["fill"] == p.fill and plan["zc"] == p.zc
            assert plan["fill_order"] == p.fill_order and plan["fill_slot"] == p.fill_slot
            assert plan["fill_evicted"] == p.fill_evicted
            assert np.array_equal(plan["loc"], p.loc)
        se, ss, es = self.moe.get_slot_table(layer)
        assert np.array_equal(se, ora.state.slot_expert)
        assert np.array_equal(ss, ora.state.slot_stamp)
        assert np.array_equal(es, ora.state.expert_slot)
        if check_slots:
            recs = self.pool.tensor.view(self.L, self.shape.n_experts, self.S).numpy()[layer]
            for s, e in enumerate(ora.slots):
                if e is not None:
                    assert np.array_equal(self.moe.read_slot(layer, s), recs[e]), (s, e)
        if check_y:
            check_output(y, r.y)
        return y, r


def check_output(y_gpu: torch.Tensor, y_ref: np.ndarray):
    yf = y_gpu.float().cpu().double().numpy()
    assert np.all(np.isfinite(yf))
    den = np.linalg.norm(y_ref)
    rel = np.linalg.norm(yf - y_ref) / (den if den > 0 else 1.0)
    assert rel <= REL_L2_TOL, rel
    assert np.abs(yf - y_ref).max() <= MAX_ABS_TOL * max(np.abs(y_ref).max(), 1e-30)
