#!/usr/bin/env python
"""Decode throughput of the expert-cached MoE stack on B200 (one JSON line on stdout).

Workload (the Qwen3-30B-A3B-shaped decode configuration): 48 independent MoE layers, d=2048,
128 SwiGLU experts of intermediate 768, top-8, bf16 weights ~N(0,0.02) in a pinned host pool
(54 GiB), HBM cache of 64 slots per layer (50 %), router logits from an AR(1) chain (rho 0.8) plus a
Zipf-style bias (alpha 1.1), layer inputs x_l = bf16(noise_l + y_{l-1}).  A step is one decode step
of `--batch` tokens through all layers: route -> plan -> fill -> expert FFN -> combine per layer.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--batch 8]

`value` is whole-job tokens/s with inputs resident in HBM; `e2e` is the same through the
host-buffer entry point (logits and x copied host->device and y device->host every layer).
`roofline` is the resident-expert streaming kernel: algorithmic bytes = resident experts x record
bytes, duration from CUDA events on the launching stream, peak from MEASURED_PEAKS.json.
With N > 1 every rank runs an independent replica (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SEED = 0
RHO, ALPHA = 0.8, 1.1
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
# DRAM bytes (read + write) of one ffn_stream_kernel launch over its algorithmic bytes, from the ncu capture
# summarised in profiles/ (same kernel, batch 8, 24 resident experts per launch)
NCU_TRAFFIC_RATIO = 1.025
NCU_TRAFFIC_SOURCE = "profiles/ffn_stream_kernel_decode_qwen3_b8.md"


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, f"/tmp/ftmoe_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for ln in open(self.path):
                parts = [p.strip() for p in ln.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_sample_seconds(pool_np, shape, n_slots, cm_args, logits_step, x_bits_by_layer, layers):
    """Times the CPU oracle (as it stands) on `layers` layers of one decode step."""
    from oracle import ftmoe_oracle as O
    cm = O.CostModel(*cm_args)
    t0 = time.perf_counter()
    for l in layers:
        ora = O.OracleLayer(shape.d, shape.inter, shape.n_experts, shape.top_k, n_slots, shape.wdtype,
                            pool_np[l], cm)
        ora.step(logits_step[l], x_bits_by_layer[l])
    return time.perf_counter() - t0


def run_reference(args):
    """The reference arm of this tier is the CPU oracle, timed as it stands on the host cores."""
    import torch
    from paper_2608_16157_b200 import workload as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape = W.QWEN3_30B
    B = args.batch
    S = shape.expert_bytes
    n_layers_pool = 2                      # the sample never needs more than two layers of weights
    pool = torch.empty(n_layers_pool * shape.n_experts * S, dtype=torch.uint8)
    W.fill_pool(pool, shape, n_layers_pool, SEED)
    pool_np = pool.view(n_layers_pool, shape.n_experts, S).numpy()
    steps_total = args.steps + args.warmup
    logits = W.ar1_logits(n_layers_pool, steps_total, B, shape.n_experts, RHO, ALPHA, SEED)
    cm_args = (S, 50000, 0, 50000, 6000000, 1, 64, 128)
    from oracle import ftmoe_oracle as O
    cm = O.CostModel(*cm_args)
    ora = O.OracleLayer(shape.d, shape.inter, shape.n_experts, shape.top_k, 64, "bf16", pool_np[0], cm)
    # size the per-step sample (batch rows of one layer) so the whole run stays within ~2.5 minutes
    x0 = W.noise_x(B, shape.d, SEED, 0, 0).view(torch.int16).numpy().view(np.uint16)
    t0 = time.perf_counter()
    ora.step(logits[0, 0][:1], x0[:1])
    t_row = time.perf_counter() - t0
    rows = int(max(1, min(B, 150.0 / max(steps_total, 1) / max(t_row, 1e-6))))
    ora.state.reset()
    times = []
    for s in range(steps_total):
        x = W.noise_x(B, shape.d, SEED, s, 0).view(torch.int16).numpy().view(np.uint16)
        t0 = time.perf_counter()
        ora.step(logits[s, 0][:rows], x[:rows])
        dt = time.perf_counter() - t0
        if s >= args.warmup:
            times.append(dt)
    per_step = sum(times) / max(len(times), 1) * 48            # one layer timed, 48 in the stack
    value = rows / per_step
    cores = len(os.sched_getaffinity(0))
    sample = f"{rows} of {B} batch rows through 1 of 48 layers per step, time scaled x48"
    line = {"impl": "reference", "metric": "moe_decode_tok_per_s", "value": value, "unit": "tok/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": "decode Qwen3-30B-A3B-shaped MoE stack (config 1)", "batch": B,
                       "layers": 48, "hidden": shape.d, "experts": shape.n_experts, "inter": shape.inter,
                       "top_k": shape.top_k, "slots_per_layer": 64},
            "cpu_baseline": {"value": value, "unit": "tok/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    from paper_2608_16157_b200 import binding as Bd
    from paper_2608_16157_b200 import workload as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    dsv3 = args.workload in ("dsv3", "dsv3_mxfp4", "dsv3_nvfp4", "dsv3_mxfp4tc")
    mxfp4 = args.workload in ("dsv3_mxfp4", "dsv3_nvfp4", "dsv3_mxfp4tc")    # the floating-point 4-bit formats
    fp4_name = {"dsv3_nvfp4": "nvfp4", "dsv3_mxfp4tc": "mxfp4 (tensor-core operand images)"}.get(args.workload, "mxfp4")
    shape = {"dsv3": W.DSV3_INT4, "dsv3_mxfp4": W.DSV3_MXFP4, "dsv3_nvfp4": W.DSV3_NVFP4,
             "dsv3_mxfp4tc": W.DSV3_MXFP4TC}[args.workload] if dsv3 else W.QWEN3_30B
    RHO, ALPHA = (0.9, 1.2) if dsv3 else (0.8, 1.1)
    L = (4 if args.layers == 48 else args.layers) if dsv3 else args.layers
    E, k, d = shape.n_experts, shape.top_k, shape.d
    S = shape.expert_bytes
    Ns = 64 if dsv3 else W.slots_for_fraction(args.cache_frac, E)
    B = (4 if args.batch == 8 else args.batch) if dsv3 else args.batch
    Wn, K = args.warmup, args.steps
    t_setup = time.perf_counter()
    from paper_2608_16157_b200 import multirank as MR
    shm_name = None
    if world > 1 and MR.shm_has_room(L * E * S):
        # one copy of the host pool for all replicas of the node: rank 0 fills a /dev/shm file, every rank
        # maps it and pins it in place
        def _fill(arr):
            W.fill_pool(torch.from_numpy(arr), shape, L, SEED, device=dev, chunk=32)
        arr, shm_name = MR.open_shared_pool(L * E * S, f"{os.environ.get('MASTER_PORT', '0')}_{args.workload}", rank,
                                            dist.barrier, fill=_fill)
        pool = Bd.RegisteredPool(arr)
    else:
        pool = Bd.HostPool(L * E * S)
        W.fill_pool(pool.tensor, shape, L, SEED, device=dev, chunk=32)
    shared = W.make_shared_records(shape, L, SEED, device=dev) if shape.n_shared else None
    log(f"[rank {rank}] pool {L * E * S / 2**30:.1f} GiB pinned+filled in {time.perf_counter() - t_setup:.1f}s")

    fill_mode = Bd.FT_FILL_SM if args.fill == "sm" else Bd.FT_FILL_COPY_ENGINE

    def make(bw):
        cfg = Bd.make_config(hidden=d, inter=shape.inter, n_experts=E, top_k=k, n_layers=L, slots_per_layer=Ns,
                             max_tokens=max(B, 8), host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                             fill_mode=fill_mode, device=local,
                             wdtype={"int4": Bd.FT_W_INT4_G128, "mxfp4": Bd.FT_W_MXFP4, "nvfp4": Bd.FT_W_NVFP4, "mxfp4tc": Bd.FT_W_MXFP4_TC,
                                     "bf16": Bd.FT_W_BF16}[shape.wdtype],
                             n_shared=shape.n_shared, shared_ptr=None if shared is None else shared.data_ptr(),
                             global_pool=args.global_pool, **bw)
        return Bd.FtMoe(cfg)

    # bandwidth profiling at deployment, then frozen into the plan's cost model
    moe = make({})
    cal = moe.calibrate()
    moe.destroy()
    log(f"[rank {rank}] calibrate MB/s: {cal}")
    bw = dict(bw_fill=max(cal["fill_MBps"], 1), bw_zc=max(cal["zc_MBps"], 1),
              bw_zc_residual=cal["zc_residual_MBps"] if args.residual else 0, bw_hbm=max(cal["hbm_MBps"], 1))
    moe = make(bw)
    if not dsv3:
        moe.set_launch_overlap(args.overlap)

    stream = torch.cuda.current_stream()
    CW = args.cache_warm_steps
    n_total = CW + Wn + K + args.prof_steps + 12

    def gen_inputs(batch):
        lg = torch.from_numpy(W.ar1_logits(L, n_total, batch, E, RHO, ALPHA, SEED)).to(dev)
        g = torch.Generator(device=dev)
        g.manual_seed(W.mix64(SEED, 77, batch))
        noise = torch.randn((n_total, L, batch, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        return lg, noise

    xbuf = torch.empty((L, max(B, 8), d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, max(B, 8), d), dtype=torch.bfloat16, device=dev)

    def step(lg, noise, s, batch):
        for l in range(L):
            if l == 0:
                x = noise[s, 0]
            else:
                x = xbuf[l, :batch]
                torch.add(noise[s, l], ybuf[l - 1, :batch], out=x)
            moe.layer(l, lg[s, l], x, ybuf[l, :batch], batch, stream)

    # With the SM-driven fill nothing in a step needs the host, so the whole step (48 x [route+plan, fill,
    # expert FFN, x = noise + y]) is captured once per batch size in a CUDA graph and replayed; the step's
    # logits and noise are copied into the graph's static input buffers first (two small device copies).
    use_graph = bool(args.graph) and args.fill == "sm"
    graphs = {}

    def graph_for(batch):
        if batch in graphs:
            return graphs[batch]
        s_lg = torch.empty((L, batch, E), dtype=torch.float32, device=dev)
        s_noise = torch.empty((L, batch, d), dtype=torch.bfloat16, device=dev)
        torch.cuda.synchronize()
        l0 = moe.launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            cs = torch.cuda.current_stream()
            for l in range(L):
                if l == 0:
                    x = s_noise[0]
                else:
                    x = xbuf[l, :batch]
                    torch.add(s_noise[l], ybuf[l - 1, :batch], out=x)
                moe.layer(l, s_lg[l], x, ybuf[l, :batch], batch, cs)
        per_step = moe.launch_count() - l0 + (L - 1) + 2
        graphs[batch] = (g, s_lg, s_noise, per_step)
        return graphs[batch]

    def step_graph(lg, noise, s, batch):
        g, s_lg, s_noise, _ = graph_for(batch)
        s_lg.copy_(lg[s], non_blocking=True)
        s_noise.copy_(noise[s], non_blocking=True)
        g.replay()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(lg, noise, batch, first, count, sample_clocks=False):
        sampler = ClockSampler(local) if sample_clocks else None
        barrier()
        if sampler:
            sampler.start()
            time.sleep(0.3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = moe.launch_count()
        if use_graph:
            graph_for(batch)
            torch.cuda.synchronize()
        e0.record(stream)
        for s in range(first, first + count):
            if use_graph:
                step_graph(lg, noise, s, batch)
            else:
                step(lg, noise, s, batch)
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        clocks = sampler.stop() if sampler else None
        if use_graph:
            launches = count * graph_for(batch)[3]
        else:
            launches = moe.launch_count() - l0 + count * (L - 1)     # + the harness's x = noise + y kernels
        if dist is not None:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, clocks, launches

    def stats_sum():
        tot = {}
        for l in range(L):
            for kk, v in moe.get_stats(l).items():
                tot[kk] = tot.get(kk, 0) + v
        return tot

    def kernel_alone(lg, noise, batch, first, count, overlap):
        """The expert-FFN kernel(s) timed alone: route, plan and fill every layer of a step first (untimed), then
        the forward calls of all L layers back to back between two CUDA events.  Returns (us per layer, record
        bytes streamed from HBM per layer)."""
        moe.set_launch_overlap(overlap)
        us, nbytes = [], []
        for s in range(first, first + count):
            st0 = stats_sum()
            for l in range(L):
                moe.route(l, lg[s, l], batch, stream)
                moe.plan(l, stream, want=False)
                moe.fill(l, None)
            torch.cuda.synchronize()
            st1 = stats_sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for l in range(L):
                moe.forward(l, noise[s, l], ybuf[l, :batch], stream)
            e1.record(stream)
            torch.cuda.synchronize()
            us.append(e0.elapsed_time(e1) * 1e3 / L)
            nbytes.append((st1["hits"] - st0["hits"] + st1["fills"] - st0["fills"] +
                           shape.n_shared * (st1["steps"] - st0["steps"])) * S / L)
        moe.set_launch_overlap(0)
        return statistics.median(us), sum(nbytes) / len(nbytes)

    results = {}
    for batch in ([B] if (args.only_batch or dsv3) else [B, 1] if B != 1 else [1]):
        lg, noise = gen_inputs(batch)
        moe.reset()
        moe.set_launch_overlap(args.overlap if not dsv3 else 0)
        # cache pre-warm: a fixed number of untimed steps from the empty cache, whatever --warmup is, so that the
        # timed region is the steady state; the first K of them are timed separately as the cold-start figure
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_cold = min(K, CW)
        c0.record(stream)
        for s in range(CW):
            step(lg, noise, s, batch)
            if s == n_cold - 1:
                c1.record(stream)
        torch.cuda.synchronize()
        cold_ms = c0.elapsed_time(c1) if n_cold > 0 else None
        for s in range(CW, CW + Wn):
            if use_graph:
                step_graph(lg, noise, s, batch)
            else:
                step(lg, noise, s, batch)
        torch.cuda.synchronize()
        st0 = stats_sum()
        ms, clocks, launches = timed(lg, noise, batch, CW + Wn, K, sample_clocks=(batch == B))
        st1 = stats_sum()
        dst = {kk: st1[kk] - st0[kk] for kk in st1}
        # ---- the roofline kernel, timed alone (one launch per layer: no split into hit / fill parts) ----
        split_saved = moe.cfg.split_min_pairs
        moe.set_split_min_pairs(0)
        p0 = CW + Wn + K
        n_alone = max(2, args.prof_steps // 4)
        alone = {}
        if not dsv3:
            for name, ov in (("overlapped", 2), ("plain", 0)):
                kernel_alone(lg, noise, batch, p0, 1, ov)                       # warm-up of the pass itself
                alone[name] = kernel_alone(lg, noise, batch, p0 + 1, n_alone, ov)
        else:
            kernel_alone(lg, noise, batch, p0, 1, 0)
            alone["plain"] = kernel_alone(lg, noise, batch, p0 + 1, n_alone, 0)
        # ---- per-kernel durations inside the step, each launch bracketed by two events (separate pass) ----
        moe.timing_enable(True)
        st2 = stats_sum()
        for s in range(p0 + 1 + n_alone, p0 + 1 + n_alone + max(2, args.prof_steps // 2)):
            step(lg, noise, s, batch)
        tim = moe.timing_read()
        st3 = stats_sum()
        moe.timing_enable(False)
        res_bytes = (st3["hits"] - st2["hits"] + st3["fills"] - st2["fills"] +
                     shape.n_shared * (st3["steps"] - st2["steps"])) * S
        moe.set_split_min_pairs(split_saved)
        # the same steps with the hits overlapping the fills, as in the timed region
        tim_ov = None
        if split_saved > 0 and batch * k >= split_saved and not dsv3:
            moe.timing_enable(True)
            for s in range(n_total - 6, n_total - 2):
                step(lg, noise, s, batch)
            tim_ov = moe.timing_read()
            moe.timing_enable(False)
        results[batch] = dict(ms=ms, clocks=clocks, launches=launches, dstats=dst, timing=tim, timing_overlapped=tim_ov,
                              alone=alone, cold_ms=cold_ms, n_cold=n_cold,
                              res_bytes=res_bytes, prof_fill_bytes=(st3["fills"] - st2["fills"]) * S,
                              lg=lg, noise=noise)
        log(f"[rank {rank}] batch {batch}: {ms / K:.3f} ms/step, {batch * K * world / (ms * 1e-3):.1f} tok/s, "
            f"per step: hits {dst['hits'] / K:.1f} fills {dst['fills'] / K:.2f} zc {dst['zc'] / K:.2f}; "
            f"kernel alone (us/launch, bytes/launch): {alone}")
        log(f"[rank {rank}]   kernel timing (us total, launches): {tim}")

    main = results[B]
    value = B * K * world / (main["ms"] * 1e-3)
    hbm_peak, peak_kind = peaks()
    tim = main["timing"]
    ffn_us, ffn_n = tim["ffn_res"]
    if dsv3:   # the int4 path streams a record with two kernels: gate/up (timed in the ffn_zc slot) + down
        ffn_us += tim["ffn_zc"][0]
    in_step = main["res_bytes"] / (ffn_us * 1e-6) / 1e9 if ffn_us > 0 else 0.0
    fill_us, fill_n = tim["fill"]
    best = main["alone"].get("overlapped") or main["alone"]["plain"]
    achieved = best[1] / (best[0] * 1e-6) / 1e9

    # end to end through the host-buffer entry point
    e2e = None
    if args.e2e_steps > 0:
        lg, noise = main["lg"], main["noise"]
        lg_h = lg.cpu().pin_memory()
        noise_h = noise.cpu().pin_memory()
        xh = torch.empty((L, B, d), dtype=torch.bfloat16).pin_memory()
        yh = torch.empty((L, B, d), dtype=torch.bfloat16).pin_memory()
        Ke = min(K, args.e2e_steps)

        def step_host(s):
            for l in range(L):
                if l == 0:
                    x = noise_h[s, 0]
                else:
                    x = xh[l]
                    torch.add(noise_h[s, l], yh[l - 1], out=x)
                moe.layer_host(l, lg_h[s, l], x, yh[l], B, stream)

        for s in range(CW + Wn + K, CW + Wn + K + 3):
            step_host(s)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for s in range(CW + Wn, CW + Wn + Ke):
            step_host(s)
        e1.record(stream)
        barrier()
        ms_e = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms_e], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms_e = float(t.item())
        e2e = {"value": B * Ke * world / (ms_e * 1e-3), "unit": "tok/s",
               "h2d_bytes_per_step": L * (B * E * 4 + B * d * 2), "d2h_bytes_per_step": L * B * d * 2,
               "steps": Ke}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        lg, noise = main["lg"], main["noise"]
        n_samp = min(args.cpu_layers, 2) if dsv3 else args.cpu_layers
        pool_np = pool.tensor.view(L, E, S).numpy()
        lg_np = lg[CW + Wn].cpu().numpy()
        xb = [noise[CW + Wn, l].cpu().view(torch.int16).numpy().view(np.uint16) for l in range(n_samp)]
        cm_args = (S, bw["bw_fill"], bw["bw_zc_residual"], bw["bw_zc"], bw["bw_hbm"], 1, 64, 128)
        sec = oracle_sample_seconds(pool_np, shape, Ns, cm_args, lg_np, xb, range(n_samp))
        cpu_baseline = {"value": B / (sec * L / n_samp), "unit": "tok/s", "cores": len(os.sched_getaffinity(0)),
                        "kind": "oracle",
                        "sample": f"{n_samp} of {L} layers of one decode step at batch {B} "
                                  f"({sec:.1f} s), time scaled x{L / n_samp:.0f}"}

    if rank == 0:
        dst = main["dstats"]
        line = {
            "metric": "moe_decode_tok_per_s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": K,
            "warmup": Wn, "ms_per_step": main["ms"] / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": (fp4_name + " weights, bf16 activations, fp32 accumulate" if mxfp4 else
                                         "int4 weights, bf16 activations, fp32 accumulate") if dsv3 else "bf16",
            "data": "synthetic",
            "config": {"workload": ("decode DeepSeek-V3-shaped " + fp4_name + " MoE stack (config 3 shapes)" if mxfp4 else
                                    "decode DeepSeek-V3-shaped int4 MoE stack (config 3)" if dsv3 else
                                    "decode Qwen3-30B-A3B-shaped MoE stack (config 1)"), "batch": B, "layers": L,
                       "hidden": d, "experts": E, "inter": shape.inter, "top_k": k, "slots_per_layer": Ns,
                       "fill_mode": args.fill, "cuda_graph": use_graph, "global_pool": bool(args.global_pool), "rho": RHO, "zipf_alpha": ALPHA,
                       "l2": "inputs larger than L2: every step streams GBs of distinct expert records from the slot "
                             "pool, far beyond the 126 MB L2; no flush needed",
                       "cache_warm_steps": CW, "launch_overlap_in_step": args.overlap,
                       "parallelism": "replicas" if world > 1 else "single",
                       "host_pool": "one /dev/shm copy shared by all ranks" if shm_name else "private pinned pool"},
            "clocks": main["clocks"],
            "e2e": e2e,
            "gpu_launches": main["launches"],
            "roofline": {
                "bound": "hbm",
                "kernel": ("tc_gateup_kernel + tc_down_kernel (one pass over each record)" if args.workload == "dsv3_mxfp4tc" else
                           "mx4_gateup_kernel + mx4_down_kernel (one pass over each record)" if mxfp4 else
                           "w4_gateup_kernel + w4_down_kernel (one pass over each record)" if dsv3
                           else "ffn_stream_kernel (expert FFN over the HBM-resident records of a layer)"),
                "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                "frac": achieved / hbm_peak if hbm_peak else None, "peak_source": peak_kind + " (burst: kernel timed alone)",
                "how": (f"kernel timed alone: route, plan and fill of all {L} layers of a step issued first (untimed), "
                        f"then the {L} forward launches back to back on the stream between two CUDA events, "
                        "launched as programmatic dependents (ft_moe_set_launch_overlap 2: a launch streams its "
                        "weights while the previous one drains and orders only its output accumulation after it); "
                        "duration = elapsed / launches, median over steps; bytes = resident experts x record bytes"
                        if "overlapped" in main["alone"] else
                        f"kernel timed alone: the {L} forward launches of a planned step back to back between two events"),
                "avg_launch_us": best[0], "bytes_per_launch": best[1], "launches_timed": L * max(2, args.prof_steps // 4),
                # DRAM read+write per launch from the ncu capture of the same kernel (profiles/): ratio to the
                # algorithmic bytes, scaled to this run's bytes per launch
                "traffic": (NCU_TRAFFIC_RATIO * best[1]) if not dsv3 else None,
                "traffic_source": (NCU_TRAFFIC_SOURCE if not dsv3 else None),
                # the same launches as plain back-to-back launches (no dependent-launch overlap)
                "plain_back_to_back": {"avg_launch_us": main["alone"]["plain"][0],
                                       "achieved": main["alone"]["plain"][1] / (main["alone"]["plain"][0] * 1e-6) / 1e9,
                                       "frac": main["alone"]["plain"][1] / (main["alone"]["plain"][0] * 1e-6) / 1e9 / hbm_peak},
                # and inside the step, every launch bracketed by its own pair of events (adds ~5 us per launch)
                "in_step_bracketed": {"avg_launch_us": ffn_us / ffn_n if ffn_n else None, "achieved": in_step,
                                      "frac": in_step / hbm_peak if hbm_peak else None,
                                      "bytes_per_launch": main["res_bytes"] / ffn_n if ffn_n else None}},
            "cpu_baseline": cpu_baseline,
            "cold_start": {"value": B * main["n_cold"] * world / (main["cold_ms"] * 1e-3) if main["cold_ms"] else None,
                           "unit": "tok/s", "steps": main["n_cold"],
                           "what": "the first steps from an empty cache (untimed part of the run, before the pre-warm ends)"},
            "per_step": {"hits": dst["hits"] / K, "fills": dst["fills"] / K, "zero_copy": dst["zc"] / K,
                         "routed_unique": dst["routed"] / K, "fill_bytes": dst["fills"] / K * S},
            "fill": {"GBps": (main["prof_fill_bytes"] / (fill_us * 1e-6) / 1e9) if fill_us > 0 else None,
                     "link_GBps_measured": cal["fill_MBps"] / 1e3, "zero_copy_GBps_measured": cal["zc_MBps"] / 1e3,
                     "zero_copy_residual_GBps_measured": cal["zc_residual_MBps"] / 1e3,
                     "hbm_read_GBps_measured": cal["hbm_MBps"] / 1e3},
            "kernel_us_per_launch": {kk: (v[0] / v[1] if v[1] else None) for kk, v in tim.items()},
            "kernel_us_per_launch_overlapped": ({kk: (v[0] / v[1] if v[1] else None) for kk, v in main["timing_overlapped"].items()}
                                                if main.get("timing_overlapped") else None),
        }
        if 1 in results and B != 1:
            r1 = results[1]
            t1 = r1["timing"]
            b1 = r1["alone"].get("overlapped") or r1["alone"]["plain"]
            a1 = b1[1] / (b1[0] * 1e-6) / 1e9
            a1p = r1["alone"]["plain"][1] / (r1["alone"]["plain"][0] * 1e-6) / 1e9
            a1s = r1["res_bytes"] / (t1["ffn_res"][0] * 1e-6) / 1e9 if t1["ffn_res"][0] > 0 else 0.0
            line["batch1"] = {"value": K * world / (r1["ms"] * 1e-3), "unit": "tok/s", "ms_per_step": r1["ms"] / K,
                              "ffn_res_GBps": a1, "ffn_res_frac": a1 / hbm_peak, "avg_launch_us": b1[0],
                              "bytes_per_launch": b1[1],
                              "plain_back_to_back_frac": a1p / hbm_peak, "in_step_bracketed_frac": a1s / hbm_peak,
                              "fills_per_step": r1["dstats"]["fills"] / K,
                              "cold_start_tok_per_s": (r1["n_cold"] * world / (r1["cold_ms"] * 1e-3)) if r1["cold_ms"] else None}
    moe.destroy()
    pool.free()
    results.clear()
    del xbuf, ybuf
    torch.cuda.empty_cache()
    if rank == 0:
        if world == 1 and not dsv3 and args.layers == 48:
            # bounded sub-records of the other single-GPU configurations (a few layers each)
            for name in [n for n in args.sub.split(",") if n and n != "none"]:
                t_sub = time.perf_counter()
                try:
                    line[name] = SUBRECORDS[name](args, dev, cal)
                except Exception as exc:      # a sub-record never takes the headline down with it
                    line[name] = {"error": f"{type(exc).__name__}: {exc}"}
                log(f"[rank 0] sub-record {name}: {time.perf_counter() - t_sub:.1f}s {line[name]}")
        print(json.dumps(line), flush=True)
    if shm_name is not None:
        MR.close_shared_pool(pool.array, shm_name, rank, dist.barrier)
    if dist is not None:
        dist.destroy_process_group()


def tensor_peaks():
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        dd = json.load(open(pk))
        return float(dd["bf16_tflops"]), float(dd["bf16_tflops_sustained"]), "measured"
    return FALLBACK_BF16_TFLOPS, 1400.0, "fallback"


def prefill_passes(args, dev, L, cal=None, shape=None, Ns=None):
    """Config 2 (or another layer shape) on L layers: one 4096-token step from a cold cache, then one on the cache it
    left behind.  Returns (per-pass records, calibration, layer constants)."""
    import torch
    from paper_2608_16157_b200 import binding as Bd
    from paper_2608_16157_b200 import workload as W
    shape = shape or W.QWEN3_30B
    E, k, d, I = shape.n_experts, shape.top_k, shape.d, shape.inter
    S = shape.expert_bytes
    Ns = Ns or W.slots_for_fraction(args.cache_frac, E)
    T = args.tokens
    pool = Bd.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, SEED, device=dev, chunk=32 if shape.wdtype == "bf16" else 16)
    common = dict(hidden=d, inter=I, n_experts=E, top_k=k, n_layers=L, slots_per_layer=Ns, max_tokens=T,
                  host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                  fill_mode=Bd.FT_FILL_SM if args.fill == "sm" else Bd.FT_FILL_COPY_ENGINE,
                  wdtype={"int4": Bd.FT_W_INT4_G128, "mxfp4": Bd.FT_W_MXFP4, "nvfp4": Bd.FT_W_NVFP4, "mxfp4tc": Bd.FT_W_MXFP4_TC,
                                     "bf16": Bd.FT_W_BF16}[shape.wdtype],
                  gemm_min_tokens=args.gemm_min_tokens)
    if shape.n_shared:
        shared = W.make_shared_records(shape, L, SEED, device=dev)
        common.update(n_shared=1, shared_ptr=shared.data_ptr())
    if cal is None:
        moe = Bd.FtMoe(Bd.make_config(**common))
        cal = moe.calibrate()
        moe.destroy()
    moe = Bd.FtMoe(Bd.make_config(bw_fill=max(cal["fill_MBps"], 1), bw_zc=max(cal["zc_MBps"], 1), bw_zc_residual=0,
                                  bw_hbm=max(cal["hbm_MBps"], 1), **common))
    stream = torch.cuda.current_stream()
    xbuf = torch.empty((L, T, d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, T, d), dtype=torch.bfloat16, device=dev)
    out = {}
    for name, step in (("cold", 0), ("warm", 1)):
        lg = torch.from_numpy(W.prefill_logits(L, T, E, ALPHA, SEED, step)).to(dev)
        g = torch.Generator(device=dev)
        g.manual_seed(W.mix64(SEED, 78, step))
        noise = torch.randn((L, T, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        st0 = {kk: sum(moe.get_stats(l)[kk] for l in range(L)) for kk in Bd.STAT_NAMES}
        moe.timing_enable(True)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = moe.launch_count()
        e0.record(stream)
        for l in range(L):
            if l == 0:
                x = noise[0]
            else:
                x = xbuf[l]
                torch.add(noise[l], ybuf[l - 1], out=x)
            moe.layer(l, lg[l], x, ybuf[l], T, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        tim = moe.timing_read()
        moe.timing_enable(False)
        st1 = {kk: sum(moe.get_stats(l)[kk] for l in range(L)) for kk in Bd.STAT_NAMES}
        dst = {kk: st1[kk] - st0[kk] for kk in st1}
        flops = 2.0 * 3 * d * I * dst["pairs_gemm"]
        gemm_us = tim["gemm1"][0] + tim["gemm2"][0]
        gather_us = tim["gather"][0]          # (4-bit experts: includes their expansion to bf16 records)
        fill_us = tim["fill"][0]
        route_us = tim["route"][0] + tim["plan"][0]
        out[name] = {"ms": ms, "tok_per_s": T / (ms * 1e-3), "launches": moe.launch_count() - l0 + L - 1,
                     "fills": dst["fills"], "zero_copy": dst["zc"], "hits": dst["hits"],
                     "pairs": dst["pairs"], "pairs_gemm": dst["pairs_gemm"],
                     "gemm_tflops": flops / (gemm_us * 1e-6) / 1e12 if gemm_us > 0 else None,
                     "gemm_with_gather_tflops": flops / ((gemm_us + gather_us) * 1e-6) / 1e12 if gemm_us > 0 else None,
                     "gemm1_tflops": (flops * 2 / 3) / (tim["gemm1"][0] * 1e-6) / 1e12 if tim["gemm1"][0] > 0 else None,
                     "gemm2_tflops": (flops / 3) / (tim["gemm2"][0] * 1e-6) / 1e12 if tim["gemm2"][0] > 0 else None,
                     "fill_GBps": dst["fills"] * S / (fill_us * 1e-6) / 1e9 if fill_us > 0 else None,
                     "route_plan_us_per_layer": route_us / L,
                     "kernel_ms": {kk: v[0] / 1e3 for kk, v in tim.items()}}
        log(f"prefill {name}: {out[name]}")
    moe.destroy()
    pool.free()
    del xbuf, ybuf
    torch.cuda.empty_cache()
    return out, cal, dict(T=T, L=L, d=d, E=E, I=I, k=k, Ns=Ns)


def prefill_double_buffered(args, dev, L, cal):
    """Config 2 on L layers with full-layer double buffering (paper Sec. 3.1): one shared slot pool, the whole
    expert set of layer l+1 is loaded by the copy engine while layer l is evaluated; every pair then runs on the
    tensor-core GEMMs.  Returns the wall time of one cold 4096-token step (the first layer's load is exposed)."""
    import torch
    from paper_2608_16157_b200 import binding as Bd
    from paper_2608_16157_b200 import workload as W
    shape = W.QWEN3_30B
    E, k, d, I = shape.n_experts, shape.top_k, shape.d, shape.inter
    S = shape.expert_bytes
    Ns = max(W.slots_for_fraction(args.cache_frac, E), (2 * E + L - 1) // L)     # the shared pool holds two layers
    T = args.tokens
    pool = Bd.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, SEED, device=dev, chunk=32)
    moe = Bd.FtMoe(Bd.make_config(hidden=d, inter=I, n_experts=E, top_k=k, n_layers=L, slots_per_layer=Ns, max_tokens=T,
                                  host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                                  fill_mode=Bd.FT_FILL_COPY_ENGINE, gemm_min_tokens=args.gemm_min_tokens, global_pool=1,
                                  bw_fill=max(cal["fill_MBps"], 1), bw_zc=max(cal["zc_MBps"], 1), bw_zc_residual=0,
                                  bw_hbm=max(cal["hbm_MBps"], 1)))
    stream = torch.cuda.current_stream()
    xbuf = torch.empty((L, T, d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, T, d), dtype=torch.bfloat16, device=dev)
    lg = torch.from_numpy(W.prefill_logits(L, T, E, ALPHA, SEED, 0)).to(dev)
    g = torch.Generator(device=dev)
    g.manual_seed(W.mix64(SEED, 78, 0))
    noise = torch.randn((L, T, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    moe.prefetch_layer(0, stream)
    for l in range(L):
        x = noise[0] if l == 0 else torch.add(noise[l], ybuf[l - 1], out=xbuf[l])
        moe.route(l, lg[l], T, stream)
        moe.plan(l, stream, want=False)
        moe.fill(l, stream)
        if l + 1 < L:
            moe.prefetch_layer(l + 1, stream)
        moe.forward(l, x, ybuf[l], stream)
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3
    st = {kk: sum(moe.get_stats(l)[kk] for l in range(L)) for kk in Bd.STAT_NAMES}
    assert moe.sync_status() == 0
    moe.destroy()
    pool.free()
    del xbuf, ybuf
    torch.cuda.empty_cache()
    return {"cold_ms": ms, "fills": st["fills"], "zero_copy": st["zc"], "slots_shared": L * Ns,
            "GBps_link": st["fills"] * S / (ms * 1e-3) / 1e9,
            "timing": "host wall clock around the step (the copy engine needs the host to read each plan record)"}


def run_prefill(args):
    """One prefill step of `--tokens` tokens through the stack, cold cache then warm (second step on the state
    the first left behind).  One JSON line; the roofline object is the tensor-core grouped GEMM."""
    import torch
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    out, cal, c = prefill_passes(args, dev, args.layers)
    tf_burst, tf_sust, peak_kind = tensor_peaks()
    w = out["warm"]
    line = {"metric": "moe_prefill_tok_per_s", "value": out["cold"]["tok_per_s"], "unit": "tok/s", "n_gpus": 1,
            "steps": 1, "warmup": 0, "ms_per_step": out["cold"]["ms"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "prefill Qwen3-30B-A3B-shaped MoE stack (config 2), cold cache", "tokens": c["T"],
                       "layers": c["L"], "hidden": c["d"], "experts": c["E"], "inter": c["I"], "top_k": c["k"],
                       "slots_per_layer": c["Ns"], "gemm_min_tokens": args.gemm_min_tokens, "fill_mode": args.fill},
            "cold": out["cold"], "warm": out["warm"],
            "roofline": {"bound": "tensor", "kernel": "gateup_gemm_kernel + down_gemm2_kernel (warm pass)",
                         "achieved": w["gemm_tflops"], "peak": tf_burst, "unit": "TFLOP/s",
                         "frac": (w["gemm_tflops"] / tf_burst) if w["gemm_tflops"] else None,
                         "frac_of_sustained": (w["gemm_tflops"] / tf_sust) if w["gemm_tflops"] else None,
                         "peak_source": peak_kind, "traffic": None},
            "fill": {"GBps": out["cold"]["fill_GBps"], "link_GBps_measured": cal["fill_MBps"] / 1e3},
            "gpu_launches": out["cold"]["launches"]}
    print(json.dumps(line), flush=True)


def sub_prefill(args, dev, cal):
    """Sub-record of the decode line: config 2 (4096-token prefill) on 4 of the 48 layers."""
    L = 4
    out, cal, c = prefill_passes(args, dev, L, cal)
    tf_burst, tf_sust, peak_kind = tensor_peaks()
    w, cd = out["warm"], out["cold"]
    dbuf = prefill_double_buffered(args, dev, L, cal)
    return {"double_buffered": dict(dbuf, vs_on_demand_cold=dbuf["cold_ms"] / cd["ms"],
                                    note="full-layer double buffering loads all 128 experts of every layer; on-demand "
                                         "loads the ~124 routed ones (64 fills + ~60 zero-copy); both are bound by "
                                         "the host link, the GEMMs of a layer take ~1 ms of its ~22 ms"),
            "config": f"prefill, config 2 shapes, {c['T']} tokens, {L} of 48 layers, {c['Ns']} slots per layer, "
                      f"experts with >= {args.gemm_min_tokens} tokens and a slot on the tcgen05 grouped GEMMs",
            "cold_ms": cd["ms"], "warm_ms": w["ms"], "cold_ms_scaled_to_48_layers": cd["ms"] * 48 / L,
            "warm_ms_scaled_to_48_layers": w["ms"] * 48 / L,
            "useful_tflops": w["gemm_tflops"], "gateup_tflops": w["gemm1_tflops"], "down_tflops": w["gemm2_tflops"],
            "frac": (w["gemm_tflops"] / tf_burst) if w["gemm_tflops"] else None,
            "frac_of_sustained": (w["gemm_tflops"] / tf_sust) if w["gemm_tflops"] else None,
            "peak_burst_tflops": tf_burst, "peak_sustained_tflops": tf_sust, "peak_source": peak_kind,
            "how": "useful (unpadded) flops of the pairs served by the GEMMs / summed CUDA-event durations of the "
                   "two GEMM kernels, warm pass",
            "fill_GBps_cold": cd["fill_GBps"], "route_plan_us_per_layer": w["route_plan_us_per_layer"],
            "pairs_on_gemm_frac": w["pairs_gemm"] / max(w["pairs"], 1), "zero_copy_experts_cold": cd["zero_copy"]}


def sub_prefill_mxfp4(args, dev, cal):
    """Sub-record: a 4096-token call on one layer of config 3's shape with MXFP4 experts and 64 slots: the slot-
    resident experts with >= gemm_min_tokens tokens are expanded to bf16 records and run on the tcgen05 GEMMs."""
    from paper_2608_16157_b200 import workload as W
    out, cal, c = prefill_passes(args, dev, 1, cal, shape=W.DSV3_MXFP4, Ns=64)
    tf_burst, tf_sust, peak_kind = tensor_peaks()
    w, cd = out["warm"], out["cold"]
    return {"config": f"prefill, config 3 layer shape (d=7168, 256 mxfp4 experts + 1 shared, I=2048, top-8), "
                      f"{c['T']} tokens, 1 layer, 64 slots",
            "cold_ms": cd["ms"], "warm_ms": w["ms"],
            "useful_tflops_gemms": w["gemm_tflops"], "useful_tflops_with_expansion": w["gemm_with_gather_tflops"],
            "frac": (w["gemm_with_gather_tflops"] / tf_burst) if w["gemm_with_gather_tflops"] else None,
            "peak_burst_tflops": tf_burst, "peak_source": peak_kind,
            "how": "useful (unpadded) flops of the pairs served by the GEMMs / CUDA-event durations of the expansion "
                   "of the GEMM-list experts to bf16 records + row gather + the two GEMM kernels, warm pass",
            "pairs_on_gemm_frac": w["pairs_gemm"] / max(w["pairs"], 1), "kernel_ms": w["kernel_ms"],
            "zero_copy_experts_warm": w["zero_copy"], "hits_warm": w["hits"]}


def sub_int4(args, dev, cal, wdtype="int4"):
    """Sub-record of the decode line: config 3 (DeepSeek-V3-shaped 4-bit decode, 4 layers, batch 4, 64 slots), with
    int4-g128 experts or (the format the paper serves) MXFP4 experts."""
    import torch
    from paper_2608_16157_b200 import binding as Bd
    from paper_2608_16157_b200 import workload as W
    shape = {"int4": W.DSV3_INT4, "mxfp4": W.DSV3_MXFP4, "nvfp4": W.DSV3_NVFP4, "mxfp4tc": W.DSV3_MXFP4TC}[wdtype]
    L, E, k, d, B, Ns = 4, shape.n_experts, shape.top_k, shape.d, 4, 64
    S = shape.expert_bytes
    warm, K = 48, 16
    pool = Bd.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, SEED, device=dev, chunk=16)
    shared = W.make_shared_records(shape, L, SEED, device=dev)
    moe = Bd.FtMoe(Bd.make_config(hidden=d, inter=shape.inter, n_experts=E, top_k=k, n_layers=L, slots_per_layer=Ns,
                                  max_tokens=8, host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                                  fill_mode=Bd.FT_FILL_SM,
                                  wdtype={"int4": Bd.FT_W_INT4_G128, "mxfp4": Bd.FT_W_MXFP4, "nvfp4": Bd.FT_W_NVFP4,
                                          "mxfp4tc": Bd.FT_W_MXFP4_TC}[wdtype], n_shared=1,
                                  shared_ptr=shared.data_ptr(), bw_fill=max(cal["fill_MBps"], 1),
                                  bw_zc=max(cal["zc_MBps"], 1), bw_zc_residual=0, bw_hbm=max(cal["hbm_MBps"], 1)))
    stream = torch.cuda.current_stream()
    n_total = warm + K + 12
    lg = torch.from_numpy(W.ar1_logits(L, n_total, B, E, 0.9, 1.2, SEED)).to(dev)
    g = torch.Generator(device=dev)
    g.manual_seed(W.mix64(SEED, 80, B))
    noise = torch.randn((n_total, L, B, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    xbuf = torch.empty((L, B, d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, B, d), dtype=torch.bfloat16, device=dev)

    def step(s):
        for l in range(L):
            x = noise[s, 0] if l == 0 else torch.add(noise[s, l], ybuf[l - 1], out=xbuf[l])
            moe.layer(l, lg[s, l], x, ybuf[l], B, stream)

    def stats_sum():
        tot = {}
        for l in range(L):
            for kk, v in moe.get_stats(l).items():
                tot[kk] = tot.get(kk, 0) + v
        return tot

    for s in range(warm):
        step(s)
    torch.cuda.synchronize()
    st0 = stats_sum()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(warm, warm + K):
        step(s)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    st1 = stats_sum()
    # the two int4 kernels (gate/up, down) timed alone: all layers planned and filled first, then the forward
    # calls back to back between two events
    us, nbytes = {2: [], 0: []}, {2: [], 0: []}
    for s in range(warm + K, warm + K + 12):
        ov = 2 if s < warm + K + 6 else 0     # six steps with the launches overlapped, six plain
        moe.set_launch_overlap(ov)
        a = stats_sum()
        for l in range(L):
            moe.route(l, lg[s, l], B, stream)
            moe.plan(l, stream, want=False)
            moe.fill(l, None)
        torch.cuda.synchronize()
        b = stats_sum()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for l in range(L):
            moe.forward(l, noise[s, l], ybuf[l], stream)
        f1.record(stream)
        torch.cuda.synchronize()
        us[ov].append(f0.elapsed_time(f1) * 1e3 / L)
        nbytes[ov].append((b["hits"] - a["hits"] + b["fills"] - a["fills"] + (b["steps"] - a["steps"])) * S / L)
    moe.set_launch_overlap(0)
    assert moe.sync_status() == 0
    moe.destroy()
    pool.free()
    hbm_peak, peak_kind = peaks()
    t_us, nb = statistics.median(us[2][1:]), sum(nbytes[2][1:]) / len(nbytes[2][1:])
    gbps = nb / (t_us * 1e-6) / 1e9
    t0_us, nb0 = statistics.median(us[0][1:]), sum(nbytes[0][1:]) / len(nbytes[0][1:])
    gbps0 = nb0 / (t0_us * 1e-6) / 1e9
    return {"config": "decode, config 3: d=7168, 256 %s experts + 1 shared, I=2048, top-8, 4 layers, 64 slots "
                      "per layer, batch 4, rho 0.9, alpha 1.2" % ("int4-g128" if wdtype == "int4" else wdtype),
            "kernels": "w4_gateup_kernel + w4_down_kernel" if wdtype == "int4" else
                       "tc_quant_x_kernel + tc_gateup_kernel + tc_down_kernel (tcgen05 kind::mxf4 block-scaled MMA on "
                       "records stored as operand images)" if wdtype == "mxfp4tc" else
                       "mx4_gateup_kernel + mx4_down_kernel" + (" (NVFP4 instances)" if wdtype == "nvfp4" else ""),
            "bound": "hbm" if wdtype in ("int4", "mxfp4tc") else "alu (logic pipe: 7 instructions per 8 weights plus a scale per MMA"
                     + (", one K=16 MMA per 16-element scale block" if wdtype == "nvfp4" else "") + "); reported against the HBM peak",
            "tok_per_s": B * K / (ms * 1e-3), "ms_per_step": ms / K,
            "fills_per_step": (st1["fills"] - st0["fills"]) / K, "cache_warm_steps": warm,
            "GBps": gbps, "frac": gbps / hbm_peak, "peak": hbm_peak, "peak_source": peak_kind,
            "avg_us_per_layer": t_us, "bytes_per_layer": nb,
            "plain_back_to_back": {"avg_us_per_layer": t0_us, "GBps": gbps0, "frac": gbps0 / hbm_peak},
            "how": "gate/up + down kernels of a layer timed alone: the 4 layers of a step planned and filled first, "
                   "then their forward calls back to back between two CUDA events, the gate/up kernels launched as "
                   "programmatic dependents (ft_moe_set_launch_overlap 2: a layer's set-up overlaps the previous "
                   "layer's tail); plain_back_to_back = the same with plain launches; bytes = (resident routed "
                   "experts + the shared expert) x record bytes"}


def sub_mxfp4(args, dev, cal):
    return sub_int4(args, dev, cal, "mxfp4")


def sub_mxfp4tc(args, dev, cal):
    return sub_int4(args, dev, cal, "mxfp4tc")


def sub_nvfp4(args, dev, cal):
    return sub_int4(args, dev, cal, "nvfp4")


SUBRECORDS = {"int4": sub_int4, "mxfp4": sub_mxfp4, "mxfp4tc": sub_mxfp4tc, "nvfp4": sub_nvfp4, "prefill": sub_prefill,
              "prefill_mxfp4": sub_prefill_mxfp4}


def run_sweep(args):
    """Cache-pressure sweep on the decode shapes: cache fraction x locality rho x batch, `--sweep-steps` steps
    each from an empty cache.  One JSON line with a record per point."""
    import torch
    from paper_2608_16157_b200 import binding as Bd
    from paper_2608_16157_b200 import workload as W
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    shape = W.QWEN3_30B
    L, E, k, d = args.layers, shape.n_experts, shape.top_k, shape.d
    S = shape.expert_bytes
    steps = args.sweep_steps
    pool = Bd.HostPool(L * E * S)
    W.fill_pool(pool.tensor, shape, L, SEED, device=dev, chunk=32)
    stream = torch.cuda.current_stream()
    points = []
    xbuf = torch.empty((L, 64, d), dtype=torch.bfloat16, device=dev)
    ybuf = torch.empty((L, 64, d), dtype=torch.bfloat16, device=dev)
    cal = None
    fracs = [float(v) for v in args.sweep_fracs.split(",")]
    rhos = [float(v) for v in args.sweep_rhos.split(",")]
    batches = [int(v) for v in args.sweep_batches.split(",")]
    for frac in fracs:
        Ns = W.slots_for_fraction(frac, E)
        common = dict(hidden=d, inter=shape.inter, n_experts=E, top_k=k, n_layers=L, slots_per_layer=Ns,
                      max_tokens=64, host_pool_ptr=pool.ptr.value, host_pool_bytes=pool.n_bytes,
                      fill_mode=Bd.FT_FILL_SM if args.fill == "sm" else Bd.FT_FILL_COPY_ENGINE)
        if cal is None:
            m0 = Bd.FtMoe(Bd.make_config(**common))
            cal = m0.calibrate()
            m0.destroy()
        moe = Bd.FtMoe(Bd.make_config(bw_fill=max(cal["fill_MBps"], 1), bw_zc=max(cal["zc_MBps"], 1),
                                      bw_zc_residual=cal["zc_residual_MBps"] if args.residual else 0,
                                      bw_hbm=max(cal["hbm_MBps"], 1), **common))
        for rho in rhos:
            for batch in batches:
                lg = torch.from_numpy(W.ar1_logits(L, steps, batch, E, rho, ALPHA, SEED)).to(dev)
                g = torch.Generator(device=dev)
                g.manual_seed(W.mix64(SEED, 79, batch))
                noise = torch.randn((steps, L, batch, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
                moe.reset()
                torch.cuda.synchronize()
                e0, e1, em = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                tail = max(1, steps // 4)            # the last quarter of the point: the cache has settled
                st_mid = None
                e0.record(stream)
                for s_ in range(steps):
                    if s_ == steps - tail:
                        torch.cuda.synchronize()
                        st_mid = {kk: sum(moe.get_stats(l)[kk] for l in range(L)) for kk in Bd.STAT_NAMES}
                        em.record(stream)
                    for l in range(L):
                        if l == 0:
                            x = noise[s_, 0]
                        else:
                            x = xbuf[l, :batch]
                            torch.add(noise[s_, l], ybuf[l - 1, :batch], out=x)
                        moe.layer(l, lg[s_, l], x, ybuf[l, :batch], batch, stream)
                e1.record(stream)
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1)
                ms_tail = em.elapsed_time(e1)
                st = {kk: sum(moe.get_stats(l)[kk] for l in range(L)) for kk in Bd.STAT_NAMES}
                pt = {"cache_frac": frac, "slots": Ns, "rho": rho, "batch": batch, "steps": steps,
                      "tok_per_s": batch * steps / (ms * 1e-3), "ms_per_step": ms / steps,
                      "hit_rate_unique": st["hits"] / max(st["routed"], 1),
                      "hit_rate_pairs": st["pairs_resident"] / max(st["pairs"], 1),
                      "fills": st["fills"], "zero_copies": st["zc"], "evictions": st["evictions"],
                      "fill_bytes": st["fills"] * S, "zero_copy_bytes": st["zc"] * S,
                      "routed_unique_per_layer_step": st["routed"] / (steps * L),
                      "resident_record_GBps": (st["hits"] + st["fills"]) * S / (ms * 1e-3) / 1e9,
                      "settled": {"steps": tail, "tok_per_s": batch * tail / (ms_tail * 1e-3),
                                  "ms_per_step": ms_tail / tail,
                                  "fills_per_step": (st["fills"] - st_mid["fills"]) / tail,
                                  "resident_record_GBps": (st["hits"] - st_mid["hits"] + st["fills"] - st_mid["fills"])
                                  * S / (ms_tail * 1e-3) / 1e9}}
                points.append(pt)
                log(f"sweep {pt}")
        moe.destroy()
    line = {"metric": "moe_decode_sweep", "unit": "tok/s", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "cache-pressure sweep on the decode shapes (config 4)", "layers": L,
                       "hidden": d, "experts": E, "inter": shape.inter, "top_k": k, "fill_mode": args.fill,
                       "zipf_alpha": ALPHA, "steps_per_point": steps, "cold_start": True,
                       "plan_uses_residual_zero_copy_rate": bool(args.residual)},
            "link_GBps_measured": cal["fill_MBps"] / 1e3, "points": points}
    print(json.dumps(line), flush=True)
    pool.free()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sweep-steps", type=int, default=128)
    ap.add_argument("--sweep-fracs", default="0.10,0.25,0.50,0.75,1.00")
    ap.add_argument("--sweep-rhos", default="0,0.5,0.9")
    ap.add_argument("--sweep-batches", default="1,16,64")
    ap.add_argument("--global-pool", type=int, default=0, help="1: one slot pool and LRU clock shared by all layers")
    ap.add_argument("--graph", type=int, default=1, help="replay each decode step as one CUDA graph (SM fill only)")
    ap.add_argument("--workload", default="qwen", choices=["qwen", "dsv3", "dsv3_mxfp4", "dsv3_nvfp4", "dsv3_mxfp4tc"])
    ap.add_argument("--mode", default="decode", choices=["decode", "prefill", "sweep"])
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--gemm-min-tokens", type=int, default=32)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--layers", type=int, default=48)
    ap.add_argument("--cache-frac", type=float, default=0.5)
    ap.add_argument("--fill", default="sm", choices=["ce", "sm"])
    ap.add_argument("--residual", type=int, default=0, help="use the measured residual zero-copy rate in the plan")
    ap.add_argument("--prof-steps", type=int, default=16)
    ap.add_argument("--e2e-steps", type=int, default=32)
    ap.add_argument("--cpu-layers", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-batch", action="store_true")
    ap.add_argument("--cache-warm-steps", type=int, default=64,
                    help="untimed steps from the empty cache before warm-up and timing (steady-state headline)")
    ap.add_argument("--sub", default="int4,mxfp4,mxfp4tc,nvfp4,prefill,prefill_mxfp4", help="bounded sub-records added to the decode line (N=1 only)")
    ap.add_argument("--overlap", type=int, default=0,
                    help="launch mode of the streaming kernel in the timed region (ft_moe_set_launch_overlap)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "prefill":
        run_prefill(args)
    elif args.mode == "sweep":
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
