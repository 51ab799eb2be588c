#!/usr/bin/env python
"""Benchmark of the DASC hot path on B200: one step = pack -> restore (zero-fill) ->
suffix refresh over one batch of synthetic state checkpoints.

Workload (N=1): the serving-scale KDA configuration -- 24 KDA layers x 32 heads x
128x128 fp32 states (2 MiB per layer and request), 64 requests, per-channel decay rates
log-uniform in [1e-3, 1] (seed 1), keep ratio 0.38 per layer -- followed by a refresh of
a 256-token bf16 suffix per request.  Inputs are far larger than L2, so no flush is needed.

Prints ONE JSON line.  `value` is pack+restore algorithmic GB/s (bytes the two copies must
move / their device time); refresh throughput, per-kernel rooflines, the end-to-end leg
(host buffers, copies timed) and the CPU oracle baseline ride along in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

WORKLOAD = "kda_serving_24x32x128x128_fp32_64req_keep0.38_suffix256_bf16"
L, H, D, N_REQ, KEEP, SUFFIX, SEED = 24, 32, 128, 64, 0.38, 256, 1
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# CPU oracle leg (the reported baseline and the whole of --impl reference)
# ----------------------------------------------------------------------------------------------

def oracle_leg(sample_req=4, sample_units=64):
    """Times the fp64 oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    from paper_2608_30386_b200 import synth

    gen = synth.generator(SEED)
    rates = synth.decay_rates(gen, L, H, D, 1e-3, 1.0)
    A_log, dt = synth.decay_params(rates)
    oplan = oracle.plan(oracle.KDA, L, H, D, A_log.numpy(), dt.numpy(), sel=oracle.SEL_TOP_RATIO, keep_ratio=KEEP,
                        scope=oracle.SCOPE_LAYER, unit_bytes=D * 4)
    dense = H * D * D
    state = synth.states(gen, (sample_req, L, dense)).numpy()
    slot = oplan.sum_r * D
    pool = np.zeros((sample_req, slot), np.float32)
    out = np.empty_like(state)
    ids = np.arange(sample_req, dtype=np.int32)
    t0 = time.perf_counter()
    oracle.pack(oplan.mask, D, state, dense, L * dense, ids, pool, slot, ids)
    t1 = time.perf_counter()
    oracle.restore(oplan.mask, D, pool, slot, ids, out, dense, L * dense, ids)
    t2 = time.perf_counter()
    pack_bytes = 2 * sample_req * slot * 4
    restore_bytes = sample_req * (slot + L * dense) * 4
    # refresh sample: `sample_units` (request, layer, head) units = 2 layers x 32 heads of one request
    Ls = max(1, sample_units // H)
    streams = synth.token_streams(gen, synth.KDA, Ls, SUFFIX, H, H, D, D, rates[:Ls])
    st = synth.states(gen, (1, Ls, H, D, D)).numpy()
    threads = oracle.max_threads()
    t3 = time.perf_counter()
    oracle.refresh(oracle.KDA, Ls, H, H, D, D, st, dense, Ls * dense, [0], synth.bf16_bits(streams.q),
                   synth.bf16_bits(streams.k), synth.bf16_bits(streams.v), streams.g.numpy(), streams.beta.numpy(),
                   [0, SUFFIX], n_threads=threads)
    t4 = time.perf_counter()
    token_heads = Ls * H * SUFFIX
    # tokens/s of the full model (all L layers and H heads per token), extrapolated from the sampled units
    refresh_tokens_per_s = token_heads / (t4 - t3) / (L * H)
    return {
        "value": (pack_bytes + restore_bytes) / (t2 - t0) / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
        "sample": (f"pack+restore of {sample_req} of {N_REQ} requests (single thread); refresh of {Ls * H} of "
                   f"{N_REQ * L * H} (request,layer,head) units x {SUFFIX} tokens on {threads} threads"),
        "pack_GBps": pack_bytes / (t1 - t0) / 1e9, "restore_GBps": restore_bytes / (t2 - t1) / 1e9,
        "refresh_tokens_per_s": refresh_tokens_per_s, "refresh_token_heads_per_s": token_heads / (t4 - t3),
        "seconds": t4 - t0,
    }


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    leg = None
    for i in range(args.warmup + args.steps):
        leg = oracle_leg(sample_req=2, sample_units=32)
        if i >= args.warmup:
            vals.append(leg)
    value = statistics.mean(v["value"] for v in vals)
    sec = statistics.mean(v["seconds"] for v in vals)
    line = {
        "impl": "reference", "metric": "pack_restore_GBps", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle on a bounded sample of the workload per step"},
        "refresh_tokens_per_s": statistics.mean(v["refresh_tokens_per_s"] for v in vals),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": leg["cores"], "kind": "oracle",
                         "sample": leg["sample"]},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# GPU legs
# ----------------------------------------------------------------------------------------------

def main():
    global N_REQ, SUFFIX, KEEP, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dasc", choices=["dasc", "reference"])
    ap.add_argument("--algo", default="auto", choices=["auto", "sequential", "chunked"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--requests", type=int, default=N_REQ, help="profiling only: shrink the batch")
    ap.add_argument("--suffix", type=int, default=SUFFIX, help="profiling only: shrink the refresh suffix")
    ap.add_argument("--keep", type=float, default=KEEP, help="keep ratio (0.25, 0.38, 0.5, 1.0 in the sweep)")
    args = ap.parse_args()
    if (args.requests, args.suffix, args.keep) != (N_REQ, SUFFIX, KEEP):
        N_REQ, SUFFIX, KEEP = args.requests, args.suffix, args.keep
        WORKLOAD = f"kda_24x32x128x128_fp32_{N_REQ}req_keep{KEEP}_suffix{SUFFIX}_bf16"
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import paper_2608_30386_b200 as dasc
    from paper_2608_30386_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    algo = {"auto": dasc.ALGO_AUTO, "sequential": dasc.ALGO_SEQUENTIAL, "chunked": dasc.ALGO_CHUNKED}[args.algo]
    pk = peaks()

    # ---- plan and inputs (replicas: every rank holds the same shape of work, its own seed) ----
    gen = synth.generator(SEED)
    rates = synth.decay_rates(gen, L, H, D, 1e-3, 1.0)
    A_log, dt = synth.decay_params(rates)
    plan = dasc.dasc_plan(dasc.KDA, L, H, H, D, D, A_log.numpy(), dt.numpy(), sel=dasc.SEL_TOP_RATIO,
                          scope=dasc.SCOPE_LAYER, keep_ratio=KEEP, device=local)
    dense = H * D * D
    layer_stride, req_stride = N_REQ * dense, dense          # layer-major active-state pool
    dgen = synth.generator(SEED + 1000 * rank, dev)
    state = synth.states(dgen, (L, N_REQ, dense), dev)
    active = torch.empty_like(state)
    slot = int(plan.slot_floats)
    pool = torch.empty((N_REQ, slot), device=dev)
    ids = torch.arange(N_REQ, dtype=torch.int32, device=dev)
    slots = torch.randperm(N_REQ, generator=gen).to(torch.int32).to(dev)
    T = N_REQ * SUFFIX
    streams = []
    for l in range(L):                                       # per layer, to bound the generator's temporaries
        s = synth.token_streams(dgen, synth.KDA, 1, T, H, H, D, D, rates[l:l + 1], device=dev)
        streams.append(s)
    q = torch.cat([s.q for s in streams]); k = torch.cat([s.k for s in streams]); v = torch.cat([s.v for s in streams])
    g = torch.cat([s.g for s in streams]); beta = torch.cat([s.beta for s in streams])
    del streams
    o = torch.empty((L, T, H, D), dtype=torch.bfloat16, device=dev)
    cu = synth.uniform_cu_seqlens(N_REQ, SUFFIX).to(dev)
    ws_bytes = dasc.dasc_refresh_workspace_bytes(plan, N_REQ, L, algo)
    ws = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device=dev) if ws_bytes else None

    pack_bytes = 2 * N_REQ * slot * 4
    restore_bytes = N_REQ * (slot + L * dense) * 4
    token_heads = N_REQ * L * H * SUFFIX
    # refresh algorithmic bytes per (token, head): q + k + v bf16, g fp32, beta, o bf16; plus the state in and out
    refresh_bytes = token_heads * (3 * D * 2 + D * 4 + 4 + D * 2) + 2 * N_REQ * L * dense * 4
    refresh_flops_min = token_heads * 7 * D * D              # token-by-token recurrence, incl. decay and read-out

    stream = torch.cuda.current_stream()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        dasc.dasc_pack(plan, state, layer_stride, req_stride, ids, pool, slots)
        if ev:
            ev[1].record(stream)
        dasc.dasc_restore(plan, pool, slots, active, layer_stride, req_stride, ids)
        if ev:
            ev[2].record(stream)
        dasc.dasc_refresh(plan, active, layer_stride, req_stride, ids, q, k, v, g, beta, cu, T, SUFFIX, o=o,
                          algo=algo, workspace=ws)
        if ev:
            ev[3].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert dasc.dasc_refresh_status(ws) == 0
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        step(events[i])
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    t_pack = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    t_restore = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
    t_refresh = sum(e[2].elapsed_time(e[3]) for e in events) / args.steps
    t_total = events[0][0].elapsed_time(events[-1][3]) / args.steps
    times = torch.tensor([t_pack, t_restore, t_refresh, t_total], dtype=torch.float64, device=dev)
    if dist:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    t_pack, t_restore, t_refresh, t_total = times.tolist()

    # ---- end-to-end leg: host buffers, copies inside the timed region -------------------------
    e2e = None
    if not args.no_e2e:
        n_e = min(16, N_REQ)                                 # requests per e2e step (bounded pinned memory)
        Te = n_e * SUFFIX
        h_state = torch.empty((L, n_e, dense), dtype=torch.float32).pin_memory()
        h_state.copy_(state[:, :n_e])
        host_streams = [x[:, :Te].contiguous().cpu().pin_memory() for x in (q, k, v, g, beta)]
        h_pool = torch.empty((n_e, slot), dtype=torch.float32).pin_memory()
        h_out = torch.empty((L, n_e, dense), dtype=torch.float32).pin_memory()
        h_o = torch.empty((L, Te, H, D), dtype=torch.bfloat16).pin_memory()
        d_state = torch.empty((L, n_e, dense), device=dev)
        d_active = torch.empty_like(d_state)
        d_pool = torch.empty((n_e, slot), device=dev)
        d_streams = [torch.empty(x.shape, dtype=x.dtype, device=dev) for x in host_streams]
        d_o = torch.empty((L, Te, H, D), dtype=torch.bfloat16, device=dev)
        cu_e = synth.uniform_cu_seqlens(n_e, SUFFIX).to(dev)
        ids_e = torch.arange(n_e, dtype=torch.int32, device=dev)
        ls_e = n_e * dense

        def e2e_step(ev):
            ev[0].record(stream)
            d_state.copy_(h_state, non_blocking=True)
            dasc.dasc_pack(plan, d_state, ls_e, dense, ids_e, d_pool, ids_e)
            dasc.dasc_restore(plan, d_pool, ids_e, d_active, ls_e, dense, ids_e)
            h_pool.copy_(d_pool, non_blocking=True)
            ev[1].record(stream)
            for dst, src in zip(d_streams, host_streams):
                dst.copy_(src, non_blocking=True)
            dasc.dasc_refresh(plan, d_active, ls_e, dense, ids_e, *d_streams, cu_e, Te, SUFFIX, o=d_o, algo=algo,
                              workspace=ws)
            h_out.copy_(d_active, non_blocking=True)
            h_o.copy_(d_o, non_blocking=True)
            ev[2].record(stream)

        n_steps_e = max(2, min(args.steps, 3))
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_steps_e + 1)]
        e2e_step(evs[0])                                     # warm-up
        barrier()
        for i in range(1, n_steps_e + 1):
            e2e_step(evs[i])
        barrier()
        t_copy = sum(e[0].elapsed_time(e[1]) for e in evs[1:]) / n_steps_e
        t_ref = sum(e[1].elapsed_time(e[2]) for e in evs[1:]) / n_steps_e
        tt = torch.tensor([t_copy, t_ref], dtype=torch.float64, device=dev)
        if dist:
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        t_copy, t_ref = tt.tolist()
        e_bytes = (2 * n_e * slot + n_e * (slot + L * dense)) * 4
        h2d = h_state.numel() * 4 + sum(x.numel() * x.element_size() for x in host_streams)
        d2h = h_pool.numel() * 4 + h_out.numel() * 4 + h_o.numel() * 2
        e2e = {"value": world * e_bytes / (t_copy * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "requests_per_step": n_e,
               "refresh_tokens_per_s": world * Te / (t_ref * 1e-3), "ms_pack_restore": t_copy, "ms_refresh": t_ref,
               "note": "pinned host buffers; H2D of states and token streams, D2H of pool, states and outputs timed"}
        del h_state, host_streams, h_pool, h_out, h_o, d_state, d_active, d_pool, d_streams, d_o

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    hbm, tf = float(pk["hbm_gbs"]), float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"]))
    src = pk["_source"]
    pack_gbs = pack_bytes / (t_pack * 1e-3) / 1e9
    restore_gbs = restore_bytes / (t_restore * 1e-3) / 1e9
    refresh_gbs = refresh_bytes / (t_refresh * 1e-3) / 1e9
    # fp32 FMA peak of the CUDA cores: 148 SMs x 128 lanes x 2 flop x max SM clock
    alu_tflops = 148 * 128 * 2 * float(pk.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
    refresh_tflops = refresh_flops_min / (t_refresh * 1e-3) / 1e12
    rl = {
        "pack": {"bound": "hbm", "achieved": pack_gbs, "peak": hbm, "unit": "GB/s", "frac": pack_gbs / hbm,
                 "traffic": None, "peak_source": src, "frac_of_8TBps_nominal": pack_gbs / 8000.0},
        "restore": {"bound": "hbm", "achieved": restore_gbs, "peak": hbm, "unit": "GB/s", "frac": restore_gbs / hbm,
                    "traffic": None, "peak_source": src, "frac_of_8TBps_nominal": restore_gbs / 8000.0},
        # By the arithmetic (about 100 flop per byte, below the ridge) HBM is the ceiling of the refresh;
        # the tensor-pipe figures beside it: tf32 flops the chunked kernel issues (163,840 per token-head)
        # against the tf32 peak taken as 0.489 x the measured sustained bf16 peak (nominal 1.1 : 2.25).
        "refresh": {"bound": "hbm", "achieved": refresh_gbs, "peak": hbm, "unit": "GB/s", "frac": refresh_gbs / hbm,
                    "traffic": None, "peak_source": src, "tflops_min_form": refresh_tflops,
                    "frac_of_fp32_alu": refresh_tflops / alu_tflops,
                    "tflops_tf32_issued": token_heads * 163840 / (t_refresh * 1e-3) / 1e12,
                    "tf32_peak": 0.489 * tf,
                    "frac_of_tf32_tensor": token_heads * 163840 / (t_refresh * 1e-3) / 1e12 / (0.489 * tf)},
    }
    dominant = max((("pack", t_pack), ("restore", t_restore), ("refresh", t_refresh)), key=lambda x: x[1])[0]
    roofline = dict(rl[dominant])
    roofline["kernel"] = dominant
    line = {
        "metric": "pack_restore_GBps", "value": world * (pack_bytes + restore_bytes) / ((t_pack + t_restore) * 1e-3) / 1e9,
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_total,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": L, "heads": H, "d_k": D, "d_v": D, "requests": N_REQ,
                   "keep_ratio": KEEP, "suffix_tokens": SUFFIX, "refresh_algo": args.algo,
                   "l2": "inputs larger than L2 (3 GiB of states, 19 GB of token streams per step)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "ms": {"pack": t_pack, "restore": t_restore, "refresh": t_refresh},
        "pack_GBps": world * pack_gbs, "restore_GBps": world * restore_gbs,
        "refresh_tokens_per_s": world * N_REQ * SUFFIX / (t_refresh * 1e-3),
        "refresh_token_heads_per_s": world * token_heads / (t_refresh * 1e-3),
        "roofline": roofline, "roofline_by_kernel": rl, "clocks": clocks, "gpu_launches": 3 * args.steps,
    }
    if e2e:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = {k2: v2 for k2, v2 in oracle_leg().items() if k2 != "seconds"}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
