#!/usr/bin/env python
"""Benchmark of the DASC hot path on B200: one step = pack -> restore (zero-fill) ->
suffix refresh over one batch of synthetic state checkpoints.

Default workload (N=1, the one the driver times): the serving-scale KDA configuration --
24 KDA layers x 32 heads x 128x128 fp32 states (2 MiB per layer and request), 64 requests,
per-channel decay rates log-uniform in [1e-3, 1] (seed 1), keep ratio 0.38 per layer --
followed by a refresh of a 256-token bf16 suffix per request.  Inputs are far larger than
L2, so no flush is needed.

Prints ONE JSON line.  `value` is pack+restore algorithmic GB/s (bytes the two copies must
move / their device time); refresh throughput, per-kernel rooflines, the end-to-end leg
(host buffers, copies timed) and the CPU oracle baseline ride along in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Other configurations (not the default line; used to fill the results table):
    --config 2            GDN head-wise, 36 layers, 32/16 heads, 128 requests, keep 0.5
    --config 3 --suffix S aggressive KDA, keep 0.2, batch 32, suffix 256 / 1024 / 4096
    --config 4            mixed serving trace: pack on one stream, restore+refresh on another
    --keep R              keep ratio of the sweep {0.25, 0.38, 0.5, 1.0} for --config 1
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

D = 128
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TF32_OVER_BF16 = 0.489        # nominal dense 1.1 : 2.25
CHUNKED_FLOPS_PER_TOKEN_HEAD = 196608   # tf32 flops the chunked kernel issues per (token, head): 32-token chunks,
                                        # MMA1 padded to M = 128, hi/lo pairs in MMA3, MMA4 and MMA5

# Traffic of a launch over its algorithmic bytes, from one ncu capture of the KDA serving workload at 8 requests and a
# 128-token suffix (a full-size launch is too large to capture; every request and token moves the same bytes, so traffic
# grows in proportion and a full launch is scaled by its units).  Traffic = dram__bytes_read.sum + 32 B x
# lts__t_sectors_srcunit_tex_op_write.sum (the sectors the SMs wrote into L2): the DRAM write counter alone misses the
# lines still dirty in the 126 MB L2 when the kernel ends (a third of the pack's writes at this size), and
# lts__t_sectors_op_write.sum counts a sector once more when its home L2 slice is on the other die (1.5000x the
# algorithmic write bytes for all three kernels).  profiles/traffic_kda_serving.md has the numbers.
NCU_CAPTURE = {  # kernel: (dram__bytes_read.sum, lts__t_sectors_srcunit_tex_op_write.sum, algorithmic bytes of that launch)
    "pack": (153370624, 4783104, 306118656),
    "restore": (153463296, 12582912, 555712512),
    "refresh_chunked": (1412594688, 18874368, 2016411648),
}
NCU_TRAFFIC_OVER_ALGORITHMIC = {k: (rd + 32 * wr) / alg for k, (rd, wr, alg) in NCU_CAPTURE.items()}

CONFIGS = {
    1: dict(name="kda_serving", kind="KDA", L=24, H_v=32, H_k=32, n_req=64, keep=0.38, rate_lo=1e-3, suffix=256, seed=1),
    2: dict(name="gdn_headwise", kind="GDN", L=36, H_v=32, H_k=16, n_req=128, keep=0.5, rate_lo=1e-4, suffix=256, seed=2),
    3: dict(name="kda_aggressive", kind="KDA", L=24, H_v=32, H_k=32, n_req=32, keep=0.2, rate_lo=1e-3, suffix=256, seed=3),
    4: dict(name="mixed_trace", kind="KDA", L=24, H_v=32, H_k=32, n_req=64, keep=0.38, rate_lo=1e-3, suffix=1024, seed=4),
}


def workload_name(c):
    codec = "_int8pool" if c.get("codec") == "int8" else ""
    return (f"{c['name']}_{c['L']}x{c['H_v']}x{D}x{D}_fp32_{c['n_req']}req_keep{c['keep']}_suffix{c['suffix']}_bf16"
            f"{codec}")


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

def oracle_leg(c, sample_req=4, sample_units=64):
    """Times the fp64 oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    from paper_2608_30386_b200 import synth

    kda = c["kind"] == "KDA"
    okind = oracle.KDA if kda else oracle.GDN
    L, H_v, H_k = c["L"], c["H_v"], c["H_k"]
    uph = D if kda else 1
    gen = synth.generator(c["seed"])
    rates = synth.skew_layers(synth.decay_rates(gen, L, H_v, uph, c["rate_lo"], 1.0), c.get("layer_skew", 0.0))
    A_log, dt = synth.decay_params(rates)
    unit_words = D if kda else D * D
    oplan = oracle.plan(okind, L, H_v, uph, A_log.numpy(), dt.numpy(), sel=oracle.SEL_TOP_RATIO,
                        keep_ratio=c["keep"], unit_bytes=unit_words * 4,
                        scope=oracle.SCOPE_MODEL if c.get("scope") == "model" else oracle.SCOPE_LAYER)
    dense = H_v * D * D
    state = synth.states(gen, (sample_req, L, dense)).numpy()
    slot = oplan.sum_r * unit_words
    pool = np.zeros((sample_req, slot), np.float32)
    out = np.empty_like(state)
    ids = np.arange(sample_req, dtype=np.int32)
    int8 = c.get("codec") == "int8"
    slot_bytes = slot // D * (D + 4) if int8 else slot * 4
    t0 = time.perf_counter()
    oracle.pack(oplan.mask, unit_words, state, dense, L * dense, ids, pool, slot, ids)
    if int8:
        codes, scales = oracle.int8_quantize(pool.reshape(-1, D))
    t1 = time.perf_counter()
    if int8:
        pool = oracle.int8_dequantize(codes, scales).reshape(sample_req, slot)
    oracle.restore(oplan.mask, unit_words, pool, slot, ids, out, dense, L * dense, ids)
    t2 = time.perf_counter()
    pack_bytes = sample_req * (slot * 4 + slot_bytes)
    restore_bytes = sample_req * (slot_bytes + L * dense * 4)
    # refresh sample: whole layers of one request (sample_units (request, layer, head) units), 256 tokens
    Ls = max(1, sample_units // H_v)
    n_tok = min(c["suffix"], 256)
    streams = synth.token_streams(gen, synth.KDA if kda else synth.GDN, Ls, n_tok, H_v, H_k, D, D, rates[:Ls])
    st = synth.states(gen, (1, Ls, H_v, D, D)).numpy()
    threads = oracle.max_threads()
    t3 = time.perf_counter()
    oracle.refresh(okind, Ls, H_v, H_k, D, D, st, dense, Ls * dense, [0], synth.bf16_bits(streams.q),
                   synth.bf16_bits(streams.k), synth.bf16_bits(streams.v), streams.g.numpy(), streams.beta.numpy(),
                   [0, n_tok], n_threads=threads)
    t4 = time.perf_counter()
    token_heads = Ls * H_v * n_tok
    return {
        "value": (pack_bytes + restore_bytes) / (t2 - t0) / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
        "sample": (f"pack+restore of {sample_req} of {c['n_req']} requests (one thread); refresh of {Ls * H_v} of "
                   f"{c['n_req'] * L * H_v} (request,layer,head) units x {n_tok} tokens on {threads} threads"),
        "pack_GBps": pack_bytes / (t1 - t0) / 1e9, "restore_GBps": restore_bytes / (t2 - t1) / 1e9,
        # tokens/s of the full model (all layers and heads per token), extrapolated from the sampled units
        "refresh_tokens_per_s": token_heads / (t4 - t3) / (L * H_v),
        "refresh_token_heads_per_s": token_heads / (t4 - t3),
        "seconds": t4 - t0,
    }


def run_reference(args, c):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    vals, leg = [], None
    for i in range(args.warmup + args.steps):
        leg = oracle_leg(c, sample_req=2, sample_units=32)
        if i >= args.warmup:
            vals.append(leg)
    value = statistics.mean(v["value"] for v in vals)
    sec = statistics.mean(v["seconds"] for v in vals)
    print(json.dumps({
        "impl": "reference", "metric": "pack_restore_GBps", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(c), "note": "CPU oracle on a bounded sample of the workload per step"},
        "refresh_tokens_per_s": statistics.mean(v["refresh_tokens_per_s"] for v in vals),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": leg["cores"], "kind": "oracle", "sample": leg["sample"]},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ----------------------------------------------------------------------------------------------
# GPU legs
# ----------------------------------------------------------------------------------------------

def build_plan(c, device):
    import paper_2608_30386_b200 as dasc
    from paper_2608_30386_b200 import synth
    kda = c["kind"] == "KDA"
    gen = synth.generator(c["seed"])
    rates = synth.skew_layers(synth.decay_rates(gen, c["L"], c["H_v"], D if kda else 1, c["rate_lo"], 1.0),
                              c.get("layer_skew", 0.0))
    A_log, dt = synth.decay_params(rates)
    kind = dasc.KDA if kda else dasc.GDN
    if c.get("mixed_heads") and kda:
        # Every head draws its own keep ratio from the sweep's set, so the per-head channel counts are ragged by
        # construction.  The selection itself stays in the library: one head-scope plan per ratio (host only), and each
        # head takes the mask of the plan with its ratio; the union goes in as an explicit mask.
        ratios = (0.25, 0.38, 0.5, 1.0)
        masks = [dasc.dasc_plan(kind, c["L"], c["H_v"], c["H_k"], D, D, A_log.numpy(), dt.numpy(), sel=dasc.SEL_TOP_RATIO,
                                scope=dasc.SCOPE_HEAD, keep_ratio=r, device=-1).mask().reshape(c["L"], c["H_v"], D)
                 for r in ratios]
        pick = torch.randint(0, len(ratios), (c["L"], c["H_v"]), generator=gen).numpy()
        mask = np.choose(pick[:, :, None], masks)
        plan = dasc.dasc_plan(kind, c["L"], c["H_v"], c["H_k"], D, D, A_log.numpy(), dt.numpy(), sel=dasc.SEL_EXPLICIT,
                              explicit_mask=mask.reshape(c["L"], -1), device=device)
        return plan, rates, gen
    plan = dasc.dasc_plan(kind, c["L"], c["H_v"], c["H_k"], D, D, A_log.numpy(), dt.numpy(),
                          sel=dasc.SEL_TOP_RATIO, scope=dasc.SCOPE_MODEL if c.get("scope") == "model" else dasc.SCOPE_LAYER,
                          keep_ratio=c["keep"], device=device)
    return plan, rates, gen


def max_over_ranks(values, device):
    """Replicas only: every rank times its own identical share of the work, and the job's time is the slowest rank's.
    Element-wise maximum of `values` over the ranks of the default process group (the values themselves when no
    group is initialised)."""
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job(per_rank_units: float, world: int, ms: float) -> float:
    """Weak scaling: every rank processes `per_rank_units` in `ms` milliseconds (the maximum over ranks)."""
    return world * per_rank_units / (ms * 1e-3)


def token_bytes_per_head(kda: bool, H_v: int, H_k: int) -> float:
    """Algorithmic bytes per (token, value head): q + k (shared by H_v/H_k value heads) + v bf16, g fp32, beta, o bf16."""
    share = H_k / H_v
    return 2 * D * 2 * share + D * 2 + (D * 4 if kda else 4) + 4 + D * 2


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dasc", choices=["dasc", "reference"])
    ap.add_argument("--algo", default="auto", choices=["auto", "sequential", "chunked"])
    ap.add_argument("--config", type=int, default=1, choices=sorted(CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--requests", type=int, default=None, help="profiling only: shrink the batch")
    ap.add_argument("--suffix", type=int, default=None, help="refresh suffix length (config 3: 256, 1024, 4096)")
    ap.add_argument("--keep", type=float, default=None, help="keep ratio (0.25, 0.38, 0.5, 1.0 in the sweep)")
    ap.add_argument("--layer-group", type=int, default=None, help="layers of token streams resident at once")
    ap.add_argument("--layout", default="ragged", choices=["ragged", "padded"],
                    help="checkpoint pool layout (Appendix B): ragged [slots][sum r_l] or padded [L][slots][R_max]")
    ap.add_argument("--scope", default="layer", choices=["layer", "model"],
                    help="selection scope of the keep ratio; 'model' makes per-layer counts differ (padding appears)")
    ap.add_argument("--mixed-heads", action="store_true",
                    help="every head draws its own keep ratio from {0.25, 0.38, 0.5, 1.0} (ragged per-head channel counts)")
    ap.add_argument("--layer-skew", type=float, default=0.0,
                    help="imbalanced per-layer decay profile: layer rates scaled by exp(skew * (l/(L-1) - 1/2))")
    ap.add_argument("--codec", default="fp32", choices=["fp32", "int8"],
                    help="checkpoint pool format: fp32 bit copies, or the Appendix D INT8 codec fused into pack/restore")
    ap.add_argument("--pool-slots", type=int, default=2048, help="config 4: slots of the bounded checkpoint pool")
    ap.add_argument("--trace-rounds", type=int, default=0, help="config 4: replay only the first rounds of the trace")
    ap.add_argument("--tp-ranks", type=int, default=8, help="virtual TP ranks of the placement leg (0 or 1 = skip it)")
    ap.add_argument("--dry-launch", action="store_true", help="start the ranks, count them over gloo, do no GPU work")
    args = ap.parse_args()
    world_env = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world_env == 1 and "DASC_BENCH_SPAWNED" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))                 # no launcher around us: start the N ranks ourselves
    if args.gpus != world_env:
        raise SystemExit(f"--gpus {args.gpus} does not match the {world_env} rank(s) that were launched")
    if args.dry_launch:
        dry_launch(args)
        return
    c = dict(CONFIGS[args.config])
    if args.requests is not None:
        c["n_req"] = args.requests
    if args.suffix is not None:
        c["suffix"] = args.suffix
    if args.keep is not None:
        c["keep"] = args.keep
    c["codec"] = args.codec
    c["scope"] = args.scope
    c["layer_skew"] = args.layer_skew
    c["mixed_heads"] = args.mixed_heads
    if args.impl == "reference":
        run_reference(args, c)
        return
    args.warmup = max(args.warmup, 3)
    if args.config == 4:
        run_mixed_trace(args, c)
        return

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
    kda = c["kind"] == "KDA"
    L, H_v, H_k, N_REQ, SUFFIX = c["L"], c["H_v"], c["H_k"], c["n_req"], c["suffix"]

    # ---- plan and inputs (replicas: every rank holds the same shape of work, its own seed) ----
    plan, rates, gen = build_plan(c, local)
    dense = H_v * D * D
    layer_stride, req_stride = N_REQ * dense, dense          # layer-major active-state pool
    dgen = synth.generator(c["seed"] + 1000 * rank, dev)
    state = synth.states(dgen, (L, N_REQ, dense), dev)
    active = torch.empty_like(state)
    slot = int(plan.slot_floats)
    int8 = args.codec == "int8"
    # bytes of one checkpoint slot in the pool: fp32 rows, or int8 codes + one fp32 scale per row
    slot_bytes = dasc.dasc_int8_slot_bytes(plan) if int8 else slot * 4
    pool = torch.empty((N_REQ, slot_bytes), dtype=torch.uint8, device=dev) if int8 else torch.empty((N_REQ, slot), device=dev)
    do_pack = dasc.dasc_pack_int8 if int8 else dasc.dasc_pack
    do_restore = dasc.dasc_restore_int8 if int8 else dasc.dasc_restore
    if args.layout == "padded":                                # Appendix B, Scheme 1: [L][slots][R_max][unit]
        if int8:
            raise SystemExit("--layout padded is an fp32 layout")
        pool = torch.empty(dasc.dasc_padded_pool_floats(plan, N_REQ), device=dev)

        def do_pack(plan, state, ls, rs, src, pool, dst):
            dasc.dasc_pack_padded(plan, state, ls, rs, src, pool, int(dst.numel()), dst)

        def do_restore(plan, pool, src, state, ls, rs, dst):
            dasc.dasc_restore_padded(plan, pool, int(src.numel()), src, state, ls, rs, dst)
    ids = torch.arange(N_REQ, dtype=torch.int32, device=dev)
    slots = torch.randperm(N_REQ, generator=gen).to(torch.int32).to(dev)
    T = N_REQ * SUFFIX
    # token streams: `group` layers resident at once; when that is fewer than all layers the same
    # buffers are replayed for every layer group (bounds memory; the work per group is identical)
    per_layer = T * (2 * H_k * D * 2 + 2 * H_v * D * 2 + H_v * (D if kda else 1) * 4 + H_v * 4)
    group = args.layer_group or max(1, min(L, int(40e9 // per_layer)))
    while L % group:
        group -= 1
    skind = synth.KDA if kda else synth.GDN
    parts = [synth.token_streams(dgen, skind, 1, T, H_v, H_k, D, D, rates[l:l + 1], device=dev) for l in range(group)]
    q, k, v, g, beta = (torch.cat([getattr(p, f) for p in parts]) for f in ("q", "k", "v", "g", "beta"))
    del parts
    o = torch.empty((group, T, H_v, D), dtype=torch.bfloat16, device=dev)
    cu = synth.uniform_cu_seqlens(N_REQ, SUFFIX).to(dev)
    ws_bytes = dasc.dasc_refresh_workspace_bytes(plan, N_REQ, group, algo)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None

    pack_bytes = N_REQ * (slot * 4 + slot_bytes)
    restore_bytes = N_REQ * (slot_bytes + L * dense * 4)
    token_heads = N_REQ * L * H_v * SUFFIX
    refresh_bytes = token_heads * token_bytes_per_head(kda, H_v, H_k) + 2 * N_REQ * L * dense * 4  # + state in and out
    refresh_flops_min = token_heads * 7 * D * D              # token-by-token recurrence, incl. decay and read-out
    n_groups = L // group

    stream = torch.cuda.current_stream()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        do_pack(plan, state, layer_stride, req_stride, ids, pool, slots)
        if ev:
            ev[1].record(stream)
        do_restore(plan, pool, slots, active, layer_stride, req_stride, ids)
        if ev:
            ev[2].record(stream)
        for gi in range(n_groups):
            dasc.dasc_refresh(plan, active, layer_stride, req_stride, ids, q, k, v, g, beta, cu, T, SUFFIX,
                              layer_begin=gi * group, layer_end=(gi + 1) * group, o=o, algo=algo, workspace=ws)
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
    t_pack, t_restore, t_refresh, t_total = max_over_ranks([t_pack, t_restore, t_refresh, t_total], dev)

    # ---- the paper's own load policy (Section 4.2): replay the last W tokens from a zero scratch state, merge the
    #      omitted units, no outputs (state-only fast path).  Same streams, W = the suffix length. ----
    wb = torch.empty(N_REQ, dtype=torch.int32, device=dev)

    def window_step():
        for gi in range(n_groups):
            dasc.dasc_refresh_window(plan, active, layer_stride, req_stride, ids, None, k, v, g, beta, cu, T, wb,
                                     window=SUFFIX, layer_begin=gi * group, layer_end=(gi + 1) * group, algo=algo,
                                     workspace=ws)

    for _ in range(3):
        window_step()
    barrier()
    ev_w = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev_w[0].record(stream)
    for _ in range(args.steps):
        window_step()
    ev_w[1].record(stream)
    barrier()
    assert dasc.dasc_refresh_status(ws) == 0
    (t_window,) = max_over_ranks([ev_w[0].elapsed_time(ev_w[1]) / args.steps], dev)

    # ---- Section 4.3 on the device: the same Store / Load with TP-balanced placement, timed apart from the step.
    #      Eight virtual ranks (eight pool buffers on this GPU, as peer mappings would appear to one rank); this rank
    #      holds the heaviest payload, so most of its units are pushed into the other ranks' pools. ----
    tp = None
    if args.layout == "ragged" and not int8 and args.tp_ranks > 1:
        Tn = args.tp_ranks
        U = np.full(Tn, int(plan.units_retained) // 4, np.int64)
        U[0] = int(plan.units_retained)
        width, _ = dasc.dasc_tp_balance(U)
        tp_pools = [torch.empty((N_REQ, width * int(plan.unit_floats)), device=dev) for _ in range(Tn)]
        for _ in range(3):
            dasc.dasc_pack_tp(plan, state, layer_stride, req_stride, ids, tp_pools, U, 0, slots)
            dasc.dasc_restore_tp(plan, tp_pools, U, 0, slots, active, layer_stride, req_stride, ids)
        barrier()
        ev_t = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        n_it = 5
        ev_t[0].record(stream)
        for _ in range(n_it):
            dasc.dasc_pack_tp(plan, state, layer_stride, req_stride, ids, tp_pools, U, 0, slots)
        ev_t[1].record(stream)
        for _ in range(n_it):
            dasc.dasc_restore_tp(plan, tp_pools, U, 0, slots, active, layer_stride, req_stride, ids)
        ev_t[2].record(stream)
        barrier()
        t_ptp, t_rtp = max_over_ranks([ev_t[0].elapsed_time(ev_t[1]) / n_it, ev_t[1].elapsed_time(ev_t[2]) / n_it], dev)
        tp = {"virtual_ranks": Tn, "units_per_rank": U.tolist(), "slot_width_units": width,
              "pack_tp_GBps": pack_bytes / (t_ptp * 1e-3) / 1e9, "restore_tp_GBps": restore_bytes / (t_rtp * 1e-3) / 1e9,
              "ms_pack_tp": t_ptp, "ms_restore_tp": t_rtp,
              "note": "all pools local to this GPU (one GPU in this run): the figures show the cost of the placement "
                      "arithmetic, not of NVLink"}
        del tp_pools

    # ---- end-to-end leg: host buffers, copies inside the timed region -------------------------
    e2e = None
    if not args.no_e2e:
        n_e = min(16, N_REQ)                                 # requests per e2e step (bounded pinned memory)
        Te = n_e * SUFFIX
        ge = min(group, 6)                                   # layers of token streams copied per refresh call
        # request-major on both sides, so that a group of requests is one contiguous transfer
        h_state = torch.empty((n_e, L, dense), dtype=torch.float32).pin_memory()
        h_state.copy_(state[:, :n_e].transpose(0, 1))
        host_streams = [x[:ge, :Te].contiguous().cpu().pin_memory() for x in (q, k, v, g, beta)]
        pool_shape, pool_dtype = ((n_e, slot_bytes), torch.uint8) if int8 else ((n_e, slot), torch.float32)
        h_pool = torch.empty(pool_shape, dtype=pool_dtype).pin_memory()
        h_out = torch.empty((n_e, L, dense), dtype=torch.float32).pin_memory()
        h_o = torch.empty((ge, Te, H_v, D), dtype=torch.bfloat16).pin_memory()
        d_state = torch.empty((n_e, L, dense), device=dev)
        d_active = torch.empty_like(d_state)
        d_pool = torch.empty(pool_shape, dtype=pool_dtype, device=dev)
        d_streams = [torch.empty(x.shape, dtype=x.dtype, device=dev) for x in host_streams]
        d_o = torch.empty((ge, Te, H_v, D), dtype=torch.bfloat16, device=dev)
        cu_e = synth.uniform_cu_seqlens(n_e, SUFFIX).to(dev)
        ids_e = torch.arange(n_e, dtype=torch.int32, device=dev)
        ls_e, rs_e = dense, L * dense
        # Store / Load in `parts` groups of requests: group i's pool goes back to the host on a second stream while
        # group i+1's states are still coming in (PCIe carries both directions at once)
        parts = 4 if (args.layout == "ragged" and n_e % 4 == 0) else 1
        s_out = torch.cuda.Stream(device=dev)
        part_done = [torch.cuda.Event() for _ in range(parts)]
        out_done = torch.cuda.Event()
        part_ids = [ids_e[i * (n_e // parts):(i + 1) * (n_e // parts)].contiguous() for i in range(parts)]

        def e2e_step(ev):
            ev[0].record(stream)
            s_out.wait_stream(stream)                          # the previous step has let go of the pool buffers
            for i in range(parts):
                a0, a1 = i * (n_e // parts), (i + 1) * (n_e // parts)
                d_state[a0:a1].copy_(h_state[a0:a1], non_blocking=True)
                do_pack(plan, d_state, ls_e, rs_e, part_ids[i], d_pool, part_ids[i])
                do_restore(plan, d_pool, part_ids[i], d_active, ls_e, rs_e, part_ids[i])
                part_done[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(part_done[i])
                    h_pool[a0:a1].copy_(d_pool[a0:a1], non_blocking=True)
            with torch.cuda.stream(s_out):
                out_done.record(s_out)
            stream.wait_event(out_done)
            ev[1].record(stream)
            for gi in range(L // ge):                        # every layer group: its streams in, its outputs out
                for dst, src in zip(d_streams, host_streams):
                    dst.copy_(src, non_blocking=True)
                dasc.dasc_refresh(plan, d_active, ls_e, rs_e, ids_e, *d_streams, cu_e, Te, SUFFIX,
                                  layer_begin=gi * ge, layer_end=(gi + 1) * ge, o=d_o, algo=algo, workspace=ws)
                h_o.copy_(d_o, non_blocking=True)
            h_out.copy_(d_active, non_blocking=True)
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
        t_copy, t_ref = max_over_ranks([t_copy, t_ref], dev)
        e_bytes = n_e * (slot * 4 + slot_bytes) + n_e * (slot_bytes + L * dense * 4)
        h2d = h_state.numel() * 4 + (L // ge) * sum(x.numel() * x.element_size() for x in host_streams)
        d2h = h_pool.numel() * h_pool.element_size() + h_out.numel() * 4 + (L // ge) * h_o.numel() * 2
        e2e = {"value": world * e_bytes / (t_copy * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "requests_per_step": n_e,
               "refresh_tokens_per_s": world * Te / (t_ref * 1e-3), "ms_pack_restore": t_copy, "ms_refresh": t_ref,
               "note": "pinned host buffers; H2D of states and token streams, D2H of pool, states and outputs timed; "
                       "Store/Load in request groups, a group's pool read back while the next group uploads"}
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
    tf32_issued = token_heads * CHUNKED_FLOPS_PER_TOKEN_HEAD / (t_refresh * 1e-3) / 1e12
    rl = {
        "pack": {"bound": "hbm", "achieved": pack_gbs, "peak": hbm, "unit": "GB/s", "frac": pack_gbs / hbm,
                 "traffic": None, "peak_source": src, "frac_of_8TBps_nominal": pack_gbs / 8000.0},
        "restore": {"bound": "hbm", "achieved": restore_gbs, "peak": hbm, "unit": "GB/s", "frac": restore_gbs / hbm,
                    "traffic": None, "peak_source": src, "frac_of_8TBps_nominal": restore_gbs / 8000.0},
        # By the arithmetic (about 100 flop per byte, below the ridge) HBM is the ceiling of the refresh;
        # the tensor-pipe figures beside it: tf32 flops the chunked kernel issues against the tf32 peak
        # taken as 0.489 x the measured sustained bf16 peak (nominal 1.1 : 2.25).
        "refresh": {"bound": "hbm", "achieved": refresh_gbs, "peak": hbm, "unit": "GB/s", "frac": refresh_gbs / hbm,
                    "traffic": None, "peak_source": src, "tflops_min_form": refresh_tflops,
                    "frac_of_fp32_alu": refresh_tflops / alu_tflops, "tflops_tf32_issued": tf32_issued,
                    "tf32_peak": TF32_OVER_BF16 * tf, "frac_of_tf32_tensor": tf32_issued / (TF32_OVER_BF16 * tf),
                    # the token-by-token minimum (7 d_k d_v flop per token-head) against the same tensor peak
                    "frac_useful_of_tf32_tensor": refresh_tflops / (TF32_OVER_BF16 * tf)},
    }
    if c["name"] == "kda_serving" and not int8:      # the workload the capture was made on
        rl["pack"]["traffic"] = NCU_TRAFFIC_OVER_ALGORITHMIC["pack"] * pack_bytes
        rl["restore"]["traffic"] = NCU_TRAFFIC_OVER_ALGORITHMIC["restore"] * restore_bytes
        if args.algo != "sequential":       # auto picks the chunked kernel for this shape
            rl["refresh"]["traffic"] = NCU_TRAFFIC_OVER_ALGORITHMIC["refresh_chunked"] * refresh_bytes / n_groups
    rl["refresh"]["launches_per_step"] = n_groups
    rl["refresh"]["algorithmic_bytes_per_launch"] = refresh_bytes / n_groups
    rl["pack"]["algorithmic_bytes_per_launch"] = pack_bytes
    rl["restore"]["algorithmic_bytes_per_launch"] = restore_bytes
    dominant = max((("pack", t_pack), ("restore", t_restore), ("refresh", t_refresh)), key=lambda x: x[1])[0]
    roofline = dict(rl[dominant])
    roofline["kernel"] = dominant
    line = {
        "metric": "pack_restore_GBps", "value": whole_job(pack_bytes + restore_bytes, world, t_pack + t_restore) / 1e9,
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_total,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(c), "kind": c["kind"], "layers": L, "v_heads": H_v, "k_heads": H_k, "d_k": D,
                   "d_v": D, "requests": N_REQ, "keep_ratio": c["keep"], "codec": args.codec, "layout": args.layout,
                   "selection_scope": "mixed per-head ratios" if args.mixed_heads else args.scope,
                   "units_retained_fraction": plan.units_retained / plan.units_total,
                   "pool_bytes": pool.numel() * pool.element_size(), "suffix_tokens": SUFFIX, "refresh_algo": args.algo,
                   "stream_layers_resident": group,
                   "l2": "inputs larger than L2 (GiBs of states and token streams per step); no flush needed",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "ms": {"pack": t_pack, "restore": t_restore, "refresh": t_refresh},
        "pack_GBps": world * pack_gbs, "restore_GBps": world * restore_gbs,
        "refresh_tokens_per_s": world * N_REQ * SUFFIX / (t_refresh * 1e-3),
        "refresh_token_heads_per_s": world * token_heads / (t_refresh * 1e-3),
        # Eq. 6 / Appendix B on this plan: temporal bytes of one checkpoint per layout and the layout gain R_max / mean r_l
        "capacity": {
            "layer_skew": args.layer_skew,
            "bytes_dense": dasc.dasc_checkpoint_bytes(plan, dasc.LAYOUT_DENSE),
            "bytes_padded": dasc.dasc_checkpoint_bytes(plan, dasc.LAYOUT_PADDED),
            "bytes_ragged": dasc.dasc_checkpoint_bytes(plan, dasc.LAYOUT_RAGGED),
            "bytes_ragged_int8": dasc.dasc_int8_slot_bytes(plan),
            "c_temp_pad": plan.c_temp_pad, "c_temp_rag": plan.c_temp_rag,
            "layout_gain_rmax_over_rbar": plan.c_temp_rag / plan.c_temp_pad if plan.units_retained else None,
        },
        # dasc_refresh_window: scratch replay of the last `suffix_tokens` tokens, merge of omitted units, no outputs
        "window_refresh_state_only": {"ms": t_window, "tokens_per_s": world * N_REQ * SUFFIX / (t_window * 1e-3),
                                      "token_heads_per_s": world * token_heads / (t_window * 1e-3)},
        "roofline": roofline, "roofline_by_kernel": rl, "clocks": clocks,
        # per step: pack, restore, and per layer group the tensor-core refresh kernel + the exact kernel's pass over
        # the units handed to it (AUTO); a single refresh kernel per group when an algorithm is forced
        "gpu_launches": (2 + n_groups * (2 if args.algo == "auto" else 1)) * args.steps,
    }
    if tp:
        line["tp_placement"] = tp
    if e2e:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1 and not args.mixed_heads:  # the oracle leg times the per-layer rule
        line["cpu_baseline"] = {k2: v2 for k2, v2 in oracle_leg(c).items() if k2 != "seconds"}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def run_mixed_trace(args, c):
    """Mixed serving trace (single GPU; Appendix C.1: a bounded pool of checkpoint slots with LRU recycling).

    The event list comes from `synth.serving_trace` (seed 4): 512 requests with prefix lengths log-uniform in
    [1 Ki, 128 Ki], one checkpoint stored every 1024 tokens, follow-up requests that hit the newest resident
    checkpoint of a shared prefix and replay the 1..1024 tokens since it.  The list is cut into rounds whose two
    sides are independent: new checkpoints are packed on one stream (the higher-priority one) while hits are restored
    and refreshed (ragged suffixes) on another.  A step is one replay of the whole trace; it is timed with the
    two streams overlapped and with each round's two sides run one after the other.  Checkpoint contents and token
    values do not affect the time: the states of a round's new checkpoints and the token streams are fixed synthetic
    buffers (six layers of streams resident, reused by every layer group and round)."""
    import paper_2608_30386_b200 as dasc
    from paper_2608_30386_b200 import synth

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    L, H, batch = c["L"], c["H_v"], c["n_req"]
    n_slots = args.pool_slots
    plan, rates, gen = build_plan(c, local)
    rounds, tstats = synth.serving_trace(c["seed"], n_slots=n_slots, batch=batch)
    if args.trace_rounds:
        rounds = rounds[:args.trace_rounds]
    dense = H * D * D
    ls, rs = batch * dense, dense
    slot = int(plan.slot_floats)
    dgen = synth.generator(c["seed"], dev)
    pool = torch.empty((n_slots, slot), device=dev)
    pool.normal_(generator=dgen)
    new_states = synth.states(dgen, (L, batch, dense), dev)
    active = torch.empty((L, batch, dense), device=dev)
    ids = torch.arange(batch, dtype=torch.int32, device=dev)
    t_max = max(max(sum(r.suffix) for r in rounds), 1)
    group = 6                                                          # layers of token streams resident at once
    parts = [synth.token_streams(dgen, synth.KDA, 1, t_max, H, H, D, D, rates[l:l + 1], device=dev) for l in range(group)]
    q, k, v, g, beta = (torch.cat([getattr(p, f) for p in parts]) for f in ("q", "k", "v", "g", "beta"))
    del parts
    o = torch.empty((group, t_max, H, D), dtype=torch.bfloat16, device=dev)
    ws = torch.zeros(dasc.dasc_refresh_workspace_bytes(plan, batch, group), dtype=torch.uint8, device=dev)
    # the copy stream gets the higher priority: its blocks are placed as soon as a refresh CTA retires
    lo_pri, hi_pri = torch.cuda.Stream.priority_range() if hasattr(torch.cuda.Stream, "priority_range") else (0, -1)
    s_pack = torch.cuda.Stream(priority=hi_pri)
    s_load = torch.cuda.Stream(priority=lo_pri)
    dev_rounds = []
    for r in rounds:
        cu = torch.zeros(len(r.suffix) + 1, dtype=torch.int64)
        cu[1:] = torch.cumsum(torch.tensor(r.suffix, dtype=torch.int64), 0) if r.suffix else cu[1:]
        dev_rounds.append((torch.tensor(r.store_slots, dtype=torch.int32, device=dev),
                           torch.tensor(r.hit_slots, dtype=torch.int32, device=dev), cu.to(torch.int32).to(dev),
                           max(r.suffix) if r.suffix else 0))
    launches = 0

    def store_side(i):
        nonlocal launches
        slots = dev_rounds[i][0]
        n = int(slots.numel())
        if n:
            dasc.dasc_pack(plan, new_states, ls, rs, ids[:n], pool, slots, stream=s_pack)
            launches += 1

    def load_side(i):
        nonlocal launches
        _, hits, cu, longest = dev_rounds[i]
        n = int(hits.numel())
        if not n:
            return
        dasc.dasc_restore(plan, pool, hits, active, ls, rs, ids[:n], stream=s_load)
        launches += 1
        for gi in range(L // group):       # the streams hold t_max tokens per layer; the call sees this round's first T
            dasc.dasc_refresh(plan, active, ls, rs, ids[:n], q, k, v, g, beta, cu, t_max, longest,
                              layer_begin=gi * group, layer_end=(gi + 1) * group, o=o, workspace=ws, stream=s_load)
            launches += 2

    def replay(overlap):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        main = torch.cuda.current_stream()
        ev0.record(main)
        s_pack.wait_event(ev0)
        s_load.wait_event(ev0)
        for i in range(len(rounds)):
            store_side(i)
            if not overlap:
                s_load.wait_stream(s_pack)
            load_side(i)
            # a round's two sides are independent of each other, consecutive rounds are not
            s_pack.wait_stream(s_load)
            s_load.wait_stream(s_pack)
        main.wait_stream(s_pack)
        main.wait_stream(s_load)
        ev1.record(main)
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1)

    steps = max(1, min(args.steps, 3))
    replay(True)                                                       # warm-up: one whole trace
    sampler = ClockSampler(local)
    sampler.start()
    launches = 0
    t_overlap = sum(replay(True) for _ in range(steps)) / steps
    counted = launches // steps
    t_serial = sum(replay(False) for _ in range(steps)) / steps
    # each side alone, for the overlap bound: max(copy, load) <= overlapped <= copy + load
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    torch.cuda.synchronize()
    ev[0].record(s_pack)
    for i in range(len(rounds)):
        store_side(i)
    ev[1].record(s_pack)
    s_load.wait_event(ev[1])
    for i in range(len(rounds)):
        load_side(i)
    ev[2].record(s_load)
    torch.cuda.synchronize()
    t_store, t_load = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    clocks = sampler.stop()
    assert dasc.dasc_refresh_status(ws) == 0
    n_store = sum(len(r.store_slots) for r in rounds)
    n_hit = sum(len(r.hit_slots) for r in rounds)
    tokens = sum(sum(r.suffix) for r in rounds)
    copy_bytes = (2 * n_store * slot + n_hit * (slot + L * dense)) * 4
    print(json.dumps({
        "metric": "pack_restore_GBps", "value": copy_bytes / (t_overlap * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": 1,
        "steps": steps, "warmup": 1, "ms_per_step": t_overlap, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(c), "trace": {k2: v2 for k2, v2 in tstats.items()},
                   "rounds_replayed": len(rounds), "requests": 512, "prefix_tokens": "log-uniform in [1024, 131072]",
                   "checkpoint_interval_tokens": 1024, "pool_slots": n_slots, "pool_bytes": pool.numel() * 4,
                   "recycling": "least recently used (host side)", "round_batch": batch,
                   "suffix_tokens": "uniform in [1, 1024]", "streams": 2, "copy_stream_priority": hi_pri,
                   "note": "a step replays the whole trace; value counts pack+restore bytes over the overlapped step, "
                           "refresh included"},
        "ms_per_step_serial": t_serial, "overlap_speedup": t_serial / t_overlap,
        "ms_store_side_alone": t_store, "ms_load_side_alone": t_load,
        "checkpoints_stored": n_store, "hits_served": n_hit,
        "refresh_tokens_per_s": tokens / (t_overlap * 1e-3), "tokens_per_step": tokens, "clocks": clocks,
        "gpu_launches": counted * steps,
    }))


# ----------------------------------------------------------------------------------------------
# N > 1 without a launcher: this script starts its own ranks
# ----------------------------------------------------------------------------------------------

def spawn_replicas(n: int) -> int:
    """`python bench.py --gpus N` started by hand: run N ranks of this script (one process per GPU, rendezvous on
    127.0.0.1) and pass rank 0's JSON line through.  Returns the exit code (non-zero if any rank failed)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DASC_BENCH_SPAWNED="1")
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    codes = [p.wait() for p in procs]
    bad = [(r, code) for r, code in enumerate(codes) if code != 0]
    if bad:
        sys.stderr.write(f"bench.py: {len(bad)} of {n} ranks failed (rank, exit code): {bad}\n")
        return 1
    return 0


def dry_launch(args):
    """Launcher check that needs no GPU: every rank joins a gloo group and is counted."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    count = torch.ones(1, dtype=torch.int64)
    if world > 1:
        dist.all_reduce(count)
    if int(count.item()) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {int(count.item())} ranks ran")
    if rank == 0:
        print(json.dumps({"dry_launch": True, "n_gpus": args.gpus, "ranks": int(count.item())}))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
