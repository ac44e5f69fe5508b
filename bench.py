#!/usr/bin/env python
"""Benchmark of the replay-attention hot path (forward + merge + backward of one response
against a resident paged prefix) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload p2m] [--impl reference]

One "step" = one group member replayed against the resident prefix: ls_replay_attn_fwd,
ls_lse_merge, ls_replay_attn_bwd.  Prints ONE JSON line (rank 0).  With N > 1 every rank
holds its own replica of the prefix and replays different members: no collective on the
data path, weak scaling.  `--gpus N` without a torchrun environment starts the N ranks itself.

  --mode replay   forward (per-shard partials) + merge + backward              (default)
  --mode fused    forward with the merge folded in + backward
  --mode score    forward with the merge folded in only (a score-only pass)
  --mode dsa      sparse replay over the 576/512 latent (index scores, top-2048, attention fwd + bwd)
  --blocks B      blockwise replay of the response in B blocks with a paged suffix: a no-grad
                  suffix pass (score + append per block), then the blocks in reverse (pop,
                  forward, backward with gradient pages)
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_14952_b200 import replicas  # noqa: E402
from paper_2607_14952_b200 import workloads as W  # noqa: E402

METRIC = "replay_attn_fwd_bwd_tflops"
UNIT = "TFLOP/s"

DQ_KERNEL_NAME = {(256, 256): "bwd_dq3_kernel", (128, 128): "bwd_dq2_kernel", (576, 512): "bwd_mla_dq_kernel"}


def packed_tiles(cfg, tile_rows=128):
    """Number of Q tiles per KV group when the library packs rows of several heads into one Q tile (a
    response shorter than a tile, and fewer tiles that way), else 0: which kernels run depends on it."""
    g = cfg.Hq // cfg.Hkv
    if g <= 1 or cfg.R >= tile_rows:
        return 0
    bh = min(g, tile_rows)
    bt = min(cfg.R, tile_rows // bh)
    tiles = -(-cfg.R // bt) * -(-g // bh)
    return tiles if tiles < g else 0


def kernel_names(cfg):
    """(forward kernel, query-gradient kernel) the library launches for this workload: the single-CTA
    kernels when a KV group is one packed tile, the pair kernels otherwise (head dim 128: single CTAs)."""
    tiles = packed_tiles(cfg)
    fwd = "fwd2_kernel" if (cfg.Dk in (256, 576) and tiles != 1) else "fwd_kernel"
    dq = DQ_KERNEL_NAME.get((cfg.Dk, cfg.Dv))
    if cfg.Dk != 576 and tiles and (tiles == 1 or cfg.Dk != 256):
        dq = "bwd_dq1_kernel"
    return fwd, dq


def measured_traffic(kernel, workload):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` at `workload`, from the
    committed ncu capture records (a JSON list of {kernel, workload, dram_bytes_per_launch, ...});
    None when no capture of that kernel at that workload is on record."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        for rec in json.load(open(path)):
            if rec.get("kernel") == kernel and rec.get("workload") == workload:
                return rec.get("dram_bytes_per_launch")
    except (OSError, ValueError):
        pass
    return None


def algorithmic_flops(cfg):
    """Forward 2(Dk+Dv) per visible (query, key) pair; backward 2(2Dk+Dv) on a prefix key (the
    prefix dK/dV products are not part of the method) and 2(3Dk+2Dv) on a response key."""
    pre = cfg.Hq * cfg.R * cfg.P
    resp = cfg.Hq * cfg.R * (cfg.R + 1) // 2
    fwd = 2 * (cfg.Dk + cfg.Dv) * (pre + resp)
    bwd_dq = 2 * (2 * cfg.Dk + cfg.Dv) * (pre + resp)
    bwd_kv = 2 * (cfg.Dk + cfg.Dv) * resp
    return fwd, bwd_dq, bwd_kv


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        time.sleep(0.25)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def launch_ranks(args):
    """`--gpus N` outside torchrun: start the N ranks (one per GPU) and pass their exit code on."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_cuda(args):
    from paper_2607_14952_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    cfg = W.CONFIGS[args.workload]
    if args.prefix:
        cfg = W.scaled(cfg, name="%s-P%d" % (cfg.name, args.prefix), P=args.prefix, needles=0)
    if args.small_r:
        # short-response regime: same resident prefix, R rows per head, finer key split so that
        # every SM streams its own slice of K/V -> bound by HBM, not by the tensor pipe
        cfg = W.scaled(cfg, name="%s-R%d" % (cfg.name, args.small_r), R=args.small_r,
                       num_shards=args.shards or 64, needles=0)
    elif args.shards:
        cfg = W.scaled(cfg, name="%s-S%d" % (cfg.name, args.shards), num_shards=args.shards)
    mode = "blocks" if args.blocks else args.mode
    fwd_f, dq_f, kv_f = algorithmic_flops(cfg)
    # algorithmic flops of one step: what the mode has to compute (the blockwise policy pass recomputes
    # the forward that the suffix pass scored, as the method prescribes)
    step_flops = {"replay": fwd_f + dq_f + kv_f, "fused": fwd_f + dq_f + kv_f, "score": fwd_f,
                  "blocks": 2 * fwd_f + dq_f + kv_f}[mode]

    torch.cuda.reset_peak_memory_stats(dev)
    nblocks = args.blocks
    rb = cfg.R // nblocks if nblocks else 0
    if nblocks and (cfg.R % nblocks or rb % cfg.page_size):
        raise SystemExit("--blocks must cut the response into whole pages")
    extra_pages = nblocks * (rb // cfg.page_size) if nblocks else 0
    k_pool, v_pool, table = W.make_prefix(cfg, dev, extra_phys_pages=extra_pages)
    pages = B.ls_prefix_pages_build(cfg.P, cfg.page_size, cfg.num_shards, cfg.Hkv, cfg.Dk, cfg.Dv, k_pool.shape[0],
                                    page_table=table, k_pool=k_pool, v_pool=None if cfg.v_aliases_k else v_pool,
                                    v_aliases_k=cfg.v_aliases_k, stream_budget_kib=args.stream_budget_kib)
    pool_bytes = (k_pool.numel() + (0 if cfg.v_aliases_k else v_pool.numel())) * 2
    S = cfg.num_shards
    n_members = max(1, min(cfg.G, 4))
    members = [W.make_member(cfg, m, dev) for m in replicas.member_ids(rank, n_members)]
    R_call = rb if nblocks else cfg.R
    buf = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
    o_bf16 = buf((cfg.R, cfg.Hq, cfg.Dv), torch.bfloat16)
    o_f32 = buf((cfg.R, cfg.Hq, cfg.Dv), torch.float32)
    lse = buf((cfg.R, cfg.Hq), torch.float32)
    dq = buf((cfg.R, cfg.Hq, cfg.Dk), torch.bfloat16)
    dk = buf((cfg.R, cfg.Hkv, cfg.Dk), torch.bfloat16)
    dv = buf((cfg.R, cfg.Hkv, cfg.Dv), torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_bytes = {k: B.ls_replay_attn_workspace_bytes(pages, R_call, cfg.Hq, cfg.scale, k)
                for k in (B.LS_WORKSPACE_FWD, B.LS_WORKSPACE_BWD, B.LS_WORKSPACE_FWD_MERGED)}
    ws = buf(ws_bytes[B.LS_WORKSPACE_BWD], torch.uint8)
    fwd_ws = buf(max(16, ws_bytes[B.LS_WORKSPACE_FWD], ws_bytes[B.LS_WORKSPACE_FWD_MERGED]), torch.uint8)
    o_part = lse_part = None
    if mode == "replay":
        o_part = buf((S + 1, cfg.R, cfg.Hq, cfg.Dv), torch.float32)
        lse_part = buf((S + 1, cfg.R, cfg.Hq), torch.float32)
    free_ids = None
    if nblocks:
        mapped = set(int(x) for x in table)
        free_ids = [p for p in range(k_pool.shape[0]) if p not in mapped][:extra_pages]
        dk_grad = buf((extra_pages, cfg.page_size, cfg.Hkv, cfg.Dk), torch.float32)
        dv_grad = buf((extra_pages, cfg.page_size, cfg.Hkv, cfg.Dv), torch.float32)
        B.ls_suffix_pages_reserve(pages, nblocks, extra_pages, dk_grad, dv_grad)
    mla = cfg.Dk == 576

    def step(q, kr, vr, d_o):
        if mode == "replay":
            B.ls_replay_attn_fwd(pages, q, kr, vr, cfg.scale, o_part=o_part, lse_part=lse_part, status=status,
                                 workspace=fwd_ws)
            B.ls_lse_merge(o_part, lse_part, o_bf16=o_bf16, o_f32=o_f32, lse=lse, status=status)
        elif mode in ("fused", "score"):
            B.ls_replay_attn_fwd_merged(pages, q, kr, vr, cfg.scale, o_bf16=o_bf16, o_f32=o_f32, lse=lse,
                                        status=status, workspace=fwd_ws)
        if mode in ("replay", "fused"):
            B.ls_replay_attn_bwd(pages, q, kr, vr, o_f32, lse, d_o, cfg.scale, workspace=ws, dq=dq, dk_resp=dk,
                                 dv_resp=dv, status=status)
        if mode == "blocks":
            ppb = rb // cfg.page_size
            sl = lambda x, b: x[b * rb:(b + 1) * rb]
            for b in range(nblocks):            # no-grad suffix pass: score the block, append its pages
                B.ls_replay_attn_fwd_merged(pages, sl(q, b), sl(kr, b), sl(vr, b), cfg.scale, o_bf16=sl(o_bf16, b),
                                            o_f32=sl(o_f32, b), lse=sl(lse, b), status=status, workspace=fwd_ws)
                B.ls_suffix_pages_append(pages, free_ids[b * ppb:(b + 1) * ppb], sl(kr, b), sl(vr, b))
            for b in reversed(range(nblocks)):  # policy pass in reverse: pop, replay, backward
                B.ls_suffix_pages_pop(pages)
                B.ls_replay_attn_fwd_merged(pages, sl(q, b), sl(kr, b), sl(vr, b), cfg.scale, o_bf16=sl(o_bf16, b),
                                            o_f32=sl(o_f32, b), lse=sl(lse, b), status=status, workspace=fwd_ws)
                B.ls_replay_attn_bwd(pages, sl(q, b), sl(kr, b), sl(vr, b), sl(o_f32, b), sl(lse, b), sl(d_o, b),
                                     cfg.scale, workspace=ws, dq=sl(dq, b), dk_resp=sl(dk, b), dv_resp=sl(dv, b),
                                     status=status, flags=B.LS_FLAG_ADD_SUFFIX_GRAD)

    # kernels of this library launched per step (memsets and copies are not kernels)
    bwd_launches = 4                                     # Delta, dQ, dK, dV
    if mla:
        # + the response block's dQ partial; + a reduce per dK / dV when their key tiles alone cannot fill the GPU
        # (head ranges); + a reduce of the part ranges when a short response spreads them over CTA pairs
        bwd_launches = 5
        if cfg.Hkv * -(-cfg.R // 64) * 3 < 148:
            bwd_launches += 2
        blocks64 = cfg.Hkv * (packed_tiles(cfg, 64) or (cfg.Hq // cfg.Hkv) * -(-cfg.R // 64))
        if blocks64 < 74 and S > 1:
            bwd_launches += 1
    launches = {"replay": 2 + bwd_launches, "fused": 1 + bwd_launches, "score": 1,
                "blocks": 0 if not nblocks else sum(1 + 2 + 1 + bwd_launches + 2 * b for b in range(nblocks))}[mode]

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    for w in range(args.warmup):
        step(*members[w % n_members])
    barrier()

    # ---- device-resident timing; the dominant kernels are timed alone through armed events
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    timed_kernels = (B.LS_KERNEL_FWD,) if mode == "score" else (B.LS_KERNEL_FWD, B.LS_KERNEL_BWD_DQ)
    kev = {k: [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
           for k in timed_kernels}
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    graph = None
    if args.graph and mode != "blocks":
        # the step's launches captured once and replayed: no host work per step (the per-call tensor maps and
        # kernel arguments are baked in, so the replays all take member 0's buffers)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(*members[0])
        graph.replay()
        barrier()
    for i in range(args.steps):
        if mode != "blocks" and graph is None:
            for k in kev:
                B.ls_profile_arm_events(k, kev[k][i][0], kev[k][i][1])
        ev[i][0].record()
        if graph is not None:
            graph.replay()
        else:
            step(*members[i % n_members])
        ev[i][1].record()
    barrier()
    if graph is not None:              # the dominant kernels' own times: one eager step with armed events
        for k in kev:
            B.ls_profile_arm_events(k, kev[k][0][0], kev[k][0][1])
        step(*members[0])
        barrier()
        for k in kev:
            kev[k] = [kev[k][0]] * args.steps
    clocks = sampler.stop() if rank == 0 else None
    step_ms = [a.elapsed_time(b) for a, b in ev]
    ms = sum(step_ms)
    k_ms = {k: (sum(a.elapsed_time(b) for a, b in kev[k]) / args.steps if mode != "blocks" else float("nan")) for k in kev}
    ms_total = replicas.max_over_ranks(ms, dev, world)
    if int(status.item()) != 0:
        raise RuntimeError("device status %d" % int(status.item()))

    # ---- end to end: host buffers in, host results out, copies inside the timed region
    outs = (o_bf16,) if mode == "score" else (o_bf16, dq, dk, dv)
    host_in = [[x.cpu().pin_memory() for x in m] for m in members]
    host_out = [torch.empty_like(x, device="cpu").pin_memory() for x in outs]
    dev_in = [torch.empty_like(x) for x in members[0]]
    h2d = sum(x.numel() * x.element_size() for x in host_in[0])
    d2h = sum(x.numel() * x.element_size() for x in host_out)

    def e2e_step(i):
        for d, hsrc in zip(dev_in, host_in[i % n_members]):
            d.copy_(hsrc, non_blocking=True)
        step(*dev_in)
        for hdst, d in zip(host_out, outs):
            hdst.copy_(d, non_blocking=True)

    e2e_step(0)
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_wall = time.perf_counter() - t0
    e2e_ms = replicas.max_over_ranks(max(e0.elapsed_time(e1), e2e_wall * 1e3), dev, world)
    peak_bytes = torch.cuda.max_memory_allocated(dev)

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return
    peaks = measured_peaks()
    ms_per_step = ms_total / args.steps
    value = replicas.aggregate_throughput(step_flops, args.steps, world, ms_total) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    fwd_tflops = fwd_f / (k_ms[B.LS_KERNEL_FWD] * 1e-3) / 1e12
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_best": min(step_ms),
        "ms_per_step_median": float(np.median(step_ms)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "%s: P=%d R=%d Hq=%d Hkv=%d Dk=%d Dv=%d page=%d shards=%d, one member per step" % (
            cfg.name, cfg.P, cfg.R, cfg.Hq, cfg.Hkv, cfg.Dk, cfg.Dv, cfg.page_size, cfg.num_shards),
            "launch": "cuda graph replay" if graph is not None else "eager",
            "mode": mode if not nblocks else "blocks x%d of %d tokens (suffix pass + reverse policy pass)" % (nblocks, rb),
            "l2": "inputs larger than L2 (%.2f GiB of K/V streamed per pass)" % (pool_bytes / 2**30),
            "parallelism": "replicas x%d" % world, "flops_per_step": step_flops,
            "prefix_positions_per_s": world * cfg.P / (ms_per_step * 1e-3)},
        "clocks": clocks,
        "e2e": {"value": world * step_flops / (e2e_ms / args.steps * 1e-3) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches * args.steps,
        "peak_device_bytes": peak_bytes,
        "device_bytes": {"page_pool": pool_bytes, "workspace_fwd": ws_bytes[B.LS_WORKSPACE_FWD],
                         "workspace_fwd_merged": ws_bytes[B.LS_WORKSPACE_FWD_MERGED],
                         "workspace_bwd": ws_bytes[B.LS_WORKSPACE_BWD],
                         "partials": 0 if o_part is None else (o_part.numel() + lse_part.numel()) * 4},
    }
    if mode in ("replay", "fused"):
        dq_tflops = dq_f / (k_ms[B.LS_KERNEL_BWD_DQ] * 1e-3) / 1e12
        kname = kernel_names(cfg)[1]
        out["roofline"] = {"bound": "tensor", "kernel": "%s (query-gradient pass over all parts)" % kname,
                           "achieved": dq_tflops, "peak": peak, "unit": UNIT, "frac": dq_tflops / peak,
                           "peak_source": "%s sustained bf16 cuBLAS (burst %.1f)" % (peaks["source"], peaks["bf16_tflops"]),
                           "ms_per_launch": k_ms[B.LS_KERNEL_BWD_DQ],
                           "traffic": measured_traffic(kname, cfg.name),
                           "algorithmic_flops_per_launch": dq_f,
                           "fwd_kernel": {"kernel": kernel_names(cfg)[0], "achieved": fwd_tflops, "frac": fwd_tflops / peak,
                                          "ms_per_launch": k_ms[B.LS_KERNEL_FWD],
                                          "traffic": measured_traffic(kernel_names(cfg)[0], cfg.name)},
                           "whole_step_frac": value / world / peak,
                           "frac_of_nominal_2250": value / world / 2250.0}
    elif mode == "score":
        kname = kernel_names(cfg)[0]
        out["roofline"] = {"bound": "tensor", "kernel": "%s (forward with the merge folded in)" % kname,
                           "achieved": fwd_tflops, "peak": peak, "unit": UNIT, "frac": fwd_tflops / peak,
                           "peak_source": "%s sustained bf16 cuBLAS (burst %.1f)" % (peaks["source"], peaks["bf16_tflops"]),
                           "ms_per_launch": k_ms[B.LS_KERNEL_FWD], "traffic": measured_traffic(kname + ":merged", cfg.name),
                           "algorithmic_flops_per_launch": fwd_f, "frac_of_nominal_2250": value / world / 2250.0}
    else:
        out["roofline"] = {"bound": "tensor", "kernel": "whole blockwise step (no single dominant launch)",
                           "achieved": value / world, "peak": peak, "unit": UNIT, "frac": value / world / peak,
                           "peak_source": "%s sustained bf16 cuBLAS" % peaks["source"], "traffic": None}
    if args.small_r and mode != "blocks":
        kv_bytes = pool_bytes
        fwd_gbs = kv_bytes / (k_ms[B.LS_KERNEL_FWD] * 1e-3) / 1e9
        fname, dqname = kernel_names(cfg)
        out["roofline"] = {"bound": "hbm", "kernel": "%s (K and V pages streamed once per launch)" % fname,
                           "achieved": fwd_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": fwd_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                           "ms_per_launch": k_ms[B.LS_KERNEL_FWD], "traffic": measured_traffic(fname, cfg.name),
                           "algorithmic_bytes_per_launch": kv_bytes, "frac_of_nominal_8000": fwd_gbs / 8000.0}
        if B.LS_KERNEL_BWD_DQ in k_ms:
            dq_gbs = kv_bytes / (k_ms[B.LS_KERNEL_BWD_DQ] * 1e-3) / 1e9
            out["roofline"]["dq_kernel"] = {"kernel": dqname, "achieved": dq_gbs, "frac": dq_gbs / peaks["hbm_gbs"],
                                            "ms_per_launch": k_ms[B.LS_KERNEL_BWD_DQ],
                                            "traffic": measured_traffic(dqname, cfg.name)}
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(cfg, seconds_target=15.0)
    print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_dsa(args):
    """Sparse (DSA) replay over the shared latent: index scores -> global top-k -> attention over the
    selected rows + the causal response block -> backward.  One step = one member; 1 GPU."""
    from paper_2607_14952_b200 import binding as B
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = W.CONFIGS["mla1m"]
    if args.prefix:
        cfg = W.scaled(cfg, name="%s-P%d" % (cfg.name, args.prefix), P=args.prefix)
    HI, TOPK = 32, 2048
    torch.cuda.reset_peak_memory_stats(dev)
    k_pool, _, table = W.make_prefix(cfg, dev)
    pages = B.ls_prefix_pages_build(cfg.P, cfg.page_size, cfg.num_shards, cfg.Hkv, cfg.Dk, cfg.Dv, k_pool.shape[0],
                                    page_table=table, k_pool=k_pool, v_aliases_k=True)
    members = []
    for m in range(2):
        ki_pool, q_index, w_index = W.make_index_inputs(cfg, HI, m, dev)
        q, kr, _, d_o = W.make_member(cfg, m, dev)
        members.append((q_index, w_index, q, kr, kr[..., :cfg.Dv].contiguous(), d_o))
    plan = B.ls_dsa_plan_create(pages, ki_pool, cfg.R, cfg.Hq, HI, TOPK)
    count = plan.count
    scores = torch.empty((cfg.R, cfg.P), dtype=torch.float32, device=dev)
    sel = torch.empty((cfg.R, count), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_f = torch.empty(int(B.lib().ls_dsa_workspace_bytes(plan.handle, B.LS_WORKSPACE_FWD)), dtype=torch.uint8, device=dev)
    ws_b = torch.empty(int(B.lib().ls_dsa_workspace_bytes(plan.handle, B.LS_WORKSPACE_BWD)), dtype=torch.uint8, device=dev)
    names = ("index_scores", "topk", "attn_fwd", "attn_bwd")

    def step(m, ev=None):
        q_index, w_index, q, kr, vr, d_o = m
        mark = (lambda i: ev[i].record()) if ev else (lambda i: None)
        mark(0)
        B.ls_dsa_index_scores(plan, q_index, w_index, scores=scores, status=status)
        mark(1)
        B.ls_dsa_topk(plan, scores, sel=sel)
        mark(2)
        _, o_f32, lse = B.ls_dsa_attn_fwd(plan, sel, q, kr, vr, cfg.scale, status=status, workspace=ws_f)
        mark(3)
        B.ls_dsa_attn_bwd(plan, q, kr, vr, o_f32, lse, d_o, cfg.scale, status=status, workspace=ws_b)
        mark(4)

    for w in range(args.warmup):
        step(members[w % 2])
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    for i in range(args.steps):
        step(members[i % 2], evs[i])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if int(status.item()) != 0:
        raise RuntimeError("device status %d" % int(status.item()))
    phase_ms = {n: float(np.mean([e[j].elapsed_time(e[j + 1]) for e in evs])) for j, n in enumerate(names)}
    step_ms = [e[0].elapsed_time(e[4]) for e in evs]
    pairs = cfg.Hq * cfg.R * count + cfg.Hq * cfg.R * (cfg.R + 1) // 2
    f_index = 2 * cfg.R * HI * cfg.P * 128
    f_fwd = 2 * (cfg.Dk + cfg.Dv) * pairs
    f_bwd = 2 * (2 * cfg.Dk + cfg.Dv) * pairs + 2 * (cfg.Dk + cfg.Dv) * cfg.Hq * cfg.R * (cfg.R + 1) // 2
    flops = f_index + f_fwd + f_bwd
    peaks = measured_peaks()
    ms = float(np.mean(step_ms))
    idx_tflops = f_index / (phase_ms["index_scores"] * 1e-3) / 1e12
    print(json.dumps({
        "metric": METRIC, "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_best": min(step_ms),
        "ms_per_step_median": float(np.median(step_ms)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "%s sparse: P=%d R=%d Hq=%d latent 576/512, %d index heads of 128, top-%d" % (
            cfg.name, cfg.P, cfg.R, cfg.Hq, HI, TOPK), "mode": "dsa (index scores, top-k, sparse attention fwd + bwd)",
            "flops_per_step": flops, "flops_index": f_index, "flops_attention": f_fwd + f_bwd, "phase_ms": phase_ms,
            "l2": "indexer-key pages %.2f GiB + scores %.2f GiB streamed per step" % (
                ki_pool.numel() * 2 / 2**30, scores.numel() * 4 / 2**30)},
        "clocks": clocks, "gpu_launches": 11 * args.steps, "peak_device_bytes": torch.cuda.max_memory_allocated(dev),
        "roofline": {"bound": "tensor", "kernel": "dsa_index_kernel (index scores, Eq. dsa-index)", "achieved": idx_tflops,
                     "peak": peaks["bf16_tflops_sustained"], "unit": UNIT, "frac": idx_tflops / peaks["bf16_tflops_sustained"],
                     "peak_source": "%s sustained bf16 cuBLAS" % peaks["source"], "ms_per_launch": phase_ms["index_scores"],
                     "traffic": measured_traffic("dsa_index_kernel", cfg.name), "algorithmic_flops_per_launch": f_index}}))


def _cpu_sample_inputs(cfg):
    """Inputs of ONE KV head on the host, drawn with the CPU generator (same distributions)."""
    one = W.scaled(cfg, Hkv=1, Hq=cfg.Hq // cfg.Hkv, needles=0)
    k_pool, v_pool, table = W.make_prefix(one, "cpu")
    q, kr, vr, d_o = W.make_member(one, 0, "cpu")
    return one, W.bf16_bits(k_pool), (W.bf16_bits(k_pool) if cfg.v_aliases_k else W.bf16_bits(v_pool)), table, \
        W.bf16_bits(q), W.bf16_bits(kr), W.bf16_bits(vr), W.bf16_bits(d_o)


def _oracle_rows(one, kp, vp, table, q, kr, vr, d_o, rows):
    from oracle import attention as oa
    t_rows = np.linspace(0, one.R - 1, rows).astype(np.int64)
    heads = np.arange(rows) % one.Hq
    t0 = time.perf_counter()
    oa.backward_rows(q[t_rows, heads], t_rows, 0, kp, vp, table, one.P, one.page_size, kr, vr,
                     float(np.float32(one.scale)), d_o[t_rows, heads])
    dt = time.perf_counter() - t0
    # algorithmic flops of those rows: forward + dQ over every visible key (+ response dK/dV share)
    vis = one.P + t_rows + 1
    flops = float((vis * (2 * (one.Dk + one.Dv) + 2 * (2 * one.Dk + one.Dv))).sum()
                  + ((t_rows + 1) * 2 * (one.Dk + one.Dv)).sum())
    return dt, flops


def cpu_baseline(cfg, seconds_target=15.0, inputs=None):
    """The fp64 oracle as it stands, timed on this machine's host cores on a bounded row sample."""
    inp = inputs or _cpu_sample_inputs(cfg)
    rows = 4
    dt, fl = _oracle_rows(*inp, rows=rows)
    for _ in range(3):                        # grow the sample until it costs about the target time
        if dt >= 0.6 * seconds_target or rows >= 256:
            break
        rows = int(max(rows + 1, min(256, rows * seconds_target / max(dt, 1e-6))))
        dt, fl = _oracle_rows(*inp, rows=rows)
    return {"value": fl / dt / 1e12, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": "%d (row, head) pairs of one KV head of %s, forward + backward over all %d visible keys, "
                      "%.1f s" % (rows, cfg.name, cfg.P + cfg.R, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = W.CONFIGS[args.workload]
    inp = _cpu_sample_inputs(cfg)
    rows = args.ref_rows
    for _ in range(args.warmup):
        _oracle_rows(*inp, rows=max(1, rows // 4))
    times, flops = [], 0.0
    for _ in range(args.steps):
        dt, fl = _oracle_rows(*inp, rows=rows)
        times.append(dt)
        flops += fl
    value = flops / sum(times) / 1e12
    sample = "%d (row, head) pairs of one KV head per step, forward + backward over all visible keys" % rows
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (bounded sample: %s)" % (cfg.name, sample)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="p2m", choices=list(W.CONFIGS))
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-rows", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", action="store_true", help="replay the step as one CUDA graph (launch-bound workloads)")
    ap.add_argument("--small-r", type=int, default=0, help="short-response regime: R rows per head")
    ap.add_argument("--shards", type=int, default=0, help="key shards for --small-r (default 64)")
    ap.add_argument("--prefix", type=int, default=0, help="override the workload's prefix length (profiling on a small case)")
    ap.add_argument("--stream-budget-kib", type=int, default=0,
                    help="K+V bytes of one (KV head, key range) stream, in KiB (0 = the library's default)")
    ap.add_argument("--mode", default="replay", choices=["replay", "fused", "score", "dsa"])
    ap.add_argument("--blocks", type=int, default=0, help="blockwise replay with a paged suffix in this many blocks")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "dsa":
        run_dsa(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args))
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
