#!/usr/bin/env python
"""Benchmark of the affix-cache refresh path (one layer-step = anchor scoring, top-K
selection, selective recomputation, KV scatter) on synthetic LLaDA-8B-shaped inputs.

    python bench.py --gpus N --steps K --warmup W            # the CUDA path (C ABI)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, timed as it stands

Prints ONE JSON line.  ``value`` is affix tokens refreshed per second over all ranks
(B*K anchors per layer-step / step time, max over ranks), timed with CUDA events on the
launching stream with the inputs resident in HBM; ``e2e`` is the same through the
host-buffer entry point with the per-step host<->device copies inside the timed region.
With N > 1 every rank refreshes its own requests (the path shards by request; weights and
the affix cache are replicated) and there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_26140_b200 import sharding, workloads as wl  # noqa: E402

METRIC = "anchor_refresh_affix_tokens_per_s"
UNIT = "affix tokens/s"
RATIO = 0.2

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from an ncu capture of the kernel as it
# stands at the commit named here; None until such a capture exists (a figure from an older kernel is not printed).
NCU_TRAFFIC = {"kernel": "gemm_tc_kernel, gate/up projection 103 x 24576 x 4096 (one launch; 204.7 MB algorithmic)",
               "bytes": 207042048, "commit": "c3e8c66"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), tflops=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops=1400.0, source="fallback")


def step_work(shape: wl.LayerShape, lay: wl.Layout, K: int):
    """Algorithmic bytes and flops of one layer-step (per rank)."""
    B, T, L, m = lay.batch, lay.ctx_len, lay.affix_len, lay.n_masked
    D, H, Hkv, d, Fm = shape.hidden, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.ffn
    n_r = B * (K + lay.n_extra)
    n_m = B * m
    w_bytes = shape.weight_bytes() + 2 * D * 2
    by = dict(
        weights=w_bytes,
        score_k=B * L * Hkv * d * 2,
        x_rows=(n_r + n_m) * D * 2,
        attn_kv=B * T * 2 * Hkv * d * 2,
        scatter=n_r * 2 * Hkv * d * 2,
        y=n_r * D * 2,
        scores=B * L * 4 + B * K * 4,
    )
    params = D * H * d + 2 * D * Hkv * d + H * d * D + 3 * D * Fm
    fl = dict(
        proj=2 * n_r * params + 2 * n_m * D * H * d,
        score=2 * n_m * L * H * d,               # the logits of Eq. 4, counted once
        attn=4 * n_r * T * H * d,
    )
    gate_up_bytes = 2 * Fm * D * 2 + n_r * D * 2 + n_r * Fm * 2
    gate_up_flops = 2 * n_r * D * 2 * Fm
    return sum(by.values()), sum(fl.values()), gate_up_bytes, gate_up_flops, n_r


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while running."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.sm, self.reasons, self.max_mhz = index, False, [], set(), None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self.stop_flag:
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def summary(self):
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def build_case(cfg: int, extra: str, batch):
    shape = {1: wl.TINY, 2: wl.LLADA_8B, 3: wl.LLADA_8B, 4: wl.DREAM_7B}[cfg]
    lay = wl.config_layout(cfg, extra, n_masked=32, batch=batch)
    return shape, lay, wl.make_case(shape, lay, RATIO, cfg_id=cfg)


# ------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle, unmodified, on the same workload; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import acache_oracle as orc
    shape, lay, case = build_case(args.config, args.extra, args.batch)
    L = lay.affix_len
    K_full = orc.k_from_ratio(L, RATIO)
    w64 = {k: (orc.bf16_bits_to_f64(v) if v is not None else None) for k, v in case.weights.items()}

    def one_step(K):
        for b in range(lay.batch):
            orc.layer_step(w64, shape, case.x[b], case.cache_k[b], case.cache_v[b], lay.ctx_len, lay.affix_start, L,
                           lay.masked_pos[b], lay.extra_rows[b], case.rope_cos, case.rope_sin, K=K)

    t0 = time.perf_counter()
    one_step(K_full)                         # calibration (untimed)
    t_full = time.perf_counter() - t0
    total = args.steps + args.warmup
    K = K_full
    if t_full * total > 150.0:               # bound the run: refresh fewer anchors per step
        K = max(4, int(K_full * 150.0 / (t_full * total)))
    for _ in range(args.warmup):
        one_step(K)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step(K)
    dt = (time.perf_counter() - t0) / args.steps
    value = lay.batch * K / dt
    cores = _threads_used()
    sample = (f"{K} of {K_full} anchors per request per step (scoring over all {L} affix keys), {lay.batch} request(s); "
              f"weights converted bf16 -> fp64 once, outside the timed steps; {cores} BLAS threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, lay, args, K),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def _threads_used():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def workload_config(shape, lay, args, K):
    return {"workload": f"{lay.name}: {shape.name} layer (hidden {shape.hidden}, {shape.n_heads}x{shape.head_dim} heads, "
                        f"{shape.n_kv_heads} KV heads, MLP {shape.ffn}), batch {lay.batch}/GPU, affix {lay.affix_len} at "
                        f"{lay.affix_start}, context {lay.ctx_len}, {lay.n_masked} masked rows, ratio {RATIO} (K={K}), "
                        f"extra rows {lay.n_extra}",
            "benchmark_config": args.config, "ratio": RATIO, "anchors_per_request": K, "rows_per_request": K + lay.n_extra,
            "l2": f"per-step weights ({shape.weight_bytes() / 1e6:.0f} MB) exceed L2; {args.instances} weight/cache "
                  "instances rotated", "parallelism": f"request-sharded x{args.gpus}"}


# ------------------------------------------------------------------------------------------
def init_rank():
    """Device, rank and (for more than one rank) the NCCL process group of this process."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    return rank, world, local, dev, dist


def time_blocks(step, steps, n_blocks, sync_all, dist, dev):
    """Times n_blocks consecutive blocks of exactly `steps` steps each with CUDA events on the launching stream
    (one event per block boundary, no synchronisation in between); per block the max over ranks.  Returns the
    per-step times in ms, one per block."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
    sync_all()
    k = 0
    ev[0].record()
    for b in range(n_blocks):
        for _ in range(steps):
            step(k)
            k += 1
        ev[b + 1].record()
    sync_all()
    ms = [ev[b].elapsed_time(ev[b + 1]) / steps for b in range(n_blocks)]
    if dist is not None:
        t = torch.tensor(ms, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = t.tolist()
    return ms


def spread(ms_per_step):
    v = np.sort(np.asarray(ms_per_step, dtype=np.float64)) * 1e3
    return {"blocks": int(v.size), "median": float(np.median(v)), "min": float(v[0]), "max": float(v[-1]),
            "p10": float(v[int(0.1 * (v.size - 1))]), "p90": float(v[int(0.9 * (v.size - 1))]), "unit": "us per step"}


def run_ours(args):
    import torch
    from paper_2608_26140_b200 import binding as ab
    from paper_2608_26140_b200 import build as abuild

    rank, world, local, dev, dist = init_rank()
    if rank == 0:
        abuild.build()
    if dist:
        dist.barrier()

    shape, lay, case = build_case(args.config, args.extra, args.batch)
    B, T, L = lay.batch, lay.ctx_len, lay.affix_len
    K = ab.k_from_ratio(L, RATIO)
    n = K + lay.n_extra
    inst = []
    for _ in range(args.instances):
        w = {k: (ab.to_device_bf16(v, dev) if v is not None else None) for k, v in case.weights.items()}
        inst.append(dict(w=w, lw=ab.Context.weights(w), x=ab.to_device_bf16(case.x, dev),
                         ck=ab.to_device_bf16(case.cache_k, dev), cv=ab.to_device_bf16(case.cache_v, dev)))
    cos, sin = torch.from_numpy(case.rope_cos).to(dev), torch.from_numpy(case.rope_sin).to(dev)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(dev) if lay.n_extra else None
    req = ab.Context.request(B, T, lay.affix_start, L, masked, extra, cos, sin)
    ctx = ab.Context.for_shape(shape, B, T, L, max(n, 1), max(lay.n_masked, 1), dev)
    scores = torch.zeros((B, L), dtype=torch.float32, device=dev)
    anchors = torch.zeros((B, max(K, 1)), dtype=torch.int32, device=dev)
    y = torch.zeros((B, max(n, 1), shape.hidden), dtype=torch.bfloat16, device=dev)
    flags = ab.F_SCORE | ab.F_SELECT

    def step(i):
        it = inst[i % len(inst)]
        ctx.layer_step(it["lw"], req, ab.Context.kv(it["ck"], it["cv"]), it["x"], 0, RATIO, flags, scores, anchors, y)

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for i in range(warmup):
        step(i)
    sync_all()
    # a first block sizes the run: at least 50 blocks of `steps` steps, and enough of them to keep the GPU busy for
    # about a second, so that the clock sampler sees the load
    est = time_blocks(step, args.steps, 1, sync_all, dist, dev)[0]
    n_blocks = args.blocks if args.blocks > 0 else int(min(2000, max(50, np.ceil(1000.0 / max(est * args.steps, 1e-3)))))
    sampler = ClockSampler(local)
    sampler.start()
    l0 = ctx.launch_count()
    blocks = time_blocks(step, args.steps, n_blocks, sync_all, dist, dev)
    launches_per_step = (ctx.launch_count() - l0) / (n_blocks * args.steps)
    ms_step = float(np.median(blocks))

    # second timed pass over the same steps with an event before every stage
    ctx.stage_timing(True)
    stage = {s: 0.0 for s in ab.STAGES}
    for i in range(args.steps):
        step(i)
        for s, v in ctx.read_stage_times().items():
            stage[s] += v / args.steps
    ctx.stage_timing(False)
    assert ctx.poll_status() == 0, "device status word set during the benchmark"

    # end to end: per-step inputs in pinned host memory, results read back to the host
    xh = torch.from_numpy(case.x.view(np.int16)).view(torch.bfloat16).pin_memory()
    sh = torch.zeros((B, L), dtype=torch.float32).pin_memory()
    ah = torch.zeros((B, max(K, 1)), dtype=torch.int32).pin_memory()
    yh = torch.zeros((B, max(n, 1), shape.hidden), dtype=torch.bfloat16).pin_memory()

    def step_host(i):
        it = inst[i % len(inst)]
        ctx.layer_step_host(it["lw"], req, ab.Context.kv(it["ck"], it["cv"]), xh, RATIO, 0, sh, ah, yh)

    for i in range(3):
        step_host(i)
    blocks_e2e = time_blocks(step_host, args.steps, args.blocks if args.blocks > 0 else max(50, n_blocks // 4), sync_all, dist, dev)
    ms_e2e = float(np.median(blocks_e2e))
    sampler.stop_flag = True
    sampler.join()
    # page-locked x is read in place: the kernels pull the masked rows and the recomputed rows, each once
    x_in_place = ctx.host_x_in_place(xh) and (lay.n_masked + n) * 4 <= T    # the entry point's own rule
    h2d = B * (lay.n_masked + n) * shape.hidden * 2 if x_in_place else xh.numel() * 2
    d2h = n * B * shape.hidden * 2 + B * K * 4 + B * L * 4

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    step_bytes, step_flops, gu_bytes, gu_flops, n_r = step_work(shape, lay, K)
    t_hbm = step_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = step_flops / (peaks["tflops"] * 1e12)
    floor_s = max(t_hbm, t_tc)
    hbm_bound = t_hbm >= t_tc
    s_step = ms_step * 1e-3
    gu_s = stage["gate_up"] * 1e-3
    gu_hbm_bound = gu_bytes / (peaks["hbm_gbs"] * 1e9) >= gu_flops / (peaks["tflops"] * 1e12)
    gu_ach, gu_peak, gu_unit = ((gu_bytes / gu_s / 1e9, peaks["hbm_gbs"], "GB/s") if gu_hbm_bound
                                else (gu_flops / gu_s / 1e12, peaks["tflops"], "TFLOP/s"))
    # the roofline of the whole fused path: the slower of its bytes at the HBM peak and its flops at the tensor peak,
    # over the measured time of one layer-step (all its launches)
    roofline = {"kernel": f"whole layer-step ({launches_per_step:.0f} launches)", "bound": "hbm" if hbm_bound else "tensor",
                "achieved": (step_bytes / s_step / 1e9) if hbm_bound else (step_flops / s_step / 1e12),
                "peak": peaks["hbm_gbs"] if hbm_bound else peaks["tflops"], "unit": "GB/s" if hbm_bound else "TFLOP/s",
                "frac": floor_s / s_step, "peak_source": peaks["source"], "floor_us": floor_s * 1e6,
                "algorithmic_bytes": step_bytes, "algorithmic_flops": step_flops,
                "traffic": NCU_TRAFFIC["bytes"] if (args.config == 2 and lay.n_extra == 0 and B == 1) else None,
                "traffic_of": NCU_TRAFFIC["kernel"], "traffic_commit": NCU_TRAFFIC["commit"],
                "dominant_kernel": {"kernel": "gate/up projection + SwiGLU (stage gate_up, from the staged pass)",
                                    "bound": "hbm" if gu_hbm_bound else "tensor", "achieved": gu_ach, "peak": gu_peak,
                                    "unit": gu_unit, "frac": gu_ach / gu_peak, "algorithmic_bytes": gu_bytes,
                                    "algorithmic_flops": gu_flops, "us_per_launch": stage["gate_up"] * 1e3}}
    value = sharding.aggregate_throughput(B * K, world, ms_step)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_step, "us_per_layer_step": ms_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(shape, lay, args, K),
        "timing": {"protocol": f"{n_blocks} consecutive blocks of {args.steps} layer-steps, one CUDA event per block boundary, "
                               "max over ranks per block; value and ms_per_step are the median block", **spread(blocks)},
        "clocks": sampler.summary(),
        "e2e": {"value": world * B * K / (ms_e2e * 1e-3), "unit": UNIT, "us_per_layer_step": ms_e2e * 1e3,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "timing": spread(blocks_e2e),
                "x_transfer": "rows read in place from page-locked host memory by the kernels" if x_in_place
                else "whole x staged by one copy"},
        "gpu_launches": int(round(launches_per_step * args.steps)),
        "gpu_launches_per_step": launches_per_step,
        "roofline": roofline,
        "stage_us": {s: v * 1e3 for s, v in stage.items()},
        "affix_tokens_covered_per_s": world * B * L / (ms_step * 1e-3),
    }
    if world == 1 and not args.no_extra:
        # free the headline workload's buffers, then the other configurations the metric names, each a short run
        del inst, ctx, xh, yh
        torch.cuda.empty_cache()
        out["extra"] = extra_records(args, peaks, dev)
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(case, shape, lay)
    print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


def probe_layer(cfg, batch, steps, peaks, dev):
    """One layer of the one-shot probe (Section 3.2) at benchmark configuration 3 or 4: every request's non-affix rows
    (256 of them masked) through the layer with the affix K/V as cached, the masked-to-affix scores (Eq. 4-5) taken
    from the layer's own attention.  Device-drawn inputs (timing only)."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    from paper_2608_26140_b200 import build as abuild
    abuild.build()
    torch.cuda.set_device(int(dev.split(":")[1]))
    shape = wl.DREAM_7B if cfg == 4 else wl.LLADA_8B
    lay = wl.config_layout(cfg, "all", n_masked=256, batch=batch)
    B, T, L, P = lay.batch, lay.ctx_len, lay.affix_len, lay.n_extra
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.SEED_BASE + 4096 * cfg + 99)

    def randn(shape_, std=1.0):
        t = torch.randn(shape_, generator=gen, device=dev, dtype=torch.bfloat16)
        return t.mul_(std) if std != 1.0 else t

    D, F = shape.hidden, shape.ffn
    w = dict(wq=randn((shape.q_dim, D), 0.02), wk=randn((shape.kv_dim, D), 0.02), wv=randn((shape.kv_dim, D), 0.02),
             wo=randn((D, shape.q_dim), 0.02), w_gate=randn((F, D), 0.02), w_up=randn((F, D), 0.02), w_down=randn((D, F), 0.02),
             attn_norm_g=randn((D,), 0.05).add_(1.0), mlp_norm_g=randn((D,), 0.05).add_(1.0))
    for k_, n_ in (("bq", shape.q_dim), ("bk", shape.kv_dim), ("bv", shape.kv_dim)):
        w[k_] = randn((n_,), 0.02) if shape.qkv_bias else None
    kv_std = 0.02 * float(np.sqrt(D))
    x = randn((B, T, D))
    ck, cv = randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std), randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std)
    cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(dev)
    req = ab.Context.request(B, T, lay.affix_start, L, masked, extra, cos, sin)
    ctx = ab.Context.for_shape(shape, B, T, L, P, lay.n_masked, dev)
    scores = torch.zeros((B, L), dtype=torch.float32, device=dev)
    y = torch.zeros((B, P, D), dtype=torch.bfloat16, device=dev)
    lw = ab.Context.weights(w)

    def step():
        ctx.layer_step(lw, req, ab.Context.kv(ck, cv), x, 0, 0.0, ab.F_SCORE, scores, None, y)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    l0 = ctx.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    launches = (ctx.launch_count() - l0) / steps
    ctx.stage_timing(True)
    step()
    stage = {k_: round(v * 1e3, 1) for k_, v in ctx.read_stage_times().items() if v}
    ctx.stage_timing(False)
    assert ctx.poll_status() == 0
    mass = float(scores.sum().item()) / (B * shape.n_heads * lay.n_masked)          # Eq. 4: every masked row's weights sum to 1
    params = D * shape.q_dim + 2 * D * shape.kv_dim + shape.q_dim * D + 3 * D * F
    flops = 2 * B * P * params + 4 * B * P * T * shape.q_dim
    med = float(np.median(ms))
    return {"metric": "probe_layer_ms", "value": med, "unit": "ms per probe layer", "n_gpus": 1, "steps": steps, "warmup": 3,
            "ms_per_step": med, "ms_min": float(min(ms)), "ms_max": float(max(ms)), "higher_is_better": False, "dtype": "bf16",
            "data": "synthetic, drawn on the device",
            "config": {"workload": f"cfg{cfg} probe layer: {shape.name}, batch {B}, affix {L} at {lay.affix_start}, {P} rows per request "
                                   f"({lay.n_masked} masked), no anchors, scores from the layer's own attention",
                       "benchmark_config": cfg},
            "gpu_launches": int(round(launches * steps)), "gpu_launches_per_step": launches, "stage_us": stage,
            "score_mass_per_masked_row_and_head": mass,
            "roofline": {"bound": "tensor", "achieved": flops / (med * 1e-3) / 1e12, "peak": peaks["tflops"], "unit": "TFLOP/s",
                         "frac": flops / (med * 1e-3) / 1e12 / peaks["tflops"], "peak_source": peaks["source"]}}


def extra_records(args, peaks, dev):
    """Short measurements of the other workloads the metric names, carried in the same JSON line: one denoising step
    at benchmark configuration 3 (32 layers, vocabulary 126464, 16 requests), three points of the configuration-5
    sweep, configuration 2 with every request row recomputed, and the KV-deviation scoring kernel.  All inputs are
    drawn on the device (timing only; parity at these sizes is in the tests)."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    out = {}
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.SEED_BASE + 77)

    def randn(shape_, std=1.0):
        t = torch.randn(shape_, generator=gen, device=dev, dtype=torch.bfloat16)
        return t.mul_(std) if std != 1.0 else t

    def dev_weights(shape, std=0.02):
        D, F = shape.hidden, shape.ffn
        dims = dict(wq=(shape.q_dim, D), wk=(shape.kv_dim, D), wv=(shape.kv_dim, D), wo=(D, shape.q_dim),
                    w_gate=(F, D), w_up=(F, D), w_down=(D, F))
        w = {k: randn(v, std) for k, v in dims.items()}
        w["attn_norm_g"] = randn((D,), 0.05).add_(1.0)
        w["mlp_norm_g"] = randn((D,), 0.05).add_(1.0)
        w["bq"] = w["bk"] = w["bv"] = None
        return w

    def timed(fn, steps, warm):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        return [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]

    shape = wl.LLADA_8B
    kv_std = 0.02 * float(np.sqrt(shape.hidden))

    # ---- configuration 3: acache_denoise_step, 32 layers + LM head + commit
    n_layers, V, n_blk = 32, 126464, 32
    lay = wl.config_layout(3, "all", n_masked=32, batch=16)
    B, T, L, P = lay.batch, lay.ctx_len, lay.affix_len, lay.n_extra
    K = ab.k_from_ratio(L, RATIO)
    n = K + P
    ws = [dev_weights(shape) for _ in range(n_layers)]
    lws = [ab.Context.weights(w) for w in ws]
    dk = [randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std) for _ in range(n_layers)]
    dv = [randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std) for _ in range(n_layers)]
    kvs = [ab.Context.kv(dk[i], dv[i]) for i in range(n_layers)]
    embed, w_lm = randn((V, shape.hidden)), randn((V, shape.hidden), 0.02)
    gain = randn((shape.hidden,), 0.05).add_(1.0)
    g = np.random.Generator(np.random.Philox(wl.SEED_BASE + 4096 * 3 + 43))
    ids = g.integers(0, V - 1, size=(B, T)).astype(np.int32)
    ids[:, lay.affix_start:lay.affix_start + L] = ids[0, lay.affix_start:lay.affix_start + L]
    ids[:, lay.masked_pos[0]] = V - 1
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    block_rows = np.stack([[K + where[int(p)] for p in lay.masked_pos[b][:n_blk]] for b in range(B)]).astype(np.int32)
    cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(dev)
    dids = torch.from_numpy(ids).to(dev)
    req = ab.Context.request(B, T, lay.affix_start, L, masked, extra, cos, sin, token_ids=dids, n_embed=V)
    ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, dev, max_vocab=V, max_block=n_blk)
    ya = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=dev)
    yb = torch.zeros_like(ya)
    da, dbr = torch.from_numpy(anchors).to(dev), torch.from_numpy(block_rows).to(dev)
    token = torch.zeros((B, n_blk), dtype=torch.int32, device=dev)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=dev)
    commit = torch.zeros((B, n_blk), dtype=torch.int32, device=dev)
    sampler = ClockSampler(int(dev.split(":")[1]))
    sampler.start()
    l0 = ctx.launch_count()
    ms = timed(lambda: ctx.denoise_step(lws, kvs, req, embed, da, K, ya, yb, dbr, n_blk, gain, w_lm, V, 0.9, token, conf, commit),
               steps=4, warm=2)
    launches = (ctx.launch_count() - l0) / 6
    sampler.stop_flag = True
    sampler.join()
    assert ctx.poll_status() == 0
    step_bytes, step_flops, _, _, _ = step_work(shape, lay, K)
    D, H, d = shape.hidden, shape.n_heads, shape.head_dim
    layer_flops = step_flops - 2 * B * lay.n_masked * D * H * d - 2 * B * lay.n_masked * L * H * d   # a refresh layer scores nothing
    flops = n_layers * layer_flops + 2 * B * n_blk * D * V
    bytes_ = n_layers * step_bytes + 2 * V * D
    floor_s = max(flops / (peaks["tflops"] * 1e12), bytes_ / (peaks["hbm_gbs"] * 1e9))
    med = float(np.median(ms))
    out["config3_denoise_step"] = {
        "workload": f"cfg3: LLaDA-8B shapes, {n_layers} layers (each its own weights and caches), vocab {V}, batch {B} sharing a "
                    f"{L}-token prefix affix, {P} request rows each, ratio {RATIO} (K={K}), {n} rows recomputed per request "
                    f"({B * n} per layer), {n_blk}-token block; acache_denoise_step = refresh forward + LM head + commit",
        "denoise_steps_per_s": 1e3 / med, "ms_per_step": med, "ms_per_step_min": float(min(ms)), "ms_per_step_max": float(max(ms)),
        "steps": len(ms), "warmup": 2, "gpu_launches_per_step": launches,
        "roofline": {"bound": "tensor", "achieved": flops / (med * 1e-3) / 1e12, "peak": peaks["tflops"], "unit": "TFLOP/s",
                     "frac": floor_s / (med * 1e-3), "floor_ms": floor_s * 1e3, "algorithmic_flops": flops,
                     "algorithmic_bytes": bytes_, "peak_source": peaks["source"]},
        "affix_tokens_refreshed_per_s": B * K * n_layers / (med * 1e-3), "clocks": sampler.summary(),
        "data": "synthetic, drawn on the device"}
    del ws, lws, dk, dv, kvs, embed, w_lm, ctx, ya, yb
    torch.cuda.empty_cache()

    # ---- layer-steps: configuration 2 with all request rows, three configuration-5 sweep points
    winst = [dev_weights(shape) for _ in range(3)]
    wl_inst = [ab.Context.weights(w) for w in winst]
    points = [("config2_all_request_rows", wl.config_layout(2, "all", n_masked=32, batch=1), RATIO),
              ("sweep_L8192_B1_r0.2", wl.sweep_layout(8192, 1, "prefix", "none"), 0.2),
              ("sweep_L2048_B8_r0.2", wl.sweep_layout(2048, 8, "prefix", "none"), 0.2),
              ("sweep_L512_B64_r0.2", wl.sweep_layout(512, 64, "prefix", "none"), 0.2)]
    for name, lay, ratio in points:
        B, T, L = lay.batch, lay.ctx_len, lay.affix_len
        K = ab.k_from_ratio(L, ratio)
        n = K + lay.n_extra
        n_c = 3 if B * T * shape.hidden * 2 < (1 << 28) else 1
        xs = [randn((B, T, shape.hidden)) for _ in range(n_c)]
        cks = [randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std) for _ in range(n_c)]
        cvs = [randn((B, T, shape.n_kv_heads, shape.head_dim), kv_std) for _ in range(n_c)]
        l = lay.affix_start
        for t in xs + cks + cvs:
            t[1:, l:l + L] = t[0:1, l:l + L]
        cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
        cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
        masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
        extra = torch.from_numpy(lay.extra_rows.copy()).to(dev) if lay.n_extra else None
        req = ab.Context.request(B, T, l, L, masked, extra, cos, sin)
        ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, dev)
        scores = torch.zeros((B, L), dtype=torch.float32, device=dev)
        anchors_d = torch.zeros((B, K), dtype=torch.int32, device=dev)
        y = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=dev)
        it = [0]

        def step():
            i = it[0]
            it[0] += 1
            ctx.layer_step(wl_inst[i % 3], req, ab.Context.kv(cks[i % n_c], cvs[i % n_c]), xs[i % n_c], 0, ratio,
                           ab.F_SCORE | ab.F_SELECT, scores, anchors_d, y)

        ms = timed(step, steps=30, warm=5)
        ctx.stage_timing(True)
        stage = {s_: 0.0 for s_ in ab.STAGES}
        for _ in range(5):
            step()
            for s_, v in ctx.read_stage_times().items():
                stage[s_] += v / 5
        ctx.stage_timing(False)
        assert ctx.poll_status() == 0
        step_bytes, step_flops, _, _, n_r = step_work(shape, lay, K)
        t_hbm, t_tc = step_bytes / (peaks["hbm_gbs"] * 1e9), step_flops / (peaks["tflops"] * 1e12)
        med = float(np.median(ms)) * 1e-3
        out[name] = {"workload": f"{lay.name}: LLaDA-8B layer, batch {B}, affix {L}, context {T}, {lay.n_masked} masked rows, "
                                 f"ratio {ratio} (K={K}), {n} rows per request",
                     "us_per_layer_step": med * 1e6, "us_min": float(min(ms)) * 1e3, "us_max": float(max(ms)) * 1e3, "steps": len(ms),
                     "affix_tokens_per_s": B * K / med, "rows": n_r,
                     "roofline": {"bound": "hbm" if t_hbm >= t_tc else "tensor", "floor_us": max(t_hbm, t_tc) * 1e6,
                                  "frac": max(t_hbm, t_tc) / med, "achieved_gbs": step_bytes / med / 1e9,
                                  "achieved_tflops": step_flops / med / 1e12, "peak_source": peaks["source"]},
                     "stage_us": {k_: round(v * 1e3, 1) for k_, v in stage.items() if v}}
        if name == "sweep_L2048_B8_r0.2":
            # the KV-deviation selector's scoring kernel on the same caches (HBM-bound: four affix rows per token)
            ms_d = timed(lambda: ctx.score_kv_deviation(req, ab.Context.kv(cks[0], cvs[0]), ab.Context.kv(cks[-1], cvs[-1]), scores),
                         steps=20, warm=3)
            by = 4 * B * L * shape.kv_dim * 2
            md = float(np.median(ms_d)) * 1e-3
            out["kv_deviation_scores_L2048_B8"] = {"us": md * 1e6, "algorithmic_bytes": by, "achieved_gbs": by / md / 1e9,
                                                   "frac_of_hbm_peak": by / md / 1e9 / peaks["hbm_gbs"]}
        del ctx, xs, cks, cvs, y
        torch.cuda.empty_cache()
    del winst, wl_inst
    torch.cuda.empty_cache()
    pr = probe_layer(4, None, 5, peaks, dev)
    out["probe_layer_cfg4"] = {k_: pr[k_] for k_ in ("config", "ms_per_step", "ms_min", "ms_max", "gpu_launches_per_step", "stage_us",
                                                     "score_mass_per_masked_row_and_head", "roofline")}
    return out


# ------------------------------------------------------------------------------------------
def run_denoise(args):
    """Benchmark configuration 3: one denoising step's model pass = 32 LLaDA-8B layers refreshing
    R = anchors + all request rows of 16 requests that share a 2048-token affix, then final norm,
    LM head and the commit rule on the current 32-token block (acache_denoise_step)."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    from paper_2608_26140_b200 import build as abuild

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        abuild.build()
    if dist:
        dist.barrier()
    shape, n_layers, V, n_blk = wl.LLADA_8B, args.layers, 126464, 32
    lay = wl.config_layout(3, "all", n_masked=32, batch=args.batch)
    B, T, L, P = lay.batch, lay.ctx_len, lay.affix_len, lay.n_extra
    K = ab.k_from_ratio(L, RATIO)
    n = K + P
    # 4 seeded weight sets tiled over the layers, one seeded cache replicated per layer (distinct
    # device buffers, so nothing is shared or cached between layers)
    host_sets = [wl.layer_weights(shape, 3, i) for i in range(min(4, n_layers))]
    dev_sets = [{k: (ab.to_device_bf16(v, dev) if v is not None else None) for k, v in w.items()} for w in host_sets]
    layers_dev, lws = [], []
    for i in range(n_layers):
        w = {k: (v.clone() if v is not None else None) for k, v in dev_sets[i % len(dev_sets)].items()} if i >= len(dev_sets) \
            else dev_sets[i]
        layers_dev.append(w)
        lws.append(ab.Context.weights(w))
    ck, cv = wl.random_kv_cache(shape, lay, wl.SEED_BASE + 4096 * 3 + 30)
    ck0, cv0 = ab.to_device_bf16(ck, dev), ab.to_device_bf16(cv, dev)
    dk = [ck0] + [ck0.clone() for _ in range(n_layers - 1)]
    dv = [cv0] + [cv0.clone() for _ in range(n_layers - 1)]
    kvs = [ab.Context.kv(dk[i], dv[i]) for i in range(n_layers)]
    embed = ab.to_device_bf16(wl.normal_bf16(wl.SEED_BASE + 4096 * 3 + 40, (V, shape.hidden), 1.0), dev)
    w_lm = ab.to_device_bf16(wl.normal_bf16(wl.SEED_BASE + 4096 * 3 + 41, (V, shape.hidden), 0.02), dev)
    gain = ab.to_device_bf16(wl.normal_bf16(wl.SEED_BASE + 4096 * 3 + 42, (shape.hidden,), 0.05, 1.0), dev)
    g = np.random.Generator(np.random.Philox(wl.SEED_BASE + 4096 * 3 + 43))
    ids = g.integers(0, V - 1, size=(B, T)).astype(np.int32)
    ids[:, lay.affix_start:lay.affix_start + L] = ids[0, lay.affix_start:lay.affix_start + L]
    ids[:, lay.masked_pos[0]] = V - 1                              # mask id
    anchors = np.stack([np.sort(g.choice(L, K, replace=False)) for _ in range(B)]).astype(np.int32)
    where = {int(p): i for i, p in enumerate(lay.extra_rows[0])}
    block_rows = np.stack([[K + where[int(p)] for p in lay.masked_pos[b][:n_blk]] for b in range(B)]).astype(np.int32)
    cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(dev)
    dids = torch.from_numpy(ids).to(dev)
    req = ab.Context.request(B, T, lay.affix_start, L, masked, extra, cos, sin, token_ids=dids, n_embed=V)
    ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, dev, max_vocab=V, max_block=n_blk)
    ya = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=dev)
    yb = torch.zeros_like(ya)
    da, dbr = torch.from_numpy(anchors).to(dev), torch.from_numpy(block_rows).to(dev)
    token = torch.zeros((B, n_blk), dtype=torch.int32, device=dev)
    conf = torch.zeros((B, n_blk), dtype=torch.float32, device=dev)
    commit = torch.zeros((B, n_blk), dtype=torch.int32, device=dev)

    def step():
        ctx.denoise_step(lws, kvs, req, embed, da, K, ya, yb, dbr, n_blk, gain, w_lm, V, 0.9, token, conf, commit)

    if args.generate:
        return run_generate(args, locals())

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sync_all()
    sampler = ClockSampler(local)
    sampler.start()
    l0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    sync_all()
    sampler.stop_flag = True
    sampler.join()
    launches = ctx.launch_count() - l0
    ms_step = sharding.max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    assert ctx.poll_status() == 0
    # end to end: token ids come from the host every step, tokens / confidence / commit flags go back
    ids_h = torch.from_numpy(ids).pin_memory()
    tok_h, conf_h, com_h = (torch.zeros((B, n_blk), dtype=torch.int32).pin_memory(),
                            torch.zeros((B, n_blk), dtype=torch.float32).pin_memory(),
                            torch.zeros((B, n_blk), dtype=torch.int32).pin_memory())

    def step_host():
        dids.copy_(ids_h, non_blocking=True)
        step()
        tok_h.copy_(token, non_blocking=True); conf_h.copy_(conf, non_blocking=True); com_h.copy_(commit, non_blocking=True)

    for _ in range(2):
        step_host()
    sync_all()
    e0.record()
    for _ in range(args.steps):
        step_host()
    e1.record()
    sync_all()
    ms_e2e = sharding.max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    peaks = load_peaks()
    lay1 = lay
    step_bytes, step_flops, gu_bytes, gu_flops, n_r = step_work(shape, lay1, K)
    # no scoring in a refresh step: drop the masked-row projection and the score pass
    D, H, d = shape.hidden, shape.n_heads, shape.head_dim
    layer_flops = step_flops - 2 * B * lay.n_masked * D * H * d - 4 * B * lay.n_masked * L * H * d
    head_flops = 2 * B * n_blk * D * V
    flops = n_layers * layer_flops + head_flops
    bytes_ = n_layers * step_bytes + 2 * V * D
    floor_s = max(flops / (peaks["tflops"] * 1e12), bytes_ / (peaks["hbm_gbs"] * 1e9))
    out = {
        "metric": "denoise_steps_per_s", "value": world / (ms_step * 1e-3), "unit": "denoising steps/s (model pass + commit)",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic; 4 seeded layer weight sets tiled over the layers, one seeded cache replicated per layer",
        "config": {"workload": f"cfg3: LLaDA-8B shapes, {n_layers} layers, vocab {V}, batch {B}/GPU sharing a {L}-token prefix "
                               f"affix, {P} request rows each, ratio {RATIO} (K={K}), {n} rows recomputed per request, "
                               f"{n_blk}-token block", "benchmark_config": 3, "layers": n_layers,
                   "l2": "per-layer weights (436 MB) exceed L2; every layer has its own weight and cache buffers",
                   "parallelism": f"request-sharded x{world}"},
        "clocks": sampler.summary(),
        "e2e": {"value": world / (ms_e2e * 1e-3), "unit": "denoising steps/s", "h2d_bytes_per_step": int(ids_h.numel() * 4),
                "d2h_bytes_per_step": int(3 * B * n_blk * 4)},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "whole step (tensor-bound)", "bound": "tensor", "achieved": flops / (ms_step * 1e-3) / 1e12,
                     "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": floor_s / (ms_step * 1e-3),
                     "peak_source": peaks["source"], "traffic": None, "algorithmic_flops": flops, "algorithmic_bytes": bytes_},
        "affix_tokens_refreshed_per_s": world * B * K * n_layers / (ms_step * 1e-3),
        "ms_per_layer": (ms_step) / n_layers,
    }
    print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
SWEEP_L = (512, 2048, 8192)
SWEEP_RATIO = (0.05, 0.10, 0.20, 0.35, 0.50)
SWEEP_B = (1, 8, 64)
SWEEP_PLACE = ("prefix", "middle", "suffix")


def run_sweep(args):
    """Benchmark configuration 5: layer-step time, per-stage time and roofline fraction over affix
    length x recompute ratio x batch x affix placement on LLaDA-8B layer shapes (anchors only,
    32 masked rows, 64 request rows).  Timing-only inputs are drawn on the device (normal
    activations and cache entries at the scale the seeded host generator uses; the affix rows of x
    and of the cache are one draw shared by the batch); parity at sweep points is covered by the tests."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    from paper_2608_26140_b200 import build as abuild

    if int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    dev = "cuda:0"
    torch.cuda.set_device(0)
    abuild.build()
    shape = wl.LLADA_8B
    peaks = load_peaks()
    host_w = wl.layer_weights(shape, 5, 0)
    n_inst = max(1, min(args.instances, 4))
    winst = []
    for _ in range(n_inst):
        w = {k: (ab.to_device_bf16(v, dev) if v is not None else None) for k, v in host_w.items()}
        winst.append((w, ab.Context.weights(w)))
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.SEED_BASE + 4096 * 5)
    kv_std = 0.02 * float(np.sqrt(shape.hidden))
    Ls = [int(v) for v in args.sweep_affix.split(",")] if args.sweep_affix else SWEEP_L
    Bs = [int(v) for v in args.sweep_batch.split(",")] if args.sweep_batch else SWEEP_B
    sampler = ClockSampler(0)
    sampler.start()
    points, launches, tot_tokens, tot_s = [], 0, 0.0, 0.0
    flags = ab.F_SCORE | ab.F_SELECT
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # light points first: after a point that draws the full power budget the SM clock stays low for a while,
    # which would be charged to the small points that follow it
    for B in Bs:
        for L in Ls:
            T = L + 96
            row = shape.n_kv_heads * shape.head_dim
            cache_bytes = 2 * B * T * row * 2
            n_cache = n_inst if cache_bytes < (1 << 28) else 1
            xs, cks, cvs = [], [], []
            for _ in range(n_cache):
                x = torch.randn((B, T, shape.hidden), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16) \
                    if B * T * shape.hidden < (1 << 30) else \
                    torch.cat([torch.randn((1, T, shape.hidden), generator=gen, device=dev, dtype=torch.bfloat16)
                               for _ in range(B)])
                ck = (torch.randn((B, T, shape.n_kv_heads, shape.head_dim), generator=gen, device=dev,
                                  dtype=torch.bfloat16) * kv_std)
                cv = (torch.randn((B, T, shape.n_kv_heads, shape.head_dim), generator=gen, device=dev,
                                  dtype=torch.bfloat16) * kv_std)
                xs.append(x); cks.append(ck); cvs.append(cv)
            cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
            cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
            for place in SWEEP_PLACE:
                lay = wl.sweep_layout(L, B, place, "none")
                l = lay.affix_start
                for x, ck, cv in zip(xs, cks, cvs):           # the affix is shared by the batch
                    x[1:, l:l + L] = x[0:1, l:l + L]
                    ck[1:, l:l + L] = ck[0:1, l:l + L]
                    cv[1:, l:l + L] = cv[0:1, l:l + L]
                masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
                req = ab.Context.request(B, T, l, L, masked, None, cos, sin)
                for ratio in SWEEP_RATIO:
                    K = ab.k_from_ratio(L, ratio)
                    ctx = ab.Context.for_shape(shape, B, T, L, K, lay.n_masked, dev)
                    scores = torch.zeros((B, L), dtype=torch.float32, device=dev)
                    anchors = torch.zeros((B, K), dtype=torch.int32, device=dev)
                    y = torch.zeros((B, K, shape.hidden), dtype=torch.bfloat16, device=dev)

                    def step(i):
                        c = i % n_cache
                        ctx.layer_step(winst[i % n_inst][1], req, ab.Context.kv(cks[c], cvs[c]), xs[c], 0, ratio, flags,
                                       scores, anchors, y)

                    for i in range(3):
                        step(i)
                    torch.cuda.synchronize()
                    e0.record(); step(3); e1.record()
                    torch.cuda.synchronize()
                    steps = int(min(args.steps, max(3, 0.2 / max(e0.elapsed_time(e1) * 1e-3, 1e-6))))
                    l0 = ctx.launch_count()
                    c0 = len(sampler.sm)
                    e0.record()
                    for i in range(steps):
                        step(i)
                    e1.record()
                    torch.cuda.synchronize()
                    clk = sampler.sm[c0:] or sampler.sm[-1:]
                    launches += ctx.launch_count() - l0
                    s_step = e0.elapsed_time(e1) * 1e-3 / steps
                    ctx.stage_timing(True)
                    stage = {s: 0.0 for s in ab.STAGES}
                    for i in range(min(steps, 5)):
                        step(i)
                        for s_, v in ctx.read_stage_times().items():
                            stage[s_] += v / min(steps, 5)
                    ctx.stage_timing(False)
                    assert ctx.poll_status() == 0, "device status word set during the sweep"
                    step_bytes, step_flops, _, _, n_r = step_work(shape, lay, K)
                    t_hbm, t_tc = step_bytes / (peaks["hbm_gbs"] * 1e9), step_flops / (peaks["tflops"] * 1e12)
                    floor = max(t_hbm, t_tc)
                    points.append({"L": L, "B": B, "place": place, "ratio": ratio, "K": K, "rows": n_r, "steps": steps,
                                   "us": s_step * 1e6, "sm_mhz": float(np.median(clk)) if clk else None, "floor_us": floor * 1e6, "bound": "hbm" if t_hbm >= t_tc else "tensor",
                                   "frac": floor / s_step, "gbs": step_bytes / s_step / 1e9,
                                   "tflops": step_flops / s_step / 1e12,
                                   "tensor_util": step_flops / s_step / 1e12 / peaks["tflops"],
                                   "stage_us": {k: round(v * 1e3, 1) for k, v in stage.items()}})
                    tot_tokens += B * K * steps
                    tot_s += s_step * steps
                    del ctx, scores, anchors, y
            del xs, cks, cvs
            torch.cuda.empty_cache()
    sampler.stop_flag = True
    sampler.join()
    fr = sorted(p["frac"] for p in points)
    by = {b: sorted(p["frac"] for p in points if p["bound"] == b) for b in ("hbm", "tensor")}
    med = lambda v: (v[len(v) // 2] if v else None)  # noqa: E731
    if args.sweep_out:
        with open(args.sweep_out, "w") as f:
            f.write("| L | B | place | ratio | K | rows | µs/layer-step | SM MHz | floor µs | bound | frac | TFLOP/s | GB/s | "
                    + " | ".join(ab.STAGES) + " |\n")
            f.write("|" + "---|" * (13 + len(ab.STAGES)) + "\n")
            for p in points:
                f.write(f"| {p['L']} | {p['B']} | {p['place']} | {p['ratio']} | {p['K']} | {p['rows']} | {p['us']:.1f} | "
                        f"{p['sm_mhz'] or 0:.0f} | {p['floor_us']:.1f} | {p['bound']} | {p['frac']:.3f} | {p['tflops']:.1f} | {p['gbs']:.0f} | "
                        + " | ".join(f"{p['stage_us'][s_]:.1f}" for s_ in ab.STAGES) + " |\n")
    print(json.dumps({
        "metric": METRIC, "value": tot_tokens / tot_s, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": 3,
        "ms_per_step": tot_s / max(1, sum(p["steps"] for p in points)) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (device-drawn, timing only)",
        "config": {"workload": f"cfg5 sweep: LLaDA-8B layer, affix {list(Ls)} x ratio {list(SWEEP_RATIO)} x batch {list(Bs)} x "
                               f"placement {list(SWEEP_PLACE)}, 64 request + 32 masked rows, anchors only; value = anchors "
                               "refreshed over all points / time over all points", "benchmark_config": 5,
                   "l2": f"{n_inst} weight instances rotated; caches rotated while smaller than 256 MB"},
        "clocks": sampler.summary(), "gpu_launches": int(launches),
        "roofline": {"bound": "mixed", "frac_min": fr[0], "frac_median": med(fr), "frac_max": fr[-1],
                     "frac_median_hbm_bound": med(by["hbm"]), "frac_median_tensor_bound": med(by["tensor"]),
                     "peak_source": peaks["source"], "peak_hbm_gbs": peaks["hbm_gbs"], "peak_tflops": peaks["tflops"]},
        "points": points,
    }))


def run_generate(args, e):
    """Benchmark configuration 3, one whole block decoded with the refresh-then-decode schedule
    (acache_generate_block): one refresh pass over R = anchors + all request rows, then decode passes
    over the block's 32 rows until every request has committed its block (random-init weights never
    reach the 0.9 threshold, so every pass commits exactly one token per request: the longest schedule)."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    ctx, dist, dev, world, rank = e["ctx"], e["dist"], e["dev"], e["world"], e["rank"]
    lay, B, T, L, K, n, V, n_blk, shape, n_layers = (e["lay"], e["B"], e["T"], e["L"], e["K"], e["n"], e["V"], e["n_blk"],
                                                   e["shape"], e["n_layers"])
    ids0 = torch.from_numpy(e["ids"]).to(dev)
    dids = e["dids"]
    block_pos = torch.from_numpy(np.ascontiguousarray(lay.masked_pos[:, :n_blk])).to(dev)
    req_d = ab.Context.request(B, T, lay.affix_start, L, e["masked"], block_pos, e["cos"], e["sin"], token_ids=dids, n_embed=V)
    rows_d = torch.arange(n_blk, dtype=torch.int32, device=dev).repeat(B, 1).contiguous()
    left = torch.zeros((B,), dtype=torch.int32, device=dev)

    shared = bool(args.shared)
    if shared:
        # one copy of every layer's cache serves the batch (batch_stride 0); what a request changes lives in its
        # private slots [B, K + e, Hkv, d] per layer
        kvs_sh = [ab.KV(e["dk"][i][0:1].data_ptr(), e["dv"][i][0:1].data_ptr(), 0, T) for i in range(n_layers)]
        ks = [torch.zeros((B, n, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev) for _ in range(n_layers)]
        vs = [torch.zeros_like(t) for t in ks]

    def block():
        dids.copy_(ids0)
        if shared:
            return ctx.generate_block_shared(e["lws"], kvs_sh, e["req"], req_d, e["embed"], e["da"], K, ks, vs, e["ya"], e["yb"],
                                             e["dbr"], rows_d, n_blk, e["gain"], e["w_lm"], V, 0.9, V - 1, n_blk + 1,
                                             e["token"], e["conf"], e["commit"], left)
        return ctx.generate_block(e["lws"], e["kvs"], e["req"], req_d, e["embed"], e["da"], K, e["ya"], e["yb"], e["dbr"], rows_d,
                                  n_blk, e["gain"], e["w_lm"], V, 0.9, V - 1, n_blk + 1, e["token"], e["conf"], e["commit"], left)

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    block()                                   # warm-up: one whole block (33 model passes at most)
    sync_all()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    l0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_blocks = max(1, min(args.steps, 3))
    e0.record()
    passes = 0
    for _ in range(n_blocks):
        passes += block()
    e1.record()
    sync_all()
    sampler.stop_flag = True
    sampler.join()
    launches = ctx.launch_count() - l0
    ms_block = sharding.max_over_ranks(e0.elapsed_time(e1), dist, dev) / n_blocks
    flags = ctx.poll_status()
    assert flags == 0, f"device status flags {flags:#x}"
    assert int(left.sum().item()) == 0, "the block was not fully decoded"
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    peaks = load_peaks()
    tokens = world * B * n_blk
    print(json.dumps({
        "metric": "generated_tokens_per_s", "value": tokens / (ms_block * 1e-3), "unit": "generated tokens/s",
        "n_gpus": world, "steps": n_blocks, "warmup": 1, "ms_per_step": ms_block, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic; random-init weights: no confidence reaches the threshold, so each pass commits one token per request",
        "config": {"workload": f"cfg3 block decode: LLaDA-8B shapes, {n_layers} layers, vocab {V}, batch {B}/GPU sharing a {L}-token "
                               f"prefix affix, one {n_blk}-token block per request: 1 refresh pass ({n} rows per request, K={K}) + "
                               f"decode passes over the block's {n_blk} rows; "
                               + ("shared affix storage: one cache per layer for the batch + private slots"
                                  if shared else "one working cache per request and layer"),
                   "benchmark_config": 3, "layers": n_layers, "storage": "shared" if shared else "private",
                   "model_passes_per_block": passes / n_blocks, "parallelism": f"request-sharded x{world}"},
        "clocks": sampler.summary(), "gpu_launches": int(launches), "ms_per_block": ms_block,
        "ms_per_model_pass": ms_block / (passes / n_blocks),
        "e2e": {"value": tokens / (ms_block * 1e-3), "unit": "generated tokens/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": int(4 * B * passes / n_blocks),
                "note": "the schedule reads 4 bytes per request back after every model pass (inside the timed region)"},
        "roofline": {"bound": "mixed", "peak_source": peaks["source"], "note": "refresh pass tensor-bound, decode passes (512 rows) near the weight-streaming floor"},
    }))
    if dist:
        dist.destroy_process_group()


def run_shared(args):
    """Shared affix storage (Section 4.1) against one working cache per request, one layer of benchmark
    configuration 3 or 4: the same refresh (scores, selection, R = anchors + all request rows) once through
    acache_layer_step on B private caches [B, T, Hkv, d], once through acache_score_anchors /
    acache_select_topk / acache_recompute_anchors on ONE cache [T, Hkv, d] (batch_stride 0) with every
    request's fresh rows in its private k_new / v_new [B, K+e, Hkv, d]."""
    import torch
    from paper_2608_26140_b200 import binding as ab
    from paper_2608_26140_b200 import build as abuild
    if int(os.environ.get("RANK", "0")) != 0:
        return
    dev = "cuda:0"
    torch.cuda.set_device(0)
    abuild.build()
    cfg = args.config
    shape = wl.LLADA_8B if cfg == 3 else wl.DREAM_7B
    lay = wl.config_layout(cfg, "all", n_masked=32, batch=args.batch)
    B, T, L, P = lay.batch, lay.ctx_len, lay.affix_len, lay.n_extra
    K = ab.k_from_ratio(L, RATIO)
    n = K + P
    w = wl.layer_weights(shape, cfg, 0)
    wd = {k: (ab.to_device_bf16(v, dev) if v is not None else None) for k, v in w.items()}
    lw = ab.Context.weights(wd)
    ck, cv = wl.random_kv_cache(shape, lay, wl.SEED_BASE + 4096 * cfg + 30)
    dk, dv = ab.to_device_bf16(ck, dev), ab.to_device_bf16(cv, dev)
    sk, sv = dk[0:1].clone(), dv[0:1].clone()                       # the shared copy
    gen = torch.Generator(device=dev); gen.manual_seed(wl.SEED_BASE + 4096 * cfg + 31)
    x = torch.randn((B, T, shape.hidden), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    x[1:, lay.affix_start:lay.affix_start + L] = x[0:1, lay.affix_start:lay.affix_start + L]
    cos_h, sin_h = wl.rope_table(T, shape.head_dim, shape.rope_theta)
    cos, sin = torch.from_numpy(cos_h).to(dev), torch.from_numpy(sin_h).to(dev)
    masked = torch.from_numpy(lay.masked_pos.copy()).to(dev)
    extra = torch.from_numpy(lay.extra_rows.copy()).to(dev)
    req = ab.Context.request(B, T, lay.affix_start, L, masked, extra, cos, sin)
    ctx = ab.Context.for_shape(shape, B, T, L, n, lay.n_masked, dev)
    scores = torch.zeros((B, L), dtype=torch.float32, device=dev)
    anchors = torch.zeros((B, K), dtype=torch.int32, device=dev)
    y = torch.zeros((B, n, shape.hidden), dtype=torch.bfloat16, device=dev)
    k_new = torch.zeros((B, n, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device=dev)
    v_new = torch.zeros_like(k_new)
    q_mask = torch.randn((B, lay.n_masked, shape.n_heads, shape.head_dim), generator=gen, device=dev,
                         dtype=torch.float32).mul_(0.02 * float(np.sqrt(shape.hidden))).to(torch.bfloat16)
    kv_priv = ab.Context.kv(dk, dv)
    kv_shared = ab.KV(sk.data_ptr(), sv.data_ptr(), 0, T)

    def private_step():
        ctx.layer_step(lw, req, kv_priv, x, 0, RATIO, ab.F_SCORE | ab.F_SELECT, scores, anchors, y)

    def shared_step():
        ctx.score_anchors(req, q_mask, kv_shared, scores)
        ctx.select_topk(scores, B, L, K, anchors)
        ctx.recompute_anchors(lw, req, kv_shared, x, 0, anchors, K, k_new, v_new, y)

    if args.decode:
        # one layer of a decode pass: only the first 32 masked rows of every request are recomputed.  Private caches:
        # acache_layer_step with ratio 0 on those rows; shared storage: the slots as a refresh left them
        # (shared_step above), then acache_recompute_rows_shared for the block's rows.
        n_blk = 32
        blk = np.ascontiguousarray(lay.masked_pos[:, :n_blk])
        dblk = torch.from_numpy(blk.copy()).to(dev)
        req_blk = ab.Context.request(B, T, lay.affix_start, L, masked, dblk, cos, sin)
        where = {int(p_): i for i, p_ in enumerate(lay.extra_rows[0])}
        slot_rows = torch.from_numpy(np.stack([[K + where[int(p_)] for p_ in blk[b]] for b in range(B)]).astype(np.int32)).to(dev)
        xb = torch.randn((B, n_blk, shape.hidden), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        yb = torch.zeros((B, n_blk, shape.hidden), dtype=torch.bfloat16, device=dev)
        shared_step()                                   # fills k_new / v_new and the anchors
        torch.cuda.synchronize()

        def private_step():                             # noqa: F811
            ctx.layer_step(lw, req_blk, kv_priv, xb, 1, 0.0, 0, None, None, yb)

        def shared_step():                              # noqa: F811
            ctx.recompute_rows_shared(lw, req_blk, req, kv_shared, xb, 1, anchors, K, slot_rows, k_new, v_new, yb)

    res = {}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, fn in (("private", private_step), ("shared", shared_step)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / args.steps
        ctx.stage_timing(True)
        fn()
        res[name + "_stage_us"] = {k_: round(v * 1e3, 1) for k_, v in ctx.read_stage_times().items() if v}
        ctx.stage_timing(False)
    assert ctx.poll_status() == 0
    row = shape.n_kv_heads * shape.head_dim * 2 * 2            # K and V bytes of one position
    kv_private, kv_shared_b = B * T * row, T * row + B * n * row
    print(json.dumps({
        "metric": METRIC, "value": B * K / (res["shared"] * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": 3,
        "ms_per_step": res["shared"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"cfg{cfg} one layer, shared affix storage: {shape.name}, batch {B} sharing a {L}-token affix, "
                               + (f"decode pass: the block's 32 rows per request ({B * 32} rows) against {n} slot rows per request"
                                  if args.decode else f"K={K} anchors + {P} request rows per request ({B * n} rows)"),
                   "benchmark_config": cfg, "pass": "decode" if args.decode else "refresh"},
        "shared_storage": {"ms_per_layer": res["shared"], "kv_bytes_per_layer": kv_shared_b, "stage_us": res["shared_stage_us"],
                           "note": "the masked-row queries are given (acache_score_anchors); the split calls do not write the cache"},
        "private_caches": {"ms_per_layer": res["private"], "kv_bytes_per_layer": kv_private, "stage_us": res["private_stage_us"],
                           "note": "acache_layer_step including the masked-row query projection"},
        "kv_bytes_ratio": kv_shared_b / kv_private,
    }))


def cpu_baseline(case, shape, lay):
    """The oracle as it stands, timed on this machine's host cores on full layer-steps of the workload: the same
    program and the same protocol as `--impl reference` (weights converted bf16 -> fp64 once, outside the timed
    steps; numpy's BLAS threads as the box gives them)."""
    from oracle import acache_oracle as orc
    L = lay.affix_len
    K = orc.k_from_ratio(L, RATIO)
    w64 = {k: (orc.bf16_bits_to_f64(v) if v is not None else None) for k, v in case.weights.items()}

    def one_step():
        for b in range(lay.batch):
            orc.layer_step(w64, shape, case.x[b], case.cache_k[b], case.cache_v[b], lay.ctx_len,
                           lay.affix_start, L, lay.masked_pos[b], lay.extra_rows[b], case.rope_cos, case.rope_sin, K=K)

    one_step()                                   # warm-up (page-in, BLAS thread pool)
    t0 = time.perf_counter()
    reps = 0
    while True:
        one_step()
        reps += 1
        if time.perf_counter() - t0 > 10.0 or reps >= 20:
            break
    dt = (time.perf_counter() - t0) / reps
    cores = _threads_used()
    return {"value": lay.batch * K / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{reps} full layer-step(s) of the same workload ({lay.batch} request(s), {K} anchors each), "
                      f"{dt:.3f} s per step; weights converted bf16 -> fp64 once, outside the timed steps; "
                      f"{cores} BLAS threads (numpy matmul, fp64)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="benchmark configuration (2 = LLaDA-8B layer, batch 1)")
    ap.add_argument("--extra", default="none", choices=["none", "all", "masked"],
                    help="request-specific rows recomputed with the anchors")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--instances", type=int, default=4, help="weight/cache instances rotated between steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--blocks", type=int, default=0,
                    help="timed blocks of --steps steps (0: at least 50 and about a second of GPU time; a small number keeps a "
                         "profiler run short)")
    ap.add_argument("--probe", action="store_true",
                    help="--config 3 or 4: time one layer of the selection-time probe (all request rows, no anchors, scores "
                         "accumulated from the layer's own attention)")
    ap.add_argument("--no-extra", action="store_true",
                    help="default run only: skip the short configuration-3 / sweep / selector measurements (key `extra`)")
    ap.add_argument("--layers", type=int, default=32, help="layers of the --config 3 denoising step")
    ap.add_argument("--shared", action="store_true",
                    help="--config 3 or 4: one layer with shared affix storage (batch_stride 0) against private caches")
    ap.add_argument("--decode", action="store_true",
                    help="with --shared: time one layer of a decode pass (32 rows per request) instead of the refresh")
    ap.add_argument("--generate", action="store_true",
                    help="--config 3: decode one whole 32-token block per request (refresh + decode passes); "
                         "with --shared over shared affix storage")
    ap.add_argument("--sweep-affix", default=None, help="--config 5: comma-separated affix lengths (default 512,2048,8192)")
    ap.add_argument("--sweep-batch", default=None, help="--config 5: comma-separated batch sizes (default 1,8,64)")
    ap.add_argument("--sweep-out", default=None, help="--config 5: also write the points as a markdown table to this file")
    ap.add_argument("--rank-echo", action="store_true", help=argparse.SUPPRESS)   # every rank prints who it is and exits (no GPU)
    args = ap.parse_args()
    plan, world = sharding.launch_plan(args.gpus, os.environ)
    if plan == "refuse":
        raise SystemExit(f"--gpus {args.gpus} but this process is rank of a {world}-rank job: start it with "
                         f"--nproc-per-node {args.gpus} (or without a launcher: bench.py starts its own ranks)")
    if plan == "spawn":
        # no launcher around this process: start the N ranks (one per GPU) and hand them the same arguments
        import subprocess
        cmd = sharding.torchrun_command(os.path.abspath(__file__), sys.argv[1:], args.gpus, sharding.free_port())
        raise SystemExit(subprocess.call(cmd))
    if args.rank_echo:
        print(json.dumps({"rank": int(os.environ.get("RANK", "0")), "world": world, "gpus": args.gpus}), flush=True)
        return
    if args.impl == "reference":
        run_reference(args)
    elif args.probe and args.config in (3, 4):
        print(json.dumps(probe_layer(args.config, args.batch, max(args.steps, 1), load_peaks(), "cuda:0")))
    elif args.shared and args.config in (3, 4) and not args.generate:
        run_shared(args)
    elif args.config == 3:
        run_denoise(args)
    elif args.config == 5:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
