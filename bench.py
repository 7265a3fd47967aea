"""Benchmark of the FreqFormer attention forward on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 64k|256k|1m|128k_sweep]
  python bench.py --impl reference ...        # the fp64 oracle timed on the host cores

A step is one ff_forward (transform, band split, router, three band operators, summary
exchange, recombination, inverse transform) over one batch of the synthetic workload.  With
N > 1 (torchrun) every rank runs its own replica of the batch: samples are independent problems,
so there is no data-path collective and the scaling is weak.  One JSON line is printed by rank 0.
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

from paper_2604_22808_b200 import configs as C          # noqa: E402
from paper_2604_22808_b200 import inputs as I           # noqa: E402

METRIC = "freqformer_attn_layer_tokens_per_s"

# dram__bytes_read.sum + dram__bytes_write.sum of the transform kernels per token and head, from the ncu
# capture of the 6-head 64K case (forward: the passes over Q, K and V; inverse: the passes over one tensor).
FP32_FMA_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 74.5: plain fp32 FMA rate of the GPU (unit counts x max clock)
# [0]: three separate axis passes; [1]: two axes in one launch (64K-class grids)
NCU_DRAM_BYTES_PER_TOKEN_HEAD = {"transform": (6554.0, 4380.0), "inverse": (2345.0, 1985.0)}
TRANSFORM_KERNELS = {"transform": ("dct_tc_kernel x3 (transform stage)", "dct2_tc_kernel + dct_tc_kernel (transform stage)"),
                     "inverse": ("exchange_tc_kernel + dct_tc_kernel x3 (inverse stage)",
                                 "exchange_tc_kernel + dct_tc_kernel + dct2_tc_kernel (inverse stage)")}
# Reported beside the 64K line by the default run: the larger workloads with the router's allocation and the
# 64K grid with every band operator present.
EXTRA_WORKLOADS = {"256k": ("256k", ""), "1m": ("1m", ""), "64k_forced_8_8_8": ("64k", "8,8,8")}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------
# Work model of one layer (per workload, given the head allocation)
# ---------------------------------------------------------------------------------------------
def band_sizes(cfg):
    L, M = cfg.low_cut, cfg.mid_cut
    n_low = L[0] * L[1] * L[2]
    n_mid = M[0] * M[1] * M[2] - n_low
    return n_low, -(-n_low // cfg.r), n_mid, cfg.N - M[0] * M[1] * M[2]


def interactions(cfg):
    """Scored (query, key) pairs of one head per band operator, and of the exchange."""
    n_low, n_bar, n_mid, n_high = band_sizes(cfg)
    nb = -(-n_mid // cfg.b)
    i_mid = 0
    for c in range(min(cfg.s, nb)):
        n_c = sum(min(cfg.b, n_mid - J * cfg.b) for J in range(c, nb, cfg.s))
        i_mid += n_c * n_c
    R = min(cfg.R, n_high - 1)
    i_high = n_high * (2 * R + 1) - R * (R + 1)
    return n_bar * n_bar, i_mid, i_high


def issued_pairs(cfg):
    """(query, key) pairs the tensor-core attention kernel computes per head and band, whole
    128 x 128 tiles including their masked parts: mid = every tile pair of a residue class, high =
    the key tiles that meet a query tile's window, low = every tile pair of the pooled band."""
    n_low, n_bar, n_mid, n_high = band_sizes(cfg)
    T = 128
    nb = -(-n_mid // cfg.b)
    i_mid = 0
    for c in range(min(cfg.s, nb)):
        blocks = len(range(c, nb, cfg.s))
        nt = -(-blocks * cfg.b // T)
        i_mid += nt * nt * T * T
    i_high = 0
    for qt in range(-(-n_high // T)):
        q0 = qt * T
        lo, hi = max(0, q0 - cfg.R), min(n_high, q0 + T + cfg.R)
        # key tiles start at the pair's first key (multiples of 128 from there); count tiles meeting [lo, hi)
        i_high += (-(-(hi - lo) // T)) * T * T
    nt_low = -(-n_bar // T)
    return nt_low * nt_low * T * T, i_mid, i_high


def layer_work(cfg, alloc):
    """Useful attention FLOPs (4 d per pair: QK^T and PV) and algorithmic HBM bytes of one forward."""
    d, e = cfg.head_dim, (4 if cfg.dtype == "fp32" else 2)
    n_low, n_bar, n_mid, n_high = band_sizes(cfg)
    pairs = interactions(cfg)
    u = cfg.N * d * e
    flops = 0
    bytes_attn = 0
    for mask in alloc:
        for l, (p, n_l) in enumerate(zip(pairs, (n_bar, n_mid, n_high))):
            if mask >> l & 1:
                flops += 4 * d * p
                bytes_attn += 4 * n_l * d * e
    heads = len(alloc)
    exch_pairs = heads * 2 * cfg.m * cfg.N
    # forward transform, counted strictly: read Q, K, V, write V~ in full but Q~, K~ only for the bands the
    # head's mask executes (what the band operators go on to read)
    frac_exec = [sum(n_l for l, n_l in enumerate((n_low, n_mid, n_high)) if mask >> l & 1) / cfg.N for mask in alloc]
    bytes_transform_strict = sum((4 + 2 * f) * u for f in frac_exec)
    return {
        "bytes_transform_strict": bytes_transform_strict,
        "attn_flops": flops,
        "exchange_flops": 4 * d * exch_pairs,
        "transform_flops": heads * 4 * 2 * cfg.N * (cfg.T + cfg.H + cfg.W) * d,
        # forward transform: read Q,K,V, write Q~,K~,V~; inverse: read Y^, write out
        "bytes_transform": heads * 6 * u,
        "bytes_inverse": heads * 2 * u,
        "bytes_attention": bytes_attn,
    }


# ---------------------------------------------------------------------------------------------
# Clock sampling during the timed region
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        """`index` is the CUDA device index; NVML numbers devices differently when CUDA_VISIBLE_DEVICES
        is set, so the handle is looked up by the device's UUID (read-only queries throughout)."""
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                try:
                    self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
                except Exception:
                    self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _loop(self):
        while not self._stop.is_set():
            try:
                self.samples.append(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM))
                mask = self._nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on a bounded sample
# ---------------------------------------------------------------------------------------------
def oracle_sample_time(cfg, alloc):
    """Times the oracle's whole layer for one head per band type present in `alloc` on the full
    grid (transform of Q,K,V, that band's operator over every row, summaries, exchange, inverse)
    and extrapolates to all heads by the allocation.  Returns (tokens/s, seconds, cores, text)."""
    from threadpoolctl import threadpool_info
    from oracle import freqformer_oracle as O
    weights = I.router_weights(cfg)
    U = I.summary_projection(cfg)
    per_band = {}
    spent = 0.0
    for l, bit in enumerate((1, 2, 4)):
        heads_l = [h for h, mk in enumerate(alloc) if mk == bit]
        if not heads_l or spent > 60.0:          # keep the sample bounded on the large workloads
            continue
        h = heads_l[0]
        Q, K, V = (I.qkv_head(cfg, t, 0, h)[None] for t in range(3))
        t0 = time.perf_counter()
        O.forward_sample(cfg, Q, K, V, weights, U, cfg.timesteps[0], alloc=[bit])
        per_band[bit] = time.perf_counter() - t0
        spent += per_band[bit]
    total = sum(per_band.get(mk, max(per_band.values())) for mk in alloc) * (cfg.batch)
    cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    text = (f"one head per allocated band type ({len(per_band)} of {len(alloc)} heads) on the full {cfg.name} grid, "
            f"whole layer each, extrapolated by the head allocation")
    return cfg.batch * cfg.N / total, spent, cores, text


# Head allocation the seeded random-init router produces at each workload's first timestep (heads per band and
# sample), so that the reference arm times the same configuration as the CUDA arm without a GPU.  The fp64 oracle
# yields the same counts (the full-size parity tests compare them).
ROUTER_HEADS_PER_BAND = {"64k": (8, 0, 16), "256k": (0, 24, 0), "1m": (9, 6, 1), "paper_ref_64k": (0, 12, 4),
                         "paper_ref_1m": (16, 0, 0)}


def config_record(cfg, timestep, forced: bool, alloc):
    io_mb = 3 * cfg.batch * cfg.heads * cfg.N * cfg.head_dim * (4 if cfg.dtype == "fp32" else 2) / 1e6
    return {"workload": cfg.name, "grid": list(cfg.grid), "batch": cfg.batch, "heads": cfg.heads,
            "head_dim": cfg.head_dim, "timestep": timestep, "allocation": "forced" if forced else "router",
            "heads_per_band": [alloc.count(1), alloc.count(2), alloc.count(4)],
            "l2": "inputs (%.0f MB) larger than L2" % io_mb}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n = cfg.heads
    forced = forced_allocation(cfg, args.alloc)
    if forced is not None:
        alloc = forced
    elif cfg.name in ROUTER_HEADS_PER_BAND and args.timestep_index == 0:
        c = ROUTER_HEADS_PER_BAND[cfg.name]
        alloc = ([1] * c[0] + [2] * c[1] + [4] * c[2]) * cfg.batch
    else:
        alloc = ([1] * (n // 3) + [2] * (n // 3) + [4] * (n - 2 * (n // 3))) * cfg.batch
    vals = []
    t_all = time.perf_counter()
    for i in range(args.warmup + args.steps):
        if i > 0 and time.perf_counter() - t_all > 240:
            break
        v, spent, cores, text = oracle_sample_time(cfg, alloc)
        if i >= args.warmup or i == args.warmup + args.steps - 1:
            vals.append(v)
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": len(vals), "warmup": args.warmup, "ms_per_step": 1e3 * cfg.batch * cfg.N / value,
            "ms_per_step_is": "extrapolated: each step times one head per allocated band type on the full grid "
                              "(%.1f s of host work) and scales by the allocation" % spent,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_record(cfg, cfg.timesteps[args.timestep_index], forced is not None, alloc),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": text},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# Multi-rank plumbing (replicas only: no data-path collective; used with NCCL on GPUs, gloo in tests)
# ---------------------------------------------------------------------------------------------
def replica_config(cfg, rank: int):
    """Every rank runs its own replica of the batch: same workload, its own seeded inputs."""
    return cfg.scaled(cfg.name, seed=cfg.seed + 1000 * rank) if rank else cfg


def reduce_max(x: float, world: int, device) -> float:
    """Slowest rank's value (the timing every rank reports)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def forced_allocation(cfg, text):
    """'L,M,H' (heads per band, summing to the head count) -> band masks of every (batch, head);
    heads [0,L) run the low band, the next M the mid band, the rest the high band."""
    if not text:
        return None
    n = [int(x) for x in text.split(",")]
    if len(n) != 3 or min(n) < 0 or sum(n) != cfg.heads:
        raise SystemExit(f"--alloc wants L,M,H summing to {cfg.heads} heads")
    return ([1] * n[0] + [2] * n[1] + [4] * n[2]) * cfg.batch


def tensor_core_path_any(cfg) -> bool:
    """Does this workload run on the tensor-core kernels (bf16, head_dim 128 or 64)?"""
    return cfg.dtype == "bf16" and cfg.head_dim in (64, 128)


def aggregate_tokens_per_s(cfg, world: int, ms_step_max: float) -> float:
    """Whole-job throughput: the tokens all ranks processed over the slowest rank's step time."""
    return cfg.batch * cfg.N * world / (ms_step_max * 1e-3)


# ---------------------------------------------------------------------------------------------
# The CUDA arm
# ---------------------------------------------------------------------------------------------
def stage_rooflines(cfg, alloc, stage_ms, peaks):
    """Per stage: achieved algorithmic rate and its fraction of the measured peak that bounds it."""
    work = layer_work(cfg, alloc)
    ms = lambda name: max(stage_ms[name], 1e-9) * 1e-3
    tc = tensor_core_path_any(cfg)
    low_tc = band_sizes(cfg)[1] >= 128
    issued = 4 * cfg.head_dim * sum(sum(p for l, p in enumerate(issued_pairs(cfg)) if (mk >> l & 1) and (l > 0 or low_tc))
                                    for mk in alloc)
    peak_t = peaks["bf16_tflops_sustained"]
    out = {
        "transform": {"bound": "hbm", "gbs": work["bytes_transform_strict"] / ms("transform") / 1e9,
                      "gbs_all_bands_written": work["bytes_transform"] / ms("transform") / 1e9},
        "inverse": {"bound": "hbm", "gbs": work["bytes_inverse"] / ms("inverse") / 1e9},
        "attention": {"bound": "tensor" if tc else "alu", "useful_tflops": work["attn_flops"] / ms("attention") / 1e12,
                      "issued_tflops": issued / ms("attention") / 1e12 if tc else None},
    }
    out["transform"]["frac"] = out["transform"]["gbs"] / peaks["hbm_gbs"]
    out["inverse"]["frac"] = out["inverse"]["gbs"] / peaks["hbm_gbs"]
    out["attention"]["frac"] = out["attention"]["useful_tflops"] / (peak_t if tc else FP32_FMA_TFLOPS)
    out["attention"]["frac_of_nominal_2250"] = out["attention"]["useful_tflops"] / 2250.0 if tc else None
    return out, work


def time_forward(plan, q, k, v, out, alloc_dev, ts, steps, warmup, B, sampler=None):
    """W untimed forwards, then K timed ones (CUDA events on the launching stream).  Returns the mean
    ms per step, the sorted per-step times, the mean stage times and the launches per stage."""
    import torch
    for _ in range(warmup):
        plan.forward(q, k, v, out, alloc=alloc_dev, timesteps=ts)
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    stage_ms = {name: 0.0 for name in B.STAGES}
    stage_launches = {}
    ev[0].record()
    for i in range(steps):
        plan.forward(q, k, v, out, alloc=alloc_dev, timesteps=ts)
        ev[i + 1].record()
        for name, (ms, n) in plan.stage_times().items():       # waits for this step's last event
            stage_ms[name] += ms / steps
            stage_launches[name] = n
    torch.cuda.synchronize()
    per_step = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
    return ev[0].elapsed_time(ev[-1]) / steps, per_step, stage_ms, stage_launches


def extra_workload(name, alloc_text, args, dev, local, peaks):
    """One more workload of the metric's 64K-1M range, device-timed only: inputs drawn on the GPU,
    router-driven or forced allocation, stage times and per-stage roofline fractions."""
    import torch
    from paper_2604_22808_b200 import binding as B
    cfg = C.BY_NAME[name]
    q, k, v = (I.qkv_full_device(cfg, t, dev) for t in range(3))
    out = torch.empty_like(q)
    plan = B.Plan(cfg, I.router_weights(cfg), device=dev)
    plan.set_profiling(True)
    ts = [cfg.timesteps[0]] * cfg.batch
    forced = forced_allocation(cfg, alloc_text)
    alloc_dev = None if forced is None else torch.tensor(forced, dtype=torch.uint8, device=dev)
    sampler = ClockSampler(local)
    steps = max(3, min(args.steps, 10))
    ms_step, per_step, stage_ms, stage_launches = time_forward(plan, q, k, v, out, alloc_dev, ts, steps, 3, B, sampler)
    clocks = sampler.stop()
    if plan.device_status() != 0:
        raise RuntimeError(B.library().ff_last_error(plan.handle).decode())
    alloc = forced if forced is not None else plan.tap(B.TAP_ALLOC).cpu().numpy().tolist()
    stages, work = stage_rooflines(cfg, alloc, stage_ms, peaks)
    res = {"kernels": plan.kernel_info(), "grid": list(cfg.grid), "batch": cfg.batch, "heads": cfg.heads, "head_dim": cfg.head_dim,
           "allocation": "router" if forced is None else "forced", "timestep": ts[0],
           "heads_per_band": [alloc.count(1), alloc.count(2), alloc.count(4)],
           "inputs": "drawn on the device (torch CUDA generator), same distribution as the parity tests' host inputs",
           "steps": steps, "warmup": 3, "ms_per_step": ms_step, "ms_per_step_best": per_step[0],
           "tokens_per_s": cfg.batch * cfg.N / (ms_step * 1e-3), "stages_ms": stage_ms, "stage_launches": stage_launches,
           "stage_roofline": stages, "useful_attention_tflops_whole_step": work["attn_flops"] / (ms_step * 1e-3) / 1e12,
           "clocks": clocks}
    plan.destroy()
    del q, k, v, out, plan
    torch.cuda.empty_cache()
    return res


def projected_workload(name, args, dev, peaks):
    """The layer with its Q/K/V and output projections (ff_forward_projected) on one workload: device time of the
    whole call, and of the two projection GEMMs as the difference to the attention path alone."""
    import torch
    from paper_2604_22808_b200 import binding as B
    cfg = C.BY_NAME[name]
    D = cfg.heads * cfg.head_dim
    gen = torch.Generator(device=dev)
    gen.manual_seed(4242 + cfg.seed)
    x = torch.randn((cfg.batch, cfg.N, D), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    wqkv = (torch.randn((3, D, D), generator=gen, device=dev, dtype=torch.float32) / D ** 0.5).to(torch.bfloat16)
    wo = (torch.randn((D, D), generator=gen, device=dev, dtype=torch.float32) / D ** 0.5).to(torch.bfloat16)
    out = torch.empty_like(x)
    plan = B.Plan(cfg, I.router_weights(cfg), host_staging=True, device=dev)
    plan.set_profiling(True)
    ts = [cfg.timesteps[0]] * cfg.batch
    steps = max(3, min(args.steps, 10))
    for _ in range(3):
        plan.forward_projected(x, wqkv, wo, out, timesteps=ts)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    inner = 0.0
    ev[0].record()
    for _ in range(steps):
        plan.forward_projected(x, wqkv, wo, out, timesteps=ts)
        inner += sum(ms for ms, _ in plan.stage_times().values())
    ev[1].record()
    torch.cuda.synchronize()
    if plan.device_status() != 0:
        raise RuntimeError(B.library().ff_last_error(plan.handle).decode())
    ms_step = ev[0].elapsed_time(ev[1]) / steps
    ms_proj = ms_step - inner / steps
    flops = 2.0 * cfg.batch * cfg.N * D * 4 * D
    res = {"grid": list(cfg.grid), "heads": cfg.heads, "head_dim": cfg.head_dim, "model_width": D, "steps": steps,
           "ms_per_step": ms_step, "tokens_per_s": cfg.batch * cfg.N / (ms_step * 1e-3), "projections_ms": ms_proj,
           "projections_tflops": flops / (ms_proj * 1e-3) / 1e12,
           "projections_frac_of_sustained_bf16": flops / (ms_proj * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]}
    plan.destroy()
    del x, wqkv, wo, out, plan
    torch.cuda.empty_cache()
    return res


def run_cuda(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2604_22808_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    dt = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
    cfg_r = replica_config(cfg, rank)
    big = cfg.N * cfg.heads * cfg.batch > 3 * 2 ** 20            # drawing on the host would take minutes
    if big:
        q, k, v = (I.qkv_full_device(cfg_r, t, dev) for t in range(3))
        host = None
    else:
        host = [torch.from_numpy(I.qkv_full(cfg_r, t)).to(dt).pin_memory() for t in range(3)]
        q, k, v = (x.to(dev, non_blocking=True) for x in host)
    out = torch.empty_like(q)
    weights = I.router_weights(cfg)
    do_e2e = not args.no_e2e and host is not None
    plan = B.Plan(cfg, weights, host_staging=do_e2e, device=dev)
    plan.set_profiling(True)
    plan.set_attention_impl(args.kernel_select)
    ts = [cfg.timesteps[args.timestep_index]] * cfg.batch
    forced = forced_allocation(cfg, args.alloc)
    alloc_dev = None if forced is None else torch.tensor(forced, dtype=torch.uint8, device=dev)
    alloc_np = None if forced is None else np.asarray(forced, np.uint8)
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max_(x):
        return reduce_max(x, world, dev)

    # device-resident timing
    for _ in range(args.warmup):
        plan.forward(q, k, v, out, alloc=alloc_dev, timesteps=ts)
    barrier()
    sampler = ClockSampler(local)
    ms_local, per_step, stage_ms, stage_launches = time_forward(plan, q, k, v, out, alloc_dev, ts, args.steps, 0, B, sampler)
    barrier()
    clocks = sampler.stop()
    ms_step = reduce_max_(ms_local)
    launches = plan.last_launches()
    kinfo = plan.kernel_info()
    if plan.device_status() != 0:
        raise RuntimeError(B.library().ff_last_error(plan.handle).decode())
    alloc = forced if forced is not None else plan.tap(B.TAP_ALLOC).cpu().numpy().tolist()
    pi = [None] if forced is not None else plan.tap(B.TAP_PI).cpu().numpy().tolist()

    # end to end through the host-buffer entry point (pinned host memory, copies inside the call)
    e2e_ms = float("nan")
    if do_e2e:
        out_host = torch.empty_like(host[0]).pin_memory()
        for _ in range(min(2, args.warmup)):
            plan.forward_host(host[0], host[1], host[2], out_host, alloc_host=alloc_np, timesteps=ts)
        barrier()
        e2e_steps = max(1, min(args.steps, 5))
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            plan.forward_host(host[0], host[1], host[2], out_host, alloc_host=alloc_np, timesteps=ts)      # synchronises the stream
        e2e_ms = reduce_max_((time.perf_counter() - t0) * 1e3 / e2e_steps)
        barrier()

    io_bytes = q.numel() * q.element_size()
    plan.destroy()
    del q, k, v, out, plan
    torch.cuda.empty_cache()

    if rank == 0:
        peaks = measured_peaks()
        tokens = cfg.batch * cfg.N * world
        stages, work = stage_rooflines(cfg, alloc, stage_ms, peaks)
        # roofline of the dominant stage (achieved and traffic are per launch of the stage's kernel)
        top = max(stage_ms, key=stage_ms.get)
        n_launch = max(1, stage_launches.get(top) or 1)
        heads_total = cfg.batch * cfg.heads
        tensor_core_path = tensor_core_path_any(cfg)                         # otherwise the generic fp32 kernels run
        if top == "attention":
            st = stages["attention"]
            roof = {"bound": st["bound"], "achieved": st["useful_tflops"], "unit": "TFLOP/s", "frac": st["frac"],
                    "peak": peaks["bf16_tflops_sustained"] if tensor_core_path else FP32_FMA_TFLOPS, "traffic": None,
                    "kernel": "attention_tc_kernel" if tensor_core_path else "attention_simt_kernel"}
        else:
            st = stages["transform" if top == "transform" else "inverse"]
            nbytes = work["bytes_transform_strict"] if top == "transform" else work["bytes_inverse"]
            # DRAM bytes per token-head and stage from the ncu capture of the 6-head 64K case; the traffic is
            # proportional to tokens x heads
            fused = int(kinfo["transform_fused"])
            per_token_head = NCU_DRAM_BYTES_PER_TOKEN_HEAD[top][fused] * cfg.head_dim / 128.0
            roof = {"bound": "hbm", "achieved": st["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": st["frac"],
                    "traffic": per_token_head * cfg.N * heads_total / n_launch if tensor_core_path else None,
                    "kernel": (TRANSFORM_KERNELS[top][fused] if tensor_core_path else "dct_pass_kernel (%s stage)" % top),
                    "algorithmic_bytes_per_launch": nbytes / n_launch,
                    "algorithmic_bytes": "read Q,K,V, write V~ and the executed band of Q~,K~" if top == "transform"
                                         else "read the band outputs once, write out once"}
        roof.update({"stage": top, "launches_per_step": stage_launches.get(top), "ms_per_step": stage_ms[top],
                     "ms_per_launch": stage_ms[top] / n_launch, "peak_source": peaks["source"]})
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v_cpu, spent, cores, text = oracle_sample_time(cfg, alloc)
            cpu = {"value": v_cpu, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": text,
                   "seconds": spent}
        line = {
            "metric": METRIC, "value": aggregate_tokens_per_s(cfg, world, ms_step), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": config_record(cfg, ts[0], forced is not None, alloc),
            "router_pi": pi[0],
            "kernels": kinfo,
            "roofline": roof,
            "cpu_baseline": cpu,
            "e2e": ({"value": tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 3 * io_bytes,
                     "d2h_bytes_per_step": io_bytes, "ms_per_step": e2e_ms} if do_e2e else None),
            "gpu_launches": launches * args.steps,
            "clocks": clocks,
            "stages_ms": stage_ms,
            "stage_roofline": stages,
            "ms_per_step_median": per_step[len(per_step) // 2], "ms_per_step_best": per_step[0],
            "ms_x_sm_mhz": ms_step * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
            "useful_attention_tflops": work["attn_flops"] / (ms_step * 1e-3) / 1e12,
            "attention_stage_issued_tflops": stages["attention"]["issued_tflops"],
            "attention_stage_tflops": stages["attention"]["useful_tflops"],
            "transform_stage_gbs": stages["transform"]["gbs"],
            "inverse_stage_gbs": stages["inverse"]["gbs"],
            "paper_context": "simulated estimates only: 9.3-27.3x attention-FLOP and 8.8-20.9x score-traffic reduction vs dense",
            # the same ratio for this workload and allocation, from the interaction counts (exchange included)
            "interaction_reduction_vs_dense": (len(alloc) * cfg.N * cfg.N) / max(1, work["attn_flops"] // (4 * cfg.head_dim)
                                                                              + len(alloc) * 2 * cfg.m * cfg.N),
        }
        # The other workloads of the metric's range, device-timed in the same run (default invocation only)
        if world == 1 and args.workload == "64k" and not args.alloc and not args.heads and not args.no_extra:
            extra = {}
            for key, (name, alloc_text) in EXTRA_WORKLOADS.items():
                extra[key] = extra_workload(name, alloc_text, args, dev, local, peaks)
            extra["64k_with_projections"] = projected_workload("64k", args, dev, peaks)
            line["workloads"] = extra
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="64k")
    ap.add_argument("--timestep-index", type=int, default=0)
    ap.add_argument("--alloc", default="", help="forced heads per band 'L,M,H' instead of the router's allocation")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--heads", type=int, default=0, help="override the number of heads (profiling on a small case)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling)")
    ap.add_argument("--no-extra", action="store_true", help="skip the additional workloads of the default run")
    ap.add_argument("--kernel-select", type=int, default=0,
                    help="ff_plan_set_attention_impl bits: 1 generic attention, 2 generic transform, 4 separate axis passes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    cfg = C.BY_NAME[args.workload]
    if args.heads:
        cfg = cfg.scaled(cfg.name + f"_{args.heads}heads", heads=args.heads)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        args.warmup = max(args.warmup, 3)
        run_cuda(args, cfg)


if __name__ == "__main__":
    main()
