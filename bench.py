#!/usr/bin/env python
"""Benchmark of the paged-attention decode + KV-swap hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2|3|4|5] [--impl ours|reference]

One step = one pa_decode call (plan + partition attention + combine) over one synthetic
batch whose KV cache is resident in HBM.  The headline number is the KV GB/s of that step
(algorithmic bytes / device time): the timed region of K steps is repeated (--repeats) and the
median region is `value`, with minimum and maximum beside it.  The same run times the swap path
(kv_swap_out / kv_swap_in between the device pool and pinned host memory, `swap`, against the
measured host-link rate), the recompute leg (`recompute`), and every other configuration
(`workloads`: the tiny one, the two other decode shapes, the full-size swap churn).  With N > 1
(torchrun) every rank runs the same workload on its own GPU (independent replicas, no
data-path collective); --seq-split and --kv-head-shard share one workload among the ranks.

Rank 0 prints ONE JSON line.
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

METRIC = "decode_attention_kv_gbps"
UNIT = "GB/s"


# --------------------------------------------------------------------------------------
# small helpers
# --------------------------------------------------------------------------------------
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:  # NVML missing: report no clocks rather than fail the bench
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or getattr(
            nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(get_reasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                    "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def aggregate_over_ranks(ms_local: float, units_local: float, dist=None):
    """Whole-job throughput inputs: (max time over ranks, units summed over ranks).

    `dist` is torch.distributed when a process group is initialised, else None.  Works on
    any backend (NCCL on GPUs, gloo in the CPU test)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_local, units_local
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def sample_sequences(spec, token_budget: int, seed: int = 7):
    """Seeded random subset of sequences holding about `token_budget` tokens (at least one)."""
    order = np.random.Generator(np.random.PCG64(seed)).permutation(spec.batch)
    pick, tot = [], 0
    for b in order:
        L = int(spec.seq_lens[b])
        if pick and tot + L > token_budget:
            continue
        pick.append(int(b))
        tot += L
        if tot >= token_budget:
            break
    return sorted(pick), tot


def compact_tables(spec, seqs):
    """Block ids used by `seqs` (concatenated) and their tables remapped onto 0..n-1."""
    ids = np.concatenate([spec.blocks_of(b) for b in seqs]).astype(np.int64)
    remap = {int(p): i for i, p in enumerate(ids)}
    mb = max(len(spec.blocks_of(b)) for b in seqs)
    tables = np.zeros((len(seqs), mb), dtype=np.int32)
    for i, b in enumerate(seqs):
        blk = spec.blocks_of(b)
        tables[i, :len(blk)] = [remap[int(p)] for p in blk]
    return ids, remap, tables, spec.seq_lens[seqs].astype(np.int32)


def compact_host_inputs(spec, seqs, q_dev, k_dev, v_dev):
    """Host copies (bf16 bit patterns) of what the oracle needs for `seqs`: their q rows and
    their KV blocks gathered into a small pool with remapped tables.  The device tensors were
    filled by the seeded generator; copying them back reproduces the generator's bits."""
    import torch

    ids, _, tables, lens = compact_tables(spec, seqs)
    idx = torch.from_numpy(ids).to(k_dev.device)
    to_bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    k = to_bits(k_dev[idx])
    v = to_bits(v_dev[idx])
    q = to_bits(q_dev[torch.tensor(seqs, device=q_dev.device)])
    return q, k, v, tables, lens


def sample_kv_bytes(spec, lens):
    return int(lens.astype(np.int64).sum()) * 2 * spec.num_kv_heads * spec.head_dim * 2


# --------------------------------------------------------------------------------------
# timing helpers
# --------------------------------------------------------------------------------------
def spread(values):
    """median / min / max of a list of per-repeat figures."""
    v = sorted(float(x) for x in values)
    return {"median": float(np.median(v)), "min": v[0], "max": v[-1], "n": len(v)}


def config_of(spec, world: int = 1, parallelism: str = ""):
    """The workload as both arms (this library and the oracle) describe it."""
    return {"workload": spec.name, "batch": spec.batch, "num_q_heads": spec.num_q_heads,
            "num_kv_heads": spec.num_kv_heads, "head_dim": spec.head_dim,
            "block_size": spec.block_size, "pool_blocks": spec.num_blocks,
            "total_context_tokens": spec.total_tokens,
            "kv_bytes_per_step": spec.kv_bytes(),
            "algorithmic_bytes_per_step": spec.algorithmic_bytes(),
            "l2": ("inputs (KV read per step) exceed the 126 MB L2; no flush"
                   if spec.kv_bytes() > 126e6 else
                   "the KV read per step fits the 126 MB L2: a launch-bound case, not a "
                   "bandwidth figure; no flush"),
            "parallelism": parallelism or ("independent replicas" if world > 1 else "1 gpu")}


# dram__bytes_read.sum + dram__bytes_write.sum of one pa_decode_kernel launch, from the ncu
# captures summarised under profiles/, keyed by (workload, context tokens, H, Hkv, D, partition
# size the plan chose).  Any other size, shape or partition size has no capture: null.
NCU_TRAFFIC = {
    ("cfg3_fullpool_mixed_gqa", 383921, 32, 8, 128, 512): 1597484800,
    ("cfg2_llama2_7b_mha", 66297, 32, 32, 128, 256): 1100038912,
}


def ncu_traffic(spec, partition_tokens: int):
    return NCU_TRAFFIC.get((spec.name, spec.total_tokens, spec.num_q_heads, spec.num_kv_heads,
                            spec.head_dim, int(partition_tokens)))


class DecodeLeg:
    """One workload resident on the device and the timed regions over it."""

    def __init__(self, torch, api, wl, spec, partition_tokens=0, dev="cuda"):
        self.torch, self.api, self.spec = torch, api, spec
        self.P = partition_tokens
        self.q = wl.q_torch(spec, dev)
        self.k, self.v = wl.pools_torch(spec, dev)
        self.tables = torch.from_numpy(spec.block_tables).to(dev)
        self.lens = torch.from_numpy(spec.seq_lens).to(dev)
        self.out = torch.empty_like(self.q)
        self.shape = api.shape_of(self.k, spec.num_q_heads)
        self.ws = torch.empty(api.pa_workspace_bytes(self.shape, spec.batch,
                                                     spec.total_tokens + 16 * spec.batch,
                                                     partition_tokens),
                              dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.step_bytes = spec.algorithmic_bytes()

    def step(self, flags=0, stream=None):
        self.api.pa_decode(self.q, self.k, self.v, self.tables, self.lens, self.spec.scale,
                           self.out, self.ws, dev_status=self.status, partition_tokens=self.P,
                           flags=flags, stream=stream)

    def region(self, steps, fn=None, dist=None):
        """Device time in ms of `steps` back-to-back steps (max over ranks)."""
        torch = self.torch
        fn = fn or self.step
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        ms, _ = aggregate_over_ranks(e0.elapsed_time(e1), 0.0, dist)
        return ms

    def kernels(self, steps):
        """Per-kernel ms per step from events the library records around each launch (an event
        between two launches removes their programmatic overlap, so this is a region of its own)."""
        api, torch = self.api, self.torch
        api.pa_profile_read()
        api.pa_profile_enable(True)
        for _ in range(steps):
            self.step()
        torch.cuda.synchronize()
        api.pa_profile_enable(False)
        plan_ms, attn_ms, comb_ms, calls = api.pa_profile_read()
        n = max(calls, 1)
        return {"plan": plan_ms / n, "attention": attn_ms / n, "combine": comb_ms / n}

    def plan_header(self):
        hdr = self.ws[:256].view(self.torch.int32).cpu().numpy()
        return {"partition_tokens": int(hdr[2]), "work_items": int(hdr[0])}

    def measure(self, steps, warmup, repeats, dist=None, world=1):
        """`repeats` timed regions of `steps` steps each, the per-kernel split, the step with
        the plan reused; throughputs are whole-job (all ranks)."""
        for _ in range(warmup):
            self.step()
        regions = [self.region(steps, dist=dist) for _ in range(repeats)]
        kern = self.kernels(steps)
        self.step()
        reuse = [self.region(steps, fn=lambda: self.step(flags=self.api.PA_FLAG_REUSE_PLAN))
                 for _ in range(min(repeats, 3))]
        assert int(self.status.item()) == 0, f"device status {int(self.status.item())}"
        gbps = lambda ms: world * self.step_bytes * steps / ms / 1e6
        peak, peak_src = measured_peaks()
        plan = self.plan_header()
        achieved = self.step_bytes / kern["attention"] / 1e6
        med = float(np.median(regions))
        return {
            "value": gbps(med), "ms_per_step": med / steps,
            "repeats": {"n": repeats, "steps_each": steps,
                        "value": spread([gbps(ms) for ms in regions]),
                        "ms_per_step": spread([ms / steps for ms in regions])},
            "frac_of_hbm_peak": gbps(med) / world / peak,
            "frac_of_nominal_8tbs": gbps(med) / world / 8000.0,
            "tokens_per_s": world * self.spec.batch * steps / (med / 1e3),
            "plan": plan,
            "kernels_ms_per_step": kern,
            "reuse_plan": {"ms_per_step": float(np.median(reuse)) / steps,
                           "value": self.step_bytes * steps / float(np.median(reuse)) / 1e6,
                           "frac_of_hbm_peak": self.step_bytes * steps / float(np.median(reuse)) / 1e6 / peak,
                           "note": "per layer of a multi-layer step: the first layer's plan is reused"},
            "roofline": {"bound": "hbm", "kernel": "pa_decode_kernel", "achieved": achieved,
                         "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(self.spec, plan["partition_tokens"]),
                         "peak_source": peak_src},
        }


# --------------------------------------------------------------------------------------
# swap timing (N = 1 only)
# --------------------------------------------------------------------------------------
def make_pools(torch, wl, layers, nb, hkv, d, layout, seed_k, seed_v, dev):
    """K and V pools as [layers, NB, Hkv, 16, D] views.  "layer": each layer's blocks together
    (one layer's attention stays inside NB x 32 KiB); "block": all layers of a block together
    (a block's whole payload is one contiguous piece, ideal for swapping, while one layer's
    attention then touches every page of the pool)."""
    n = nb * hkv * 16 * d
    if layout == "layer":
        return (wl.normal_bf16_torch(0, layers * n, seed_k, dev).view(layers, nb, hkv, 16, d),
                wl.normal_bf16_torch(0, layers * n, seed_v, dev).view(layers, nb, hkv, 16, d))
    store = wl.normal_bf16_torch(0, 2 * layers * n, seed_k, dev).view(nb, layers, 2, hkv, 16, d)
    return store[:, :, 0].permute(1, 0, 2, 3, 4), store[:, :, 1].permute(1, 0, 2, 3, 4)


class HostLink:
    """The host link's rate per direction: one contiguous pinned copy of `nbytes`, repeated;
    the best of all repeats taken before and after the legs it bounds is the denominator."""

    def __init__(self, torch, host, nbytes, stream):
        self.torch, self.host, self.nbytes, self.stream = torch, host, nbytes, stream
        self.dev_buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.d2h, self.h2d = [], []

    def _time(self, fn):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            fn()
            e1.record(self.stream)
        e1.synchronize()
        return self.nbytes / e0.elapsed_time(e1) / 1e6

    def sample(self, reps=10):
        h = self.host[:self.nbytes]
        for _ in range(reps):
            self.d2h.append(self._time(lambda: h.copy_(self.dev_buf, non_blocking=True)))
            self.h2d.append(self._time(lambda: self.dev_buf.copy_(h, non_blocking=True)))

    def summary(self):
        return {"bytes": self.nbytes, "d2h_gbps": max(self.d2h), "h2d_gbps": max(self.h2d),
                "samples_per_direction": len(self.d2h),
                "d2h_spread": spread(self.d2h), "h2d_spread": spread(self.h2d),
                "harmonic_mean_gbps": 2.0 / (1.0 / max(self.d2h) + 1.0 / max(self.h2d))}


def swap_cpu_baseline(torch, k_pool, v_pool, n_blocks, what):
    """The swap oracle (nested loops over the fixed host layout, one thread), as it stands, on a
    host mirror of the pools: gather `n_blocks` scattered blocks into an image, scatter the
    image into as many other blocks."""
    import oracle

    to_bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    k, v = to_bits(k_pool), to_bits(v_pool)
    nb = k.shape[1]
    perm = np.random.Generator(np.random.PCG64(0x5B)).permutation(nb)
    src, dst = perm[:n_blocks].astype(np.int32), perm[n_blocks:2 * n_blocks].astype(np.int32)
    nbytes = n_blocks * k.shape[0] * 2 * k.shape[2] * k.shape[3] * k.shape[4] * 2
    reps = max(1, int(2e8 // max(nbytes, 1)))          # small cases are repeated to be timeable
    t0 = time.perf_counter()
    for _ in range(reps):
        image = oracle.swap_out(k, v, src)
    t_out = (time.perf_counter() - t0) / reps
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.swap_in(k, v, image, dst)
    t_in = (time.perf_counter() - t0) / reps
    return {"out_gbps": nbytes / t_out / 1e9, "in_gbps": nbytes / t_in / 1e9, "unit": "GB/s",
            "cores": 1, "kind": "oracle", "bytes_each_way": nbytes, "passes": reps,
            "sample": what}


def bench_swap(args, torch, api, wl, decode_step, decode_bytes):
    dev = "cuda"
    layers, hkv, d, nb = 32, 8, 128, args.swap_pool_blocks
    k_pool, v_pool = make_pools(torch, wl, layers, nb, hkv, d, args.pool_layout, 0x51, 0x52, dev)
    bb = api.kv_block_bytes(k_pool, v_pool)
    tokens = [int(t) for t in args.swap_tokens.split(",")]
    max_blocks = max(tokens) // 16
    host = torch.empty(max_blocks * bb, dtype=torch.uint8, pin_memory=True)
    staging = torch.empty(args.swap_staging_mib << 20, dtype=torch.uint8, device=dev)
    side = torch.cuda.Stream()
    rng = np.random.Generator(np.random.PCG64(0x5A))

    def timed(fn, reps=5):
        out = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(side):
                e0.record(side)
                fn()
                e1.record(side)
            e1.synchronize()
            out.append(e0.elapsed_time(e1))
        return out

    # host-link ceiling: contiguous pinned copies (up to 2 GiB) per direction, sampled before
    # and after the swap legs; the best sample is the denominator of every fraction below
    link = HostLink(torch, host, min(max_blocks * bb, 2 << 30), side)
    link.sample(10)

    rows = []
    for n_tok in tokens:
        n = n_tok // 16
        perm = rng.permutation(nb)
        src, dst = perm[:n].astype(np.int32), perm[n:2 * n].astype(np.int32)
        nbytes = n * bb
        row = {"tokens": n_tok, "blocks": n, "bytes": nbytes}
        for mode, stg in (("staged", staging), ("direct", None)):
            t_out = timed(lambda: api.kv_swap_out(k_pool, v_pool, src, host, stg, stream=side))
            t_in = timed(lambda: api.kv_swap_in(k_pool, v_pool, host, dst, stg, stream=side))
            row[mode] = {"out_gbps": nbytes / float(np.median(t_out)) / 1e6,
                         "in_gbps": nbytes / float(np.median(t_in)) / 1e6,
                         "out_gbps_spread": spread([nbytes / t / 1e6 for t in t_out]),
                         "in_gbps_spread": spread([nbytes / t / 1e6 for t in t_in])}
        rows.append(row)

    # reference point: no kernel at all, one cudaMemcpyAsync per contiguous piece of the
    # smallest eviction (32 KiB per (block, layer, K|V) in the layer layout, a block's whole
    # 2 MiB in the block layout), issued from this Python loop
    n = tokens[0] // 16
    src = rng.permutation(nb)[:n]
    img = host[:n * bb].view(torch.bfloat16).view(n, layers, 2, hkv, 16, d)

    def naive_out():
        for i, b in enumerate(src.tolist()):
            if args.pool_layout == "block":   # K and V of all layers of block b are adjacent
                blk = hkv * 16 * d
                img[i].copy_(k_pool[:, b].as_strided((layers, 2, hkv, 16, d),
                                                     (2 * blk, blk, 16 * d, d, 1)),
                             non_blocking=True)
            else:
                for l in range(layers):
                    img[i, l, 0].copy_(k_pool[l, b], non_blocking=True)
                    img[i, l, 1].copy_(v_pool[l, b], non_blocking=True)

    t_naive = min(timed(naive_out, reps=2))
    naive = {"tokens": tokens[0], "bytes": n * bb,
             "copies": n * (1 if args.pool_layout == "block" else 2 * layers),
             "out_gbps": n * bb / t_naive / 1e6}

    # churn: evict + restore on the side stream while decode steps run on the main stream
    n = tokens[-1] // 16
    perm = rng.permutation(nb)
    src, dst = perm[:n].astype(np.int32), perm[n:2 * n].astype(np.int32)
    nbytes = n * bb

    def churn_once():
        api.kv_swap_out(k_pool, v_pool, src, host, staging, stream=side)
        api.kv_swap_in(k_pool, v_pool, host, dst, staging, stream=side)

    t_alone = timed(churn_once, reps=3)
    main = torch.cuda.current_stream()
    overlapped, dec_over, steps_total = [], [], 0
    for _ in range(3):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            e[0].record(side)
            churn_once()
            e[1].record(side)
        steps = 0
        e[2].record(main)
        t_host0 = time.perf_counter()
        while True:
            for _ in range(8):
                decode_step()
            steps += 8
            e[3].record(main)
            e[3].synchronize()
            if e[1].query() or time.perf_counter() - t_host0 > 5.0:
                break
        torch.cuda.synchronize()
        overlapped.append(2 * nbytes / e[0].elapsed_time(e[1]) / 1e6)
        dec_over.append(steps * decode_bytes / e[2].elapsed_time(e[3]) / 1e6)
        steps_total += steps
    link.sample(10)
    ls = link.summary()
    for row in rows:
        for mode in ("staged", "direct"):
            row[mode]["out_frac_of_link"] = row[mode]["out_gbps"] / ls["d2h_gbps"]
            row[mode]["in_frac_of_link"] = row[mode]["in_gbps"] / ls["h2d_gbps"]
    naive["out_frac_of_link"] = naive["out_gbps"] / ls["d2h_gbps"]
    alone = 2 * nbytes / float(np.median(t_alone)) / 1e6
    churn = {"tokens": tokens[-1], "swap_bytes_each_way": nbytes, "repeats": 3,
             "swap_alone_gbps": alone, "swap_alone_frac_of_link": alone / ls["harmonic_mean_gbps"],
             "swap_overlapped_gbps": float(np.median(overlapped)),
             "swap_overlapped_frac_of_link": float(np.median(overlapped)) / ls["harmonic_mean_gbps"],
             "decode_overlapped_gbps": float(np.median(dec_over)),
             "decode_steps_during_swap": steps_total}
    # the swap oracle on the host cores: workload 1's size exactly (a one-layer pool of 40
    # blocks of [8, 16, 64], 7 blocks moved) and a scaled-down mirror of workload 4 (32 layers,
    # 8 KV heads, head_dim 128 as there, but 256 blocks instead of 60000; 64 blocks = 1024
    # tokens moved each way)
    cpu = None
    if not args.no_cpu:
        k1 = wl.normal_bf16_torch(0, 40 * 8 * 16 * 64, 0x61, dev).view(1, 40, 8, 16, 64)
        v1 = wl.normal_bf16_torch(0, 40 * 8 * 16 * 64, 0x62, dev).view(1, 40, 8, 16, 64)
        cpu = {"workload1_size": swap_cpu_baseline(
                   torch, k1, v1, 7, "1 layer x 40 blocks x [8,16,64] (workload 1's pool), 7 blocks"),
               "workload4_mirror": swap_cpu_baseline(
                   torch, k_pool[:, :256], v_pool[:, :256], 64,
                   "32 layers x 256 blocks x [8,16,128] (workload 4's block shape, pool scaled "
                   "down from 60000 blocks), 64 blocks = 1024 tokens")}
    return {"pool": {"layers": layers, "kv_heads": hkv, "head_dim": d, "blocks": nb,
                     "block_bytes": bb, "staging_mib": args.swap_staging_mib,
                     "layout": args.pool_layout},
            "host_link": ls, "sizes": rows, "memcpy_per_piece": naive, "churn": churn,
            "cpu_baseline": cpu}


# --------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------
def init_ranks(torch, need_group=False):
    """(rank, world, local, dist or None).  One process per GPU; NCCL for plumbing only."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1 or need_group:
        import torch.distributed as dist

        # the communicator's own log lines (rank count, transport) go to stderr
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        if "MASTER_ADDR" in os.environ:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29655", rank=0,
                                    world_size=1, device_id=torch.device("cuda", local))
    return rank, world, local, dist


def e2e_leg(torch, api, leg, steps, repeats, dist):
    """The same step through pa_decode_host: q, lengths (and small block tables) copied from
    pinned host memory inside the timed region, the result posted to pinned host memory."""
    spec = leg.spec
    qh, th, lh = leg.q.cpu().pin_memory(), leg.tables.cpu().pin_memory(), leg.lens.cpu().pin_memory()
    oh = torch.empty_like(qh).pin_memory()
    io = torch.empty(api.pa_host_io_bytes(leg.shape, spec.batch, th.shape[1]), dtype=torch.uint8,
                     device="cuda")

    def step_e2e():
        api.pa_decode_host(qh, leg.k, leg.v, th, lh, spec.scale, oh, io, leg.ws,
                           dev_status=leg.status, partition_tokens=leg.P)

    for _ in range(3):
        step_e2e()
    regions = [leg.region(steps, fn=step_e2e, dist=dist) for _ in range(repeats)]
    leg.step()
    torch.cuda.synchronize()
    assert torch.equal(oh.view(torch.int16), leg.out.cpu().view(torch.int16))
    # lengths are copied; the query rows of a KV head's group (at most 8 heads per group, head_dim
    # 64 or 128; otherwise q is copied once) and the table entries are fetched in place over the
    # link, once per (work item, KV head); output rows are posted in place
    used_entries = int(((spec.seq_lens.astype(np.int64) + spec.block_size - 1) // spec.block_size).sum())
    table_bytes = th.numel() * 4
    group = spec.num_q_heads // spec.num_kv_heads
    units = leg.plan_header()["work_items"] * spec.num_kv_heads
    q_in_place = units * group * spec.head_dim * 2
    kv_us = spec.kv_bytes() / 6.4e6
    q_bytes = (q_in_place if group <= 8 and spec.head_dim <= 128 and q_in_place / 50e3 <= 0.65 * kv_us
               else qh.numel() * 2)   # the library's own rule for reading q in place
    h2d = q_bytes + lh.numel() * 4 + (used_entries * 4 * spec.num_kv_heads
                                      if table_bytes >= (256 << 10) else table_bytes)
    return regions, h2d, oh.numel() * 2


def graph_leg(torch, leg, steps):
    """The step captured once into a CUDA graph and replayed (reported beside `value`)."""
    stream = torch.cuda.current_stream()
    try:
        cap = torch.cuda.Stream()
        cap.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(cap):
            leg.step(stream=cap)                    # set-up calls happen outside the capture
            cap.synchronize()
            with torch.cuda.graph(g, stream=cap):
                leg.step(stream=cap)
            for _ in range(3):
                g.replay()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(cap)
            for _ in range(steps):
                g.replay()
            g1.record(cap)
            g1.synchronize()
            ms = g0.elapsed_time(g1) / steps
        stream.wait_stream(cap)
        return {"ms_per_step": ms, "value": leg.step_bytes / ms / 1e6, "error": None}
    except Exception as exc:  # a capture that the driver refuses is reported, not fatal
        torch.cuda.synchronize()
        return {"ms_per_step": None, "value": None, "error": str(exc)[:200]}


def workload1_leg(torch, api, wl, args):
    """Workload 1: the tiny decode, then sequence 2's blocks swapped out and back into other
    free blocks and the decode repeated (same bits).  Launch-bound: reported in microseconds."""
    spec = wl.config_spec(1)
    leg = DecodeLeg(torch, api, wl, spec, partition_tokens=64)
    res = leg.measure(max(args.steps, 20), 5, 5)
    first = leg.out.clone()
    src, dst = spec.blocks_of(2), spec.free_blocks[:7]
    kp, vp = leg.k.unsqueeze(0), leg.v.unsqueeze(0)
    host = torch.zeros(7 * api.kv_block_bytes(kp, vp), dtype=torch.uint8).pin_memory()
    stream = torch.cuda.current_stream()
    times = []
    for _ in range(20):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        api.kv_swap_out(kp, vp, src, host)
        api.kv_swap_in(kp, vp, host, dst)
        e1.record(stream)
        e1.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    t2 = spec.block_tables.copy()
    t2[2, :7] = dst
    leg.tables = torch.from_numpy(t2).cuda()
    leg.step()
    torch.cuda.synchronize()
    same = bool(torch.equal(first.view(torch.int16), leg.out.view(torch.int16)))
    assert same, "decode after the swap round trip differs"
    return {"config": config_of(spec), "value": res["value"], "ms_per_step": res["ms_per_step"],
            "repeats": res["repeats"], "us_per_decode_call": res["ms_per_step"] * 1e3,
            "kernels_ms_per_step": res["kernels_ms_per_step"], "plan": res["plan"],
            "bound": "launch latency (234 KB of KV per call)",
            "swap_round_trip": {"blocks": 7, "bytes_each_way": int(host.numel()),
                                "us_out_plus_in": spread(times),
                                "decode_bits_unchanged": same}}


def workloads_object(torch, api, wl, args, main_index):
    """Every other configuration in the same run: decode workloads 1, 2, 5 here, workload 4
    (full-size churn) by the caller once this process has released its other buffers."""
    out = {}
    for idx in (1, 2, 5):
        if idx == main_index:
            continue
        if idx == 1:
            out[wl.config_spec(1).name] = workload1_leg(torch, api, wl, args)
            continue
        spec = wl.config_spec(idx)
        leg = DecodeLeg(torch, api, wl, spec, args.partition_tokens)
        res = leg.measure(args.steps, max(args.warmup, 3), max(3, args.repeats - 2))
        res["config"] = config_of(spec)
        for key in ("tokens_per_s", "frac_of_nominal_8tbs"):
            res.pop(key, None)
        out[spec.name] = res
        del leg
        torch.cuda.empty_cache()
    if not args.decode_shape:
        # the head_dim 256 layer shape (16 query / 8 KV heads) on the headline workload's
        # lengths and pool occupancy: the third kind of layer the decode kernel is built for
        base = wl.config_spec(3)
        spec = wl.make_spec(f"{base.name}_h16_kv8_d256", seq_lens=base.seq_lens, num_q_heads=16,
                            num_kv_heads=8, head_dim=256, num_blocks=base.num_blocks,
                            seed=base.seed)
        leg = DecodeLeg(torch, api, wl, spec, args.partition_tokens)
        res = leg.measure(args.steps, max(args.warmup, 3), max(3, args.repeats - 2))
        res["config"] = config_of(spec)
        for key in ("tokens_per_s", "frac_of_nominal_8tbs"):
            res.pop(key, None)
        out[spec.name] = res
        del leg
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch

    from paper_2602_07878_b200 import api, build as lib_build
    from paper_2602_07878_b200 import workloads as wl

    rank, world, local, dist = init_ranks(torch)
    if rank == 0:
        lib_build.build()
    if dist is not None:
        dist.barrier()

    spec = wl.config_spec(args.workload)
    if args.decode_shape:
        # the workload's lengths and pool occupancy with another layer shape (H, Hkv, D)
        hq, hkv, hd = (int(x) for x in args.decode_shape.split(","))
        spec = wl.make_spec(f"{spec.name}_h{hq}_kv{hkv}_d{hd}", seq_lens=spec.seq_lens,
                            num_q_heads=hq, num_kv_heads=hkv, head_dim=hd,
                            num_blocks=spec.num_blocks, seed=spec.seed)
    leg = DecodeLeg(torch, api, wl, spec, args.partition_tokens)
    warmup = max(args.warmup, 3)
    n0 = api.pa_launch_count()
    leg.step()
    launches_per_step = api.pa_launch_count() - n0
    # every timed region of the headline (device-resident and end-to-end) runs under the sampler
    with ClockSampler(local, period_s=0.002) as clocks:
        res = leg.measure(args.steps, warmup, args.repeats, dist=dist, world=world)
        e2e_regions, h2d, d2h = e2e_leg(torch, api, leg, args.steps, args.repeats, dist)
    e2e_ms = float(np.median(e2e_regions))
    e2e_gbps = lambda ms: world * leg.step_bytes * args.steps / ms / 1e6

    line = {
        "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": res["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": config_of(spec, world),
        "repeats": res["repeats"],
        "tokens_per_s": res["tokens_per_s"],
        "frac_of_hbm_peak": res["frac_of_hbm_peak"],
        "frac_of_nominal_8tbs": res["frac_of_nominal_8tbs"],
        "e2e": {"value": e2e_gbps(e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps,
                "value_spread": spread([e2e_gbps(ms) for ms in e2e_regions])},
        "gpu_launches": int(launches_per_step * args.steps),
        "plan": res["plan"], "reuse_plan": res["reuse_plan"],
        "kernels_ms_per_step": res["kernels_ms_per_step"],
        "roofline": res["roofline"],
        "clocks": clocks.summary(),
    }

    if rank == 0 and world == 1:
        line["graph_replay"] = graph_leg(torch, leg, args.steps)
        peak = res["roofline"]["peak"]
        line["probes"] = bench_probes(torch, api, peak, res["value"], res["roofline"]["achieved"])
        line["kv_append"] = bench_append(torch, api, spec, leg.k, leg.v)
        if not args.no_recompute:
            rshape = tuple(int(x) for x in args.recompute_shape.split(",")) if args.recompute_shape else None
            line["recompute"] = bench_recompute(torch, api, spec, leg.k, leg.v, leg.tables,
                                                args.recompute_chunk, args.recompute_split,
                                                shape=rshape, cpu=not args.no_cpu,
                                                clock_ms=args.recompute_clock_ms)
        def resources(fn):
            """A leg that cannot get its memory (device pool, gigabytes of pinned host memory)
            is reported as skipped; a library error or a failed check still ends the run."""
            try:
                return fn()
            except api.PagedKVError:
                raise
            except RuntimeError as exc:   # torch: out of device memory, pinning failed
                torch.cuda.empty_cache()
                return {"skipped": f"{type(exc).__name__}: {str(exc)[:160]}"}

        if not args.no_swap:
            line["swap"] = resources(lambda: bench_swap(args, torch, api, wl, leg.step, leg.step_bytes))
        if not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline(args, spec, leg.q, leg.k, leg.v)
        if not args.no_workloads:
            line["workloads"] = resources(lambda: workloads_object(torch, api, wl, args, args.workload))
            # workload 4 at full size needs 126 GB of pool and 8 GiB of pinned host memory:
            # release everything else first, then run it if the device has the room
            del leg
            torch.cuda.empty_cache()
            free, _ = torch.cuda.mem_get_info()
            if "skipped" in line["workloads"]:
                pass
            elif free >= 150 * (1 << 30):
                line["workloads"]["cfg4_swap_churn"] = resources(lambda: churn_leg(args, torch, api, wl))
            else:
                line["workloads"]["cfg4_swap_churn"] = {
                    "skipped": f"{free / 2**30:.0f} GiB free on the device, 150 GiB wanted "
                               "(126 GB pool + staging + workspace)"}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def run_sharded(args):
    """`--seq-split` / `--kv-head-shard`: ONE workload's step shared by the N ranks (strong
    scaling: the job's KV bytes are fixed).

    Sequence split: every context is cut by blocks over the ranks; a step = partial attention
    over the rank's slice, an all-gather of the partial records over NCCL, the merge.
    KV-head shard (tensor-parallel ranks): rank r attends with KV heads [r Hkv/N, (r+1) Hkv/N)
    and their query heads; no exchange inside the path.
    Every rank generates the whole synthetic pool and reads only its part of it."""
    import torch

    from paper_2602_07878_b200 import api, build as lib_build, kvshard, seqsplit
    from paper_2602_07878_b200 import workloads as wl

    rank, world, local, dist = init_ranks(torch, need_group=True)
    if rank == 0:
        lib_build.build()
    dist.barrier()
    dev = "cuda"
    spec = wl.config_spec(args.workload)
    q = wl.q_torch(spec, dev)
    k, v = wl.pools_torch(spec, dev)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    P = args.partition_tokens
    if args.seq_split:
        t_np, l_np = seqsplit.shard_context(spec.block_tables, spec.seq_lens, rank, world,
                                            spec.block_size)
        tables, lens = torch.from_numpy(t_np).to(dev), torch.from_numpy(l_np).to(dev)
        shape = api.shape_of(k, spec.num_q_heads)
        local_tokens = int(l_np.sum())
        ws = torch.empty(api.pa_workspace_bytes(shape, spec.batch, local_tokens + 16 * spec.batch, P),
                         dtype=torch.uint8, device=dev)
        n = api.pa_partial_floats(shape, spec.batch)
        part = torch.empty(n, dtype=torch.float32, device=dev)
        gathered = torch.empty((world, n), dtype=torch.float32, device=dev)
        exchange_bytes = n * 4

        def step():
            seqsplit.decode(q, k, v, tables, lens, spec.scale, out, ws, part, gathered,
                            dev_status=status, partition_tokens=P)

        # bytes this rank's kernels must move per step: its slice of the KV, q, its table
        # entries, its record out, all records in, the output rows
        kv_local = local_tokens * 2 * spec.num_kv_heads * spec.head_dim * 2
        rank_bytes = (kv_local + q.numel() * 2 + int(((l_np + 15) // 16).sum()) * 4 + spec.batch * 4
                      + n * 4 * (1 + world) + out.numel() * 2)
        how = (f"sequence split over {world} rank(s): partial attention, all-gather of partial "
               "records (NCCL), merge")
    else:
        tables = torch.from_numpy(spec.block_tables).to(dev)
        lens = torch.from_numpy(spec.seq_lens).to(dev)
        ws = torch.empty(kvshard.workspace_bytes(world, k, spec.num_q_heads, spec.batch,
                                                 spec.total_tokens + 16 * spec.batch, P),
                         dtype=torch.uint8, device=dev)
        exchange_bytes = 0

        def step():
            kvshard.decode(rank, world, q, k, v, tables, lens, spec.scale, out, ws,
                           dev_status=status, partition_tokens=P)

        used = int(((spec.seq_lens.astype(np.int64) + 15) // 16).sum())
        rank_bytes = (spec.kv_bytes() + 2 * q.numel() * 2) // world + used * 4 + spec.batch * 4
        how = (f"KV heads sharded over {world} rank(s) (tensor parallel): each rank runs "
               "pa_decode_strided on its heads; no exchange inside the path")

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    dist.barrier()
    stream = torch.cuda.current_stream()
    n0 = api.pa_launch_count()
    regions, mine = [], []
    with ClockSampler(local, period_s=0.002) as clocks:
        for _ in range(args.repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            dist.barrier()
            e0.record(stream)
            for _ in range(args.steps):
                step()
            e1.record(stream)
            torch.cuda.synchronize()
            mine.append(e0.elapsed_time(e1))
            regions.append(aggregate_over_ranks(mine[-1], 0.0, dist)[0])
    launches = (api.pa_launch_count() - n0) // args.repeats
    total = torch.tensor([float(rank_bytes)], dtype=torch.float64, device=dev)
    dist.all_reduce(total)
    per_rank = torch.zeros(world, dtype=torch.float64, device=dev)
    per_rank[rank] = float(np.median(mine)) / args.steps
    dist.all_reduce(per_rank)
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    peak, peak_src = measured_peaks()
    med = float(np.median(regions))
    gbps = lambda ms: float(total.item()) * args.steps / ms / 1e6
    cfg = config_of(spec, world, how)
    cfg["exchange_bytes_per_rank_per_step"] = exchange_bytes
    line = {
        "metric": METRIC, "value": gbps(med), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": med / args.steps, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": cfg,
        "repeats": {"n": args.repeats, "steps_each": args.steps,
                    "value": spread([gbps(ms) for ms in regions])},
        "ms_per_step_per_rank": [float(x) for x in per_rank.tolist()],
        "tokens_per_s": spec.batch * args.steps / (med / 1e3),
        "frac_of_hbm_peak": gbps(med) / world / peak, "peak_source": peak_src,
        "gpu_launches": int(launches), "clocks": clocks.summary(),
    }
    dist.barrier()
    dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def bench_probes(torch, api, copy_peak, step_gbps, kernel_gbps, gib=2, reps=5):
    """Practical read ceilings measured in the same run: a read-only stream and 4 KiB gathers
    (one bulk copy per granule, as the attention kernel fetches its tiles) over a 2 GiB buffer."""
    buf = torch.empty(gib << 30, dtype=torch.uint8, device="cuda")
    buf.zero_()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = {"bytes": buf.numel(), "copy_peak_gbps": copy_peak, "nominal_gbps": 8000.0}
    for name, scattered in (("read_stream_gbps", False), ("read_gather_4k_gbps", True)):
        best = 0.0
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            api.pa_probe_read(buf, scattered, status)
            e1.record()
            e1.synchronize()
            best = max(best, buf.numel() / e0.elapsed_time(e1) / 1e6)
        out[name] = best
    # how fast 2 KB tiled TMA boxes (the K/V box of the attention kernels) can be issued and
    # delivered out of L2: a 64 MiB buffer walked 32 times, 16 boxes per SM and ring slot,
    # issued by 1, 2, 4 or 8 warps
    small = buf[:64 << 20]
    clock_hz = 1.965e9
    rows = []
    for warps, boxes in ((1, 16), (2, 8), (4, 4), (8, 2)):
        api.pa_probe_tma_issue(small, warps, boxes, 2, status)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        n = api.pa_probe_tma_issue(small, warps, boxes, 32, status)
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        rows.append({"warps": warps, "boxes_per_instruction": boxes, "gbps": n * 2048 / ms / 1e6,
                     "ns_per_box_per_sm": ms * 1e6 / (n / 148.0),
                     "bytes_per_clock_per_sm_at_1965mhz": n * 2048 / 148.0 / (ms * 1e-3 * clock_hz)})
    out["tma_issue_l2_resident"] = rows
    assert int(status.item()) == 0
    out["attention_kernel_frac_of_gather"] = kernel_gbps / out["read_gather_4k_gbps"]
    out["step_frac_of_gather"] = step_gbps / out["read_gather_4k_gbps"]
    return out


def bench_append(torch, api, spec, k, v, calls=200):
    """kv_append of one token per sequence into its last slot (the rows written are the ones
    already there, so the pool keeps its content).  Launch-latency bound: reported in us
    between back-to-back calls issued from Python."""
    lens = spec.seq_lens.astype(np.int64)
    rows = np.nonzero(lens > 0)[0]
    pos = lens[rows] - 1
    blk = spec.block_tables[rows, pos // spec.block_size].astype(np.int64)
    slots_np = np.full(spec.batch, -1, np.int64)
    slots_np[rows] = blk * spec.block_size + pos % spec.block_size
    slots = torch.from_numpy(slots_np).cuda()
    safe = slots.clamp(min=0)
    k_new = k[safe // 16, :, safe % 16, :].contiguous()
    v_new = v[safe // 16, :, safe % 16, :].contiguous()
    for _ in range(5):
        api.kv_append(k, v, k_new, v_new, slots)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(calls):
        api.kv_append(k, v, k_new, v_new, slots)
    e1.record()
    e1.synchronize()
    nbytes = 2 * 2 * k_new.numel() * 2          # K and V rows, read + written
    us = e0.elapsed_time(e1) * 1e3 / calls
    return {"us_per_call": us, "tokens": int(len(rows)), "bytes": nbytes,
            "gbps": nbytes / us / 1e3, "bound": "launch latency / host issue rate (2 MB moved per call)"}


def bench_recompute(torch, api, spec, k, v, tables, chunk=512, split=0, max_splits=16, shape=None,
                    cpu=False, clock_ms=500.0):
    """Recomputation recovery of the longest sequence of the batch: causal prefill attention
    over its cached tokens in chunks of `chunk` query tokens (one pa_prefill_split call per
    chunk, context growing, the block table passed no wider than the context).  A dense
    contraction: reported in TFLOP/s against the bf16 tensor peak."""
    b = int(np.argmax(spec.seq_lens))
    L = int(spec.seq_lens[b])
    H, D = spec.num_q_heads, spec.head_dim
    if shape is not None:
        # another layer shape (query heads, KV heads, head_dim): the same sequence length over a
        # pool of its own with a shuffled block table
        H, hkv, D = shape
        nb = (L + 15) // 16
        k = torch.empty(nb + 64, hkv, 16, D, dtype=torch.bfloat16, device="cuda").normal_()
        v = torch.empty_like(k).normal_()
        g = torch.Generator().manual_seed(0x2602)
        tables = torch.randperm(nb + 64, generator=g)[:nb].to(torch.int32).view(1, nb).cuda()
        b = 0
    q = torch.empty(L, H, D, dtype=torch.bfloat16, device="cuda").normal_()
    out = torch.empty_like(q)
    tab = tables[b:b + 1].contiguous()
    ws = torch.empty(api.pa_prefill_split_workspace_bytes(api.shape_of(k, H), 1, min(chunk, L),
                                                          max_splits),
                     dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    calls = []
    for start in range(0, L, chunk):
        end = min(L, start + chunk)
        calls.append((start, end, torch.tensor([end], dtype=torch.int32, device="cuda"),
                      torch.tensor([0, end - start], dtype=torch.int32, device="cuda"),
                      tab[:, :(end + 15) // 16].contiguous()))
    shapes = []

    def run():
        shapes.clear()
        for start, end, ctx, cu, t in calls:
            api.pa_prefill_split(q[start:end], k, v, t, ctx, cu, spec.scale, out[start:end], ws,
                                 kv_split_tokens=split, dev_status=status)
            shapes.append(api.pa_prefill_last_launch())

    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run()
    e1.record()
    e1.synchronize()
    ms = e0.elapsed_time(e1)
    # clocks under this load: the leg repeated for about half a second while NVML is sampled
    with ClockSampler(torch.cuda.current_device()) as cs:
        for _ in range(int(clock_ms / max(ms, 1e-3))):
            run()
        torch.cuda.synchronize()
    # 4 * D flops per (query, visible key, head): QK^T and PV, 2 flops per multiply-add
    pairs = sum((end - start) * (start + end + 1) // 2 for start, end, _, _, _ in calls)
    flops = 4.0 * D * H * pairs
    peak = sustained = None
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            peaks = json.load(f)
            peak = float(peaks["bf16_tflops"])
            sustained = float(peaks.get("bf16_tflops_sustained", 0.0)) or None
    assert int(status.item()) == 0
    cpu_part = None
    if cpu:
        # the prefill oracle, as it stands, on the last 16 query tokens of the sequence (the
        # sequence's blocks copied to the host in table order), timed and compared with the
        # rows the last call wrote
        import oracle

        n_s = min(16, L)
        nb_seq = (L + 15) // 16
        ids = tab[0, :nb_seq].long()
        to_bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        kh, vh, qh = to_bits(k[ids]), to_bits(v[ids]), to_bits(q[L - n_s:])
        t0 = time.perf_counter()
        ref = oracle.pa_prefill(qh, kh, vh, np.arange(nb_seq, dtype=np.int32)[None], [L], [0, n_s],
                                spec.scale)
        dt = time.perf_counter() - t0
        got = out[L - n_s:].float().cpu().numpy().astype(np.float64)
        err = np.abs(got - ref).max(axis=-1) / np.abs(ref).max(axis=-1)
        cpu_part = {"value": 4.0 * D * H * n_s * (2 * L - n_s + 1) / 2 / dt / 1e12, "unit": "TFLOP/s",
                    "cores": oracle.threads(), "kind": "oracle", "seconds": dt,
                    "sample": f"the last {n_s} of {L} query tokens, one pass",
                    "max_row_rel_err_of_gpu_rows": float(err.max())}
    return {"tokens": L, "chunk": chunk, "calls": len(calls), "ms": ms, "tflops": flops / ms / 1e9,
            "cpu_baseline": cpu_part,
            "shape": {"num_q_heads": H, "num_kv_heads": int(k.shape[1]), "head_dim": D},
            "clocks": cs.summary(),
            "last_call_launch": {"tiles_per_cta": shapes[-1][0], "kv_split_tokens": shapes[-1][1],
                                 "kv_splits": shapes[-1][2]},
            "bound": "tensor", "peak_tflops": peak,
            "frac": (flops / ms / 1e9 / peak) if peak else None,
            # context: the library GEMM's rate over seconds under the power cap (the leg above is
            # a burst of a few milliseconds; "clocks" were sampled over half a second of repeats)
            "peak_tflops_sustained": sustained,
            "tokens_per_s": L / (ms / 1e3)}


def cpu_baseline(args, spec, q, k, v):
    """The fp64 oracle, as it stands, on the host cores, over a bounded sample of the batch."""
    import oracle

    budget = int(spec.total_tokens * args.cpu_fraction)
    seqs, tot = sample_sequences(spec, budget)
    qh, kh, vh, tables, lens = compact_host_inputs(spec, seqs, q, k, v)
    t0 = time.perf_counter()
    oracle.pa_decode(qh, kh, vh, tables, lens, spec.scale)
    dt = time.perf_counter() - t0
    return {"value": sample_kv_bytes(spec, lens) / dt / 1e9, "unit": UNIT,
            "cores": oracle.threads(), "kind": "oracle", "seconds": dt,
            "sample": f"{len(seqs)} of {spec.batch} sequences of {spec.name} "
                      f"({tot} of {spec.total_tokens} context tokens), one pass"}



# --------------------------------------------------------------------------------------
# reference arm: the oracle on the host cores
# --------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    from paper_2602_07878_b200 import workloads as wl

    spec = wl.config_spec(args.workload)
    # size the per-step sample so that warmup + steps end within a couple of minutes:
    # the oracle streams roughly 0.2 GB/s of KV per core
    est_gbps = 0.2 * oracle.threads()
    budget_bytes = 120.0 / max(1, args.steps + args.warmup) * est_gbps * 1e9
    tok_bytes = 2 * spec.num_kv_heads * spec.head_dim * 2
    budget_tok = int(min(spec.total_tokens, max(256, budget_bytes / tok_bytes)))
    seqs, tot = sample_sequences(spec, budget_tok)
    try:
        import torch

        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        # generator output produced on the device and copied back (same bits as on the host)
        q = wl.q_torch(spec, "cuda")
        k, v = wl.pools_torch(spec, "cuda")
        qh, kh, vh, tables, lens = compact_host_inputs(spec, seqs, q, k, v)
        del q, k, v
    else:
        ids, remap, tables, lens = compact_tables(spec, seqs)
        kh, vh = wl.pool_block_np(spec, "k", ids), wl.pool_block_np(spec, "v", ids)
        for blk, slot in wl.tail_slots(spec):
            if blk in remap:
                kh[remap[blk], :, slot:] = wl.BF16_NAN_BITS
                vh[remap[blk], :, slot:] = wl.BF16_NAN_BITS
        qh = wl.q_np(spec)[seqs]
    nbytes = sample_kv_bytes(spec, lens)
    for _ in range(args.warmup):
        oracle.pa_decode(qh, kh, vh, tables, lens, spec.scale)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.pa_decode(qh, kh, vh, tables, lens, spec.scale)
    dt = time.perf_counter() - t0
    value = nbytes * args.steps / dt / 1e9
    sample = (f"{len(seqs)} of {spec.batch} sequences of {spec.name} ({tot} of "
              f"{spec.total_tokens} context tokens) per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(spec, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------------------
# workload 4: preemption swap churn at full size (1 GPU)
# --------------------------------------------------------------------------------------
def churn_leg(args, torch, api, wl):
    """32-layer pool of 60000 blocks at 98 % occupancy.  For each eviction size N the victims'
    blocks go to pinned host memory and come back into other blocks on a side stream while
    the remaining batch is decoded, layer by layer, on the main stream.  One decode step =
    32 pa_decode calls (one per layer; the plan is made once and reused)."""
    dev = "cuda"
    spec = wl.config_spec(4)
    layers, nb = spec.num_layers, spec.num_blocks
    n = nb * spec.block_elems
    k_pool, v_pool = make_pools(torch, wl, layers, nb, spec.num_kv_heads, spec.head_dim,
                                args.pool_layout, spec.seed_k, spec.seed_v, dev)
    q = wl.q_torch(spec, dev)
    tables = torch.from_numpy(spec.block_tables).to(dev)
    out = torch.empty_like(q)
    shape = api.shape_of(k_pool[0], spec.num_q_heads)
    ws = torch.empty(api.pa_workspace_bytes(shape, spec.batch, spec.total_tokens + 16 * spec.batch),
                     dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    bb = api.kv_block_bytes(k_pool, v_pool)
    tokens = [1024, 4096, 16384, 65536]
    host = torch.empty(tokens[-1] // 16 * bb, dtype=torch.uint8, pin_memory=True)
    staging = torch.empty(args.swap_staging_mib << 20, dtype=torch.uint8, device=dev)
    side, main = torch.cuda.Stream(), torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    link = HostLink(torch, host, 2 << 30, main)
    link.sample(5)

    rows = []
    with ClockSampler(torch.cuda.current_device()) as clocks:
        for n_tok in tokens:
            seqs, src, dst = wl.pick_victims(spec, n_tok, seed=100 + n_tok)
            lens_np = spec.seq_lens.copy()
            lens_np[seqs] = 0                       # the victims are not in the running batch
            lens = torch.from_numpy(lens_np).to(dev)
            step_bytes = layers * dataclass_replace(spec, lens_np).algorithmic_bytes()

            def decode_step():
                for layer in range(layers):
                    api.pa_decode(q, k_pool[layer], v_pool[layer], tables, lens, spec.scale, out,
                                  ws, flags=api.PA_FLAG_REUSE_PLAN if layer else 0,
                                  dev_status=status)

            def swap_round():
                api.kv_swap_out(k_pool, v_pool, src, host, staging, stream=side)
                api.kv_swap_in(k_pool, v_pool, host, dst, staging, stream=side)
                # and back, so that every round starts from the same pool
                api.kv_swap_out(k_pool, v_pool, dst, host, staging, stream=side)
                api.kv_swap_in(k_pool, v_pool, host, src, staging, stream=side)

            nbytes = len(src) * bb
            for _ in range(2):
                decode_step()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record(main)
            for _ in range(args.churn_steps):
                decode_step()
            b.record(main); b.synchronize()
            dec_alone = args.churn_steps * step_bytes / a.elapsed_time(b) / 1e6
            alone = []
            for _ in range(2 if n_tok >= 65536 else 3):
                a, b = ev(), ev()
                with torch.cuda.stream(side):
                    a.record(side); swap_round(); b.record(side)
                b.synchronize()
                alone.append(4 * nbytes / a.elapsed_time(b) / 1e6)
            # overlapped
            e = [ev() for _ in range(4)]
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                e[0].record(side); swap_round(); e[1].record(side)
            steps = 0
            e[2].record(main)
            t0 = time.perf_counter()
            while True:
                decode_step()
                steps += 1
                e[3].record(main); e[3].synchronize()
                if e[1].query() or time.perf_counter() - t0 > 20.0:
                    break
            torch.cuda.synchronize()
            rows.append({"tokens": n_tok, "blocks": int(len(src)), "bytes_each_way": nbytes,
                         "victim_sequences": len(seqs),
                         "swap_alone_gbps": float(np.median(alone)),
                         "swap_alone_gbps_spread": spread(alone),
                         "swap_overlapped_gbps": 4 * nbytes / e[0].elapsed_time(e[1]) / 1e6,
                         "decode_alone_gbps": dec_alone,
                         "decode_overlapped_gbps": steps * step_bytes / e[2].elapsed_time(e[3]) / 1e6,
                         "decode_steps_during_swap": steps,
                         "decode_step_bytes": step_bytes})
    assert int(status.item()) == 0
    link.sample(5)
    ls = link.summary()
    for r in rows:
        r["swap_alone_frac_of_link"] = r["swap_alone_gbps"] / ls["harmonic_mean_gbps"]
        r["swap_overlapped_frac_of_link"] = r["swap_overlapped_gbps"] / ls["harmonic_mean_gbps"]
    peak, peak_src = measured_peaks()
    best = max(r["decode_alone_gbps"] for r in rows)
    return {"value": best, "unit": UNIT, "steps": args.churn_steps,
            "config": {"workload": spec.name, "batch": spec.batch, "layers": layers,
                       "pool_blocks": nb, "allocated_blocks": nb - len(spec.free_blocks),
                       "pool_bytes": 2 * layers * n * 2, "block_bytes": bb,
                       "pool_layout": args.pool_layout,
                       "total_context_tokens": spec.total_tokens,
                       "step": "32 pa_decode calls (one per layer, plan reused) over the non-evicted batch",
                       "staging_mib": args.swap_staging_mib},
            "frac_of_hbm_peak": best / peak, "peak_source": peak_src,
            "host_link": ls, "churn": rows, "clocks": clocks.summary()}


def run_churn(args):
    import torch

    from paper_2602_07878_b200 import api, build as lib_build
    from paper_2602_07878_b200 import workloads as wl

    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("workload 4 holds 126 GB per GPU and is run on one GPU")
    lib_build.build()
    torch.cuda.set_device(0)
    res = churn_leg(args, torch, api, wl)
    print(json.dumps(dict({"metric": METRIC, "n_gpus": 1, "warmup": 2, "higher_is_better": True,
                           "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                           "data": "synthetic"}, **res)))


def dataclass_replace(spec, seq_lens):
    import dataclasses

    return dataclasses.replace(spec, seq_lens=seq_lens)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--repeats", type=int, default=7,
                    help="how many times the timed region of --steps steps is repeated "
                         "(value = the median region; min and max are reported beside it)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3, 4, 5],
                    help="decode workload of the headline (3 = full-pool mixed-length GQA; "
                         "4 = only the full-size swap churn, 126 GB pool, 1 GPU)")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the `workloads` object (the other configurations, full-size churn)")
    ap.add_argument("--churn-steps", type=int, default=3)
    ap.add_argument("--partition-tokens", type=int, default=0,
                    help="force the decode partition size (0 = chosen per call on the device)")
    ap.add_argument("--seq-split", action="store_true",
                    help="split every context over the ranks (one all-gather per step) "
                         "instead of running independent replicas")
    ap.add_argument("--kv-head-shard", action="store_true",
                    help="shard the KV heads over the ranks (tensor parallel, no exchange) "
                         "instead of running independent replicas")
    ap.add_argument("--no-swap", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-recompute", action="store_true")
    ap.add_argument("--recompute-chunk", type=int, default=512,
                    help="query tokens per pa_prefill call of the recompute leg")
    ap.add_argument("--decode-shape", default="",
                    help="H,Hkv,D of the decode legs when they should differ from the workload's "
                         "(e.g. 16,8,256); lengths and occupancy stay the workload's")
    ap.add_argument("--recompute-shape", default="",
                    help="H,Hkv,D of the recompute leg when it should differ from the workload's "
                         "(e.g. 16,8,256)")
    ap.add_argument("--recompute-clock-ms", type=float, default=500.0,
                    help="how long the recompute leg is repeated while the clocks are sampled "
                         "(0 = not at all, e.g. under a profiler)")
    ap.add_argument("--recompute-split", type=int, default=0,
                    help="kv_split_tokens of the recompute leg (0 = library's choice, -1 = never)")
    ap.add_argument("--cpu-fraction", type=float, default=1.0,
                    help="fraction of the batch's tokens the CPU baseline pass covers")
    ap.add_argument("--swap-pool-blocks", type=int, default=6144)
    ap.add_argument("--pool-layout", default="layer", choices=["layer", "block"],
                    help="multi-layer pools of the swap legs and of workload 4: each layer's blocks "
                         "together, or all layers of a block together")
    ap.add_argument("--swap-tokens", default="1024,4096,16384")
    ap.add_argument("--swap-staging-mib", type=int, default=256)
    args = ap.parse_args()
    if args.impl == "reference":
        if args.workload == 4:
            args.workload = 3      # the oracle arm times decode attention; 4 shares 3's mix
        run_reference(args)
    elif args.workload == 4:
        run_churn(args)
    elif args.seq_split or args.kv_head_shard:
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
