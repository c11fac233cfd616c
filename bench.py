#!/usr/bin/env python
"""Benchmark of the PPSA decode-step attention path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload cfg3] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic input: the
attention of all layers of one decode step (2 full layers, 2 token-selection
layers with top-k, 28 sparse layers for the 32-layer workloads). The default
workload is the Llama-3-8B-shaped 128K-context configuration the metric is
quoted on. The path does not shard (one GPU per the method); with N > 1 every
rank runs an independent replica and the line reports the aggregate.

The CPU oracle appears only in the `cpu_baseline` leg and in `--impl reference`.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2410_05076_b200 import synth  # noqa: E402

METRIC = "us_per_decode_step_attention_all_layers"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) of one full-attention launch at the cfg3 shape, from the ncu
# capture summarised in profiles/attn_topk_kernels_cfg3_ncu_full.md (dram__bytes_read.sum + dram__bytes_write.sum).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"cfg3": 536.94e6 + 3.86e6}


def describe(w: synth.Workload) -> str:
    lay = "paged(16)" if w.paged else "contiguous [B][Hkv][N][K|V][d]"
    return (f"{w.name}: B{w.batch} {w.num_q_heads}q/{w.num_kv_heads}kv d{w.head_dim} L{w.num_layers} "
            f"ctx{w.ctx}{'(ragged)' if w.ragged else ''} k{w.k} bf16 {lay}, "
            f"{w.sched.count(0)} full + {w.sched.count(1)} select + {w.sched.count(2)} sparse layers")


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def build_workload(w: synth.Workload, device):
    qs = [synth.make_q(w, i, device) for i in range(w.num_layers)]
    if w.paged:
        pt, total = synth.make_page_table(w)
        layers = [synth.make_layer(w, i, device, layout="paged", q=qs[i], page_table=pt, num_pages=total)
                  for i in range(w.num_layers)]
    else:
        layers = [synth.make_layer(w, i, device, q=qs[i]) for i in range(w.num_layers)]
    return qs, layers


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
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
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's figure: every multi-GPU time is the max over ranks (replicas finish together)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_step(ms_per_step: float, world: int) -> float:
    """N replicas complete N decode steps in the time of the slowest one."""
    return ms_per_step * 1e3 / world


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def oracle_sample(w: synth.Workload, qs, layers, host_cache=None, index_heads=None):
    """Time the CPU oracle, as it stands, on one layer of each type and scale by the layer mix.
    Only the oracle calls are timed; the host copies of the sampled layers may be cached by the caller."""
    import oracle
    from oracle import adapter

    first = {t: w.sched.index(t) for t in (0, 1, 2) if t in w.sched}
    times, rho = {}, None
    order = sorted(first.items(), key=lambda kv: (kv[0] == 2, kv[1]))    # selection before sparse
    for t, i in order:
        if host_cache is not None and i in host_cache:
            okv, qb = host_cache[i]
        else:
            okv, qb = adapter.kv_from_layer(layers[i]), adapter.bits(qs[i])
            if host_cache is not None:
                host_cache[i] = (okv, qb)
        t0 = time.perf_counter()
        if t == 0:
            oracle.full_attn(okv, qb)
        elif t == 1:
            _, idx, cnt = oracle.select_attn(okv, qb, w.k, index_heads)
            rho = (idx, cnt)
        else:
            if rho is None:
                _, idx, cnt = oracle.select_attn(okv, qb, w.k, index_heads)
                rho = (idx, cnt)
                t0 = time.perf_counter()
            oracle.sparse_attn(okv, qb, rho[0], rho[1])
        times[t] = time.perf_counter() - t0
        del okv
    total = sum(times[t] * w.sched.count(t) for t in times)
    sample = ("one layer of each type timed once (layers " + ",".join(str(first[t]) for t in sorted(first)) +
              f"), scaled by the {w.sched.count(0)}+{w.sched.count(1)}+{w.sched.count(2)} layer mix")
    return total * 1e6, oracle.num_threads(), sample, {int(t): times[t] * 1e6 for t in times}


def run_reference(args, w, rank):
    """The reference arm of this tier is the CPU oracle on the host cores."""
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    # Only the three sampled layers are materialised.
    need = sorted({w.sched.index(t) for t in (0, 1, 2) if t in w.sched})
    qs = {i: synth.make_q(w, i, dev) for i in need}
    layers = {i: synth.make_layer(w, i, dev, q=qs[i]) for i in need} if not w.paged else None
    if w.paged:
        pt, total = synth.make_page_table(w)
        layers = {i: synth.make_layer(w, i, dev, layout="paged", q=qs[i], page_table=pt, num_pages=total)
                  for i in need}
    vals, cache = [], {}
    for it in range(args.warmup + args.steps):
        us, cores, sample, _ = oracle_sample(w, qs, layers, cache, index_heads={'qhead': w.num_q_heads, 'kvhead': w.num_kv_heads, 'shared': 1}[args.granularity])
        if it >= args.warmup:
            vals.append(us)
    v = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "us", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": v / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(w)},
            "cpu_baseline": {"value": v, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def profile_case(td, w, dev, steps):
    """One layer of each type (about 1.5 GiB at cfg3), run in the order full, select, sparse."""
    need = [w.sched.index(t) if t in w.sched else 0 for t in (0, 1, 2)]
    qs = {i: synth.make_q(w, i, dev) for i in set(need)}
    if w.paged:
        pt, total = synth.make_page_table(w)
        layers = {i: synth.make_layer(w, i, dev, layout="paged", q=qs[i], page_table=pt, num_pages=total)
                  for i in set(need)}
    else:
        layers = {i: synth.make_layer(w, i, dev, q=qs[i]) for i in set(need)}
    torch.cuda.synchronize()
    idx = cnt = None
    for _ in range(steps):
        td.full_attn(layers[need[0]], qs[need[0]])
        _, idx, cnt = td.select_attn(layers[need[1]], qs[need[1]], w.k)
        td.sparse_attn(layers[need[2]], qs[need[2]], idx, cnt)
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": w.name, "steps": steps, "launches": td.launch_count()}))


def sweep(td, dev, reps):
    """Configuration 5: context 4K..256K x budget 512..8192. Every point rotates over enough distinct
    copies of the two layers that each launch finds its KV cache cold in L2."""
    points = []
    for ctx in synth.SWEEP_CTX:
        w0 = synth.sweep_point(ctx, 512)
        layer_bytes = ctx * w0.num_kv_heads * 512
        copies = max(2, min(24, -(-400 * 2 ** 20 // layer_bytes)))
        qs = [synth.make_q(w0, 0, dev), synth.make_q(w0, 1, dev)]
        # sparse layers gather as little as 8 MiB each: 20 distinct caches keep a chain of them cold
        sp_copies = max(copies, 20)
        sel_layers, sp_layers = [], []
        for c in range(sp_copies):
            wc = synth.sweep_point(ctx, 512)
            wc.seed += 1000 * c
            if c < copies:
                sel_layers.append(synth.make_layer(wc, 0, dev, q=qs[0]))
            sp_layers.append(synth.make_layer(wc, 1, dev, q=qs[1]))
        outs = [torch.empty(1, w0.num_q_heads, w0.head_dim, dtype=torch.float32, device=dev)
                for _ in range(max(copies, sp_copies) + 1)]

        def timed(kinds, lays, qq, k):
            st = td.make_step(kinds, lays, qq, outs[:len(kinds)], k)
            for _ in range(2):
                st()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                st()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) * 1e3 / reps

        for k in synth.SWEEP_K:
            kk = min(k, ctx)
            # all launches go through tidal_decode_step (no host gaps): a chain of selection layers over
            # the distinct copies, and one selection layer followed by a chain of sparse layers
            t_sel_chain = timed([synth.LAYER_SELECT] * copies, sel_layers, [qs[0]] * copies, kk)
            t_one = timed([synth.LAYER_SELECT], sel_layers[:1], qs[:1], kk)
            t_sp_chain = timed([synth.LAYER_SELECT] + [synth.LAYER_SPARSE] * sp_copies,
                               sel_layers[:1] + sp_layers, [qs[0]] + [qs[1]] * sp_copies, kk)
            sel_us, sp_us = t_sel_chain / copies, (t_sp_chain - t_one) / sp_copies
            points.append({"ctx": ctx, "k": k, "select_us_incl_topk": sel_us, "sparse_us": sp_us,
                           "select_GBs": layer_bytes / sel_us / 1e3,
                           "sparse_GBs": w0.num_q_heads * kk * 516 / sp_us / 1e3,
                           "select_over_sparse": sel_us / sp_us, "copies": [copies, sp_copies]})
        del sel_layers, sp_layers
        torch.cuda.empty_cache()
    assert td.device_status() == 0
    print(json.dumps({"sweep": "cfg5: B1 32q/8kv d128; per-layer cost of a selection layer (attention + top-k) and "
                      "of a sparse layer, from chains of layers run through tidal_decode_step over distinct "
                      "KV copies (cold in L2), CUDA events", "reps": reps, "points": points}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="tidal", choices=["tidal", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--granularity", default="qhead", choices=["qhead", "kvhead", "shared"],
                    help="one token set per query head (default), per KV head, or shared by all heads "
                         "(the latter two rank by the sum of the member heads' scaled logits)")
    ap.add_argument("--sweep", action="store_true",
                    help="context x budget sweep (Llama-3-8B head shapes, one selection + one sparse layer): "
                         "prints one JSON line with the selection-layer and sparse-layer cost of every point")
    ap.add_argument("--profile-case", action="store_true",
                    help="small capture target for ncu: one full, one selection and one sparse layer of "
                         "the workload, each run --steps times, nothing else")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "tidal" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = synth.workload(args.workload)

    if args.impl == "reference":
        run_reference(args, w, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU implementation")
    from paper_2410_05076_b200 import binding

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    # An ordinary (non-default) stream: the library then records each step's launches once as a CUDA
    # graph and replays it, and every event below is recorded on this same stream.
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    td = binding.Tidal(local)
    if args.profile_case:
        profile_case(td, w, dev, args.steps)
        return
    if args.sweep:
        sweep(td, dev, max(3, min(args.steps, 30)))
        return
    qs, layers = build_workload(w, dev)
    outs = [torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.float32, device=dev) for _ in layers]
    gran = {"qhead": binding.SEL_PER_QHEAD, "kvhead": binding.SEL_PER_KVHEAD, "shared": binding.SEL_SHARED}[args.granularity]
    index_heads = {"qhead": w.num_q_heads, "kvhead": w.num_kv_heads, "shared": 1}[args.granularity]
    # rows a sparse layer gathers: one list per index head, read once per KV head it serves
    gather_lists = w.num_q_heads if args.granularity == "qhead" else w.num_kv_heads
    step = td.make_step(w.sched, layers, qs, outs, w.k, gran)
    kv_bytes = [l.kv_bytes() for l in layers]

    # ---- device-resident timing: the headline value -------------------------------------------
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    launches0 = td.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop()
    launches = td.launch_count() - launches0
    ms_total = e0.elapsed_time(e1)
    ms_step = max_over_ranks(ms_total, dist, dev) / args.steps
    status = td.device_status()
    if status != binding.OK:
        raise SystemExit(f"device status {status} after the timed region")

    # ---- per-layer events: the dominant kernel's own duration, live ------------------------------
    # The same launches as a step, issued layer by layer through the C-ABI with an event between
    # layers. Layers of type FULL are exactly one launch of the streaming attention kernel.
    nrep = max(3, min(args.steps, 20))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(w.num_layers + 1)] for _ in range(nrep)]
    idx, cnt = step.idx, step.idx_count
    for r in range(nrep):
        evs[r][0].record()
        for i, tkind in enumerate(w.sched):
            if tkind == synth.LAYER_FULL:
                td.full_attn(layers[i], qs[i], out=outs[i])
            elif tkind == synth.LAYER_SELECT:
                td.select_attn(layers[i], qs[i], w.k, gran, out=outs[i], idx=idx, idx_count=cnt)
            else:
                td.sparse_attn(layers[i], qs[i], idx, cnt, out=outs[i])
            evs[r][i + 1].record()
    torch.cuda.synchronize()
    per_type = {0: [], 1: [], 2: []}
    for r in range(nrep):
        for i, tkind in enumerate(w.sched):
            per_type[tkind].append(evs[r][i].elapsed_time(evs[r][i + 1]) * 1e3)
    layer_us = {k: (sum(v) / len(v) if v else None) for k, v in per_type.items()}
    full_layers = [i for i, tk in enumerate(w.sched) if tk == synth.LAYER_FULL]
    dense_bytes = sum(kv_bytes[i] for i in full_layers) / max(1, len(full_layers)) if full_layers else kv_bytes[0]
    dense_us = layer_us[0] if layer_us[0] else layer_us[1]
    peak, peak_kind = measured_peak_gbs()
    achieved = dense_bytes / (dense_us * 1e-6) / 1e9
    sparse_bytes = w.batch * gather_lists * min(w.k, w.ctx) * 512 + w.batch * index_heads * min(w.k, w.ctx) * 4
    roofline = {"bound": "hbm", "kernel": "attn_kernel<FULL> (full-attention layers; the selection layers run the same loop)",
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(w.name), "bytes_per_launch": dense_bytes,
                "us_per_launch": dense_us}
    layers_report = {
        "note": "full_us / select_us_incl_topk / sparse_us: one C-ABI call per layer from Python with an event "
                "between calls (includes host gaps); *_in_step: the same kernels back to back inside tidal_decode_step",
        "full_us": layer_us[0], "select_us_incl_topk": layer_us[1], "sparse_us": layer_us[2],
        "select_frac_of_8TBs": (dense_bytes / (layer_us[1] * 1e-6) / 1e9 / NOMINAL_HBM_GBS) if layer_us[1] else None,
        "sparse_GBs": (sparse_bytes / (layer_us[2] * 1e-6) / 1e9) if layer_us[2] else None,
        "sparse_frac_of_8TBs": (sparse_bytes / (layer_us[2] * 1e-6) / 1e9 / NOMINAL_HBM_GBS) if layer_us[2] else None,
    }
    step_bytes = sum(kv_bytes[i] if tk != synth.LAYER_SPARSE else sparse_bytes for i, tk in enumerate(w.sched))

    # ---- the same layers in situ: sub-schedules run through tidal_decode_step (no host gaps between
    # launches, programmatic dependent launch active), differences of CUDA-event times ------------------
    def time_schedule(ids, kinds):
        st = td.make_step(kinds, [layers[i] for i in ids], [qs[i] for i in ids], [outs[i] for i in ids], w.k, gran)
        for _ in range(3):
            st()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(nrep):
            st()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / nrep

    # The streaming kernel back to back over distinct layer caches (any layer's cache can be run as a
    # full or as a selection layer): the dominant kernel's own duration without host gaps.
    nchain = min(8, w.num_layers)
    if nchain >= 2:
        chain_ids = list(range(nchain))
        full_chain_us = time_schedule(chain_ids, [synth.LAYER_FULL] * nchain) / nchain
        sel_chain_us = time_schedule(chain_ids, [synth.LAYER_SELECT] * nchain) / nchain
        chain_bytes = sum(kv_bytes[i] for i in chain_ids) / nchain
        achieved = chain_bytes / (full_chain_us * 1e-6) / 1e9
        roofline.update({"achieved": achieved, "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                         "bytes_per_launch": chain_bytes, "us_per_launch": full_chain_us,
                         "measured": f"{nchain} launches of the full-attention kernel over {nchain} distinct layer caches "
                                     "through tidal_decode_step, CUDA events on the launching stream, average per launch"})
        layers_report.update({"full_us_in_step": full_chain_us, "select_us_incl_topk_in_step": sel_chain_us,
                              "select_in_step_frac_of_8TBs": chain_bytes / sel_chain_us / 1e3 / NOMINAL_HBM_GBS})

    sel_ids = [i for i, tk in enumerate(w.sched) if tk == synth.LAYER_SELECT]
    sp_ids = [i for i, tk in enumerate(w.sched) if tk == synth.LAYER_SPARSE]
    if sel_ids and len(sp_ids) >= 2:
        t_sel = time_schedule(sel_ids[:1], [synth.LAYER_SELECT])
        t_chain = time_schedule(sel_ids[:1] + sp_ids, [synth.LAYER_SELECT] + [synth.LAYER_SPARSE] * len(sp_ids))
        sp_in = (t_chain - t_sel) / len(sp_ids)
        layers_report.update({
            "select_us_alone_in_decode_step_call": t_sel,
            "sparse_us_in_step": sp_in,
            "sparse_in_step_GBs": sparse_bytes / sp_in / 1e3,
            "sparse_in_step_frac_of_8TBs": sparse_bytes / sp_in / 1e3 / NOMINAL_HBM_GBS,
        })

    # ---- end to end through the host-buffer entry point ----------------------------------------------
    q_host = torch.stack([q.cpu() for q in qs]).contiguous().pin_memory()
    out_host = torch.empty(w.num_layers, w.batch, w.num_q_heads, w.head_dim, dtype=torch.float32).pin_memory()
    step_host = td.make_step_host(w.sched, layers, q_host, out_host, w.k, gran)
    for _ in range(args.warmup):
        step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step_host()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_us = max_over_ranks(e2e_s, dist, dev) / args.steps * 1e6
    if not torch.allclose(out_host[0].to(dev), outs[0], rtol=0, atol=1e-3):
        raise SystemExit("host-buffer step and device step disagree")

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        us, cores, sample, _ = oracle_sample(w, qs, layers, index_heads=index_heads)
        cpu = {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": whole_job_us_per_step(ms_step, world), "unit": "us", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": describe(w), "replicas": world, "granularity": args.granularity,
                       "launch": "tidal_decode_step on a non-default stream: the step's kernels are recorded once as a "
                                 "CUDA graph by the library and replayed (gpu_launches counts the kernels, not the graphs)",
                       "l2": ("every layer has its own KV cache: %.2f GiB are streamed or gathered from per step, %s the "
                              "126 MB L2%s" % (sum(kv_bytes) / 2**30,
                                              "far more than" if sum(kv_bytes) > 4 * 126e6 else "NOT more than a few times",
                                              "" if sum(kv_bytes) > 4 * 126e6 else ": this workload is L2-warm and not a bandwidth figure")),
                       "step_bytes": step_bytes,
                       "step_frac_of_8TBs": step_bytes / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
            "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_us / world, "unit": "us", "h2d_bytes_per_step": q_host.numel() * 2,
                    "d2h_bytes_per_step": out_host.numel() * 4},
            "roofline": roofline, "layers": layers_report, "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
