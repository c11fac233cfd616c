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
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")


def ncu_traffic(workload: str) -> dict:
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of each kernel, as
    `python -m paper_2410_05076_b200.ncu_summary` extracted them from an ncu capture. Lines read
    `<workload> <kernel> <bytes>`; a missing file or workload gives an empty dict (traffic: null)."""
    out = {}
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 3 and parts[0] == workload:
                    out[parts[1]] = float(parts[2])
    except OSError:
        pass
    return out


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


def build_workload(w: synth.Workload, device, kv_dtype: str = "bf16"):
    """Queries and per-layer caches; with kv_dtype 'fp8' every cache is stored as E4M3 codes with
    per-KV-head scales (the bf16 original of a layer is dropped as soon as it has been converted)."""
    qs = [synth.make_q(w, i, device) for i in range(w.num_layers)]
    conv = synth.to_fp8 if kv_dtype == "fp8" else (lambda l: l)
    if w.paged:
        pt, total = synth.make_page_table(w)
        layers = [conv(synth.make_layer(w, i, device, layout="paged", q=qs[i], page_table=pt, num_pages=total))
                  for i in range(w.num_layers)]
    else:
        layers = [conv(synth.make_layer(w, i, device, q=qs[i])) for i in range(w.num_layers)]
    return qs, layers


def row_bytes(kv_dtype: str) -> int:
    """Bytes of one gathered position of one KV head: a key row and a value row."""
    return 256 if kv_dtype == "fp8" else 512


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


def oracle_sample(w: synth.Workload, qs, layers, host_cache=None, index_heads=None, repeats: int = 3):
    """Time the CPU oracle, as it stands, on one layer of each type (median of `repeats` runs each)
    and scale by the layer mix. Only the oracle calls are timed; the host copies of the sampled layers
    may be cached by the caller."""
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
        if t == 2 and rho is None:
            _, idx, cnt = oracle.select_attn(okv, qb, w.k, index_heads)
            rho = (idx, cnt)
        samples = []
        for _ in range(repeats):
            t0 = time.perf_counter()
            if t == 0:
                oracle.full_attn(okv, qb)
            elif t == 1:
                _, idx, cnt = oracle.select_attn(okv, qb, w.k, index_heads)
                rho = (idx, cnt)
            else:
                oracle.sparse_attn(okv, qb, rho[0], rho[1])
            samples.append(time.perf_counter() - t0)
        times[t] = statistics.median(samples)
        del okv
    total = sum(times[t] * w.sched.count(t) for t in times)
    sample = (f"one layer of each type (layers " + ",".join(str(first[t]) for t in sorted(first)) +
              f"), median of {repeats} runs each, scaled by the {w.sched.count(0)}+{w.sched.count(1)}+{w.sched.count(2)} layer mix")
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


def profile_case(td, w, dev, steps, kv_dtype="bf16"):
    """One layer of each type (about 1.5 GiB at cfg3), run in the order full, select, sparse."""
    need = [w.sched.index(t) if t in w.sched else 0 for t in (0, 1, 2)]
    qs = {i: synth.make_q(w, i, dev) for i in set(need)}
    conv = synth.to_fp8 if kv_dtype == "fp8" else (lambda l: l)
    if w.paged:
        pt, total = synth.make_page_table(w)
        layers = {i: conv(synth.make_layer(w, i, dev, layout="paged", q=qs[i], page_table=pt, num_pages=total))
                  for i in set(need)}
    else:
        layers = {i: conv(synth.make_layer(w, i, dev, q=qs[i])) for i in set(need)}
    torch.cuda.synchronize()
    idx = cnt = None
    outs = [torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.float32, device=dev) for _ in range(3)]
    step = td.make_step([synth.LAYER_FULL, synth.LAYER_SELECT, synth.LAYER_SPARSE], [layers[i] for i in need],
                        [qs[i] for i in need], outs, w.k)
    for _ in range(steps):
        # the single-layer entry points (fused selection kernel) ...
        td.full_attn(layers[need[0]], qs[need[0]])
        _, idx, cnt = td.select_attn(layers[need[1]], qs[need[1]], w.k)
        td.sparse_attn(layers[need[2]], qs[need[2]], idx, cnt)
        # ... and the same three layers as a step (selection layer in two passes where that applies)
        step()
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
    return {"sweep": "cfg5: B1 32q/8kv d128; per-layer cost of a selection layer (attention + top-k) and "
                     "of a sparse layer, from chains of layers run through tidal_decode_step over distinct "
                     "KV copies (cold in L2), CUDA events", "reps": reps, "points": points}


def time_schedule(td, kinds, layers, qs, outs, k, gran, nrep):
    """One sub-schedule run through tidal_decode_step nrep times (no host gaps between its launches, the
    library's step graph and the overlap between layers active): CUDA events, microseconds per run."""
    st = td.make_step(list(kinds), list(layers), list(qs), list(outs), k, gran)
    for _ in range(3):
        st()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(nrep):
        st()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / nrep


def layers_in_step(td, w, layers, qs, outs, gran, nrep):
    """Per-layer-type cost inside a step, from differences of sub-schedule times over the workload's own
    layer caches (every launch finds its cache cold in L2):
      full    a chain of full-attention layers over distinct caches, per layer;
      sparse  (selection layer + all sparse layers) minus (that selection layer alone), per sparse layer;
      select  the workload's schedule from its first selection layer on, minus the same schedule with the
              second selection layer run as a sparse layer, plus one sparse layer: a selection layer
              (attention + top-k) in its real surroundings, including what it costs the sparse layer after
              it, which must wait for the new index list."""
    ts = lambda ids, kinds: time_schedule(td, kinds, [layers[i] for i in ids], [qs[i] for i in ids],
                                          [outs[i] for i in ids], w.k, gran, nrep)
    F, S, P = synth.LAYER_FULL, synth.LAYER_SELECT, synth.LAYER_SPARSE
    out = {}
    nchain = min(8, w.num_layers)
    if nchain >= 2:
        out["full_us"] = ts(range(nchain), [F] * nchain) / nchain
        out["full_bytes"] = sum(layers[i].kv_bytes() for i in range(nchain)) / nchain
    sel_ids = [i for i, tk in enumerate(w.sched) if tk == S]
    sp_ids = [i for i, tk in enumerate(w.sched) if tk == P]
    if sel_ids and sp_ids:
        t_sel = ts(sel_ids[:1], [S])
        t_chain = ts(sel_ids[:1] + sp_ids, [S] + [P] * len(sp_ids))
        out["sparse_us"] = (t_chain - t_sel) / len(sp_ids)
        out["select_alone_us"] = t_sel
        if len(sel_ids) >= 2:
            tail = list(range(sel_ids[0], w.num_layers))
            kinds = [w.sched[i] for i in tail]
            kinds_one = [P if (i == sel_ids[1]) else w.sched[i] for i in tail]
            out["select_us"] = ts(tail, kinds) - ts(tail, kinds_one) + out["sparse_us"]
            out["select_bytes"] = layers[sel_ids[1]].kv_bytes()
        else:
            out["select_us"] = t_sel
            out["select_bytes"] = layers[sel_ids[0]].kv_bytes()
    return out


def quick_workload(td, name, dev, gran, nrep, kv_dtype: str = "bf16"):
    """Step time and per-layer-type times of another configuration (compact: for the line's other_workloads)."""
    w = synth.workload(name)
    qs, layers = build_workload(w, dev, kv_dtype)
    outs = [torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.float32, device=dev) for _ in layers]
    step_us = time_schedule(td, w.sched, layers, qs, outs, w.k, gran, nrep)
    lt = layers_in_step(td, w, layers, qs, outs, gran, max(3, nrep // 2))
    sparse_bytes = sum(min(w.k, n) for n in w.ctx_lens()) * w.num_q_heads * (row_bytes(kv_dtype) + 4)
    res = {"workload": describe(w) + (" [KV as FP8 E4M3 codes]" if kv_dtype == "fp8" else ""), "step_us": round(step_us, 2)}
    if "full_us" in lt:
        res["full_us"] = round(lt["full_us"], 2)
        res["full_frac_of_8TBs"] = round(lt["full_bytes"] / lt["full_us"] / 1e3 / NOMINAL_HBM_GBS, 3)
    if "select_us" in lt:
        res["select_us_incl_topk"] = round(lt["select_us"], 2)
        res["select_frac_of_8TBs"] = round(lt["select_bytes"] / lt["select_us"] / 1e3 / NOMINAL_HBM_GBS, 3)
    if "sparse_us" in lt:
        res["sparse_us"] = round(lt["sparse_us"], 2)
        res["sparse_frac_of_8TBs"] = round(sparse_bytes / lt["sparse_us"] / 1e3 / NOMINAL_HBM_GBS, 3)
    assert td.device_status() == 0
    del qs, layers, outs
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="tidal", choices=["tidal", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv-dtype", default="bf16", choices=["bf16", "fp8"],
                    help="element type of the KV cache: bf16 (the metric's configuration) or fp8 (E4M3 codes with "
                         "per-KV-head scales; reported as a variant, never as the headline)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the compact figures for cfg1, cfg2, cfg64, cfg4 and the cfg5 sweep")
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
        profile_case(td, w, dev, args.steps, args.kv_dtype)
        return
    if args.sweep:
        print(json.dumps(sweep(td, dev, max(3, min(args.steps, 30)))), flush=True)
        return
    qs, layers = build_workload(w, dev, args.kv_dtype)
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

    # ---- the layers in situ: the dominant kernel's own duration, live -------------------------------
    nrep = max(3, min(args.steps, 20))
    peak, peak_kind = measured_peak_gbs()
    lt = layers_in_step(td, w, layers, qs, outs, gran, nrep)
    k_eff = [min(w.k, n) for n in w.ctx_lens()]
    sparse_bytes = sum(k_eff) * (gather_lists * row_bytes(args.kv_dtype) + index_heads * 4)
    traffic = ncu_traffic(w.name)

    def kernel_entry(kernel, bytes_per_launch, us, traffic_key, launches_per_step, note=None):
        if not us:
            return None
        ach = bytes_per_launch / us / 1e3
        e = {"kernel": kernel, "achieved": ach, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
             "frac": ach / peak, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
             "traffic": traffic.get(traffic_key), "bytes_per_launch": bytes_per_launch, "us_per_launch": us,
             "launches_per_step": launches_per_step, "share_of_step": launches_per_step * us / (ms_step * 1e3)}
        if note:
            e["note"] = note
        return e

    n_full, n_sel, n_sp = w.sched.count(0), w.sched.count(1), w.sched.count(2)
    sparse_entry = kernel_entry("attn_kernel<SPARSE> (sparse layers: gather of the selected K/V rows)", sparse_bytes,
                                lt.get("sparse_us"), "sparse", n_sp)
    full_entry = kernel_entry("attn_kernel<FULL> (full-attention layers)", lt.get("full_bytes", 0), lt.get("full_us"),
                              "full", n_full)
    select_entry = kernel_entry("attn_kernel<SELECT> + top-k (selection layers)", lt.get("select_bytes", 0),
                                lt.get("select_us"), "select", n_sel,
                                "bytes_per_launch counts the KV cache only; the scores (4 B per position and query "
                                "head, written once and read back from L2) are not in the denominator")
    if select_entry:
        # inside a step the selection layer runs as key pass + value pass where that applies, else fused
        two_pass = args.granularity == "qhead" and w.batch == 1 and traffic.get("score") is not None
        parts = ("score", "value", "topk") if two_pass else ("select", "topk")
        select_entry["traffic"] = sum(traffic[k] for k in parts) if all(traffic.get(k) is not None for k in parts) else None
        select_entry["kernel"] = ("score_pass_kernel + value_pass_kernel + top-k (selection layers, two passes)" if two_pass
                                  else select_entry["kernel"])
    # the kernel with the largest share of the step leads; the others follow as siblings
    entries = [e for e in (sparse_entry, full_entry, select_entry) if e]
    entries.sort(key=lambda e: -e["share_of_step"])
    roofline = {"bound": "hbm"}
    roofline.update(entries[0])
    roofline["measured"] = ("per-launch time = difference of sub-schedule times run through tidal_decode_step over the "
                            "workload's own layer caches (cold in L2), CUDA events on the launching stream; traffic = "
                            "dram__bytes_read.sum + dram__bytes_write.sum of one launch from the ncu capture summarised "
                            "under profiles/ (null if not captured for this workload)")
    roofline["target"] = "north star: selection and sparse layers at >= 0.70 of 8 TB/s (frac_of_nominal_8TBs)"
    roofline["siblings"] = entries[1:]
    step_bytes = sum(kv_bytes[i] if tk != synth.LAYER_SPARSE else sparse_bytes for i, tk in enumerate(w.sched))
    layers_report = {
        "note": "microseconds per layer inside tidal_decode_step (see roofline.measured); sum_check = "
                "full*n_full + select*n_select + sparse*n_sparse, to be compared with value",
        "full_us_in_step": lt.get("full_us"), "select_us_incl_topk_in_step": lt.get("select_us"),
        "sparse_us_in_step": lt.get("sparse_us"), "select_us_alone_in_decode_step_call": lt.get("select_alone_us"),
        "sum_check_us": sum((lt.get(kx) or 0) * n for kx, n in (("full_us", n_full), ("select_us", n_sel), ("sparse_us", n_sp))),
    }
    # the same step with the overlap between layers switched off: every layer reads its query only after
    # the layer before it has finished, as a model with projections between the layers would need it
    td.set_layer_overlap(False)
    no_overlap_us = time_schedule(td, w.sched, layers, qs, outs, w.k, gran, nrep)
    td.set_layer_overlap(True)
    layers_report["step_us_without_layer_overlap"] = no_overlap_us

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
    h2d_bytes, d2h_bytes = q_host.numel() * 2, out_host.numel() * 4

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        us, cores, sample, _ = oracle_sample(w, qs, layers, index_heads=index_heads)
        cpu = {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample}

    # ---- the other configurations, compactly (one GPU, default run only) ------------------------------
    other = None
    if rank == 0 and world == 1 and not args.no_other_workloads and args.workload == "cfg3" and args.kv_dtype == "bf16":
        del step, step_host, qs, layers, outs
        torch.cuda.empty_cache()
        other = {"note": "step_us: the whole schedule through tidal_decode_step, CUDA events; per-layer figures as "
                         "in `layers`; fractions are algorithmic bytes / time / 8 TB/s (cfg1 is latency-bound: 5 MB per step)"}
        for name in ("cfg1", "cfg2", "cfg64", "cfg4"):
            other[name] = quick_workload(td, name, dev, gran, max(3, min(args.steps, 10)))
        # the headline workload with an 8-bit cache: half the bytes per layer (fractions are of those bytes)
        other["cfg3_kv_fp8"] = quick_workload(td, "cfg3", dev, gran, max(3, min(args.steps, 10)), "fp8")
        sw = sweep(td, dev, 3)
        other["cfg5_sweep"] = {"what": sw["sweep"], "columns": ["ctx", "k", "select_us_incl_topk", "sparse_us"],
                               "points": [[p["ctx"], p["k"], round(p["select_us_incl_topk"], 1), round(p["sparse_us"], 2)]
                                          for p in sw["points"]]}

    if rank == 0:
        line = {
            "metric": METRIC, "value": whole_job_us_per_step(ms_step, world), "unit": "us", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.kv_dtype == "bf16" else "fp8_e4m3 cache, fp16 products, fp32 accumulation",
            "data": "synthetic",
            "config": {"workload": describe(w) + ("" if args.kv_dtype == "bf16" else " [KV as FP8 E4M3 codes: a variant, not the metric's configuration]"),
                       "replicas": world, "granularity": args.granularity,
                       "launch": "tidal_decode_step on a non-default stream: the step's kernels are recorded once as a "
                                 "CUDA graph by the library and replayed (gpu_launches counts the kernels, not the graphs)",
                       "l2": ("every layer has its own KV cache: %.2f GiB are streamed or gathered from per step, %s the "
                              "126 MB L2%s" % (sum(kv_bytes) / 2**30,
                                              "far more than" if sum(kv_bytes) > 4 * 126e6 else "NOT more than a few times",
                                              "" if sum(kv_bytes) > 4 * 126e6 else ": this workload is L2-warm and not a bandwidth figure")),
                       "step_bytes": step_bytes,
                       "step_frac_of_8TBs": step_bytes / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
            "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_us / world, "unit": "us", "h2d_bytes_per_step": h2d_bytes,
                    "d2h_bytes_per_step": d2h_bytes},
            "roofline": roofline, "layers": layers_report, "cpu_baseline": cpu, "other_workloads": other,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
