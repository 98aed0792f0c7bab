#!/usr/bin/env python
"""Throughput of the SpindleKV prefill reduction pass (all layers of one prompt) on B200.

One "step" = the whole hot path over one synthetic prompt batch: plan, evict every deep layer
(window scores, top-k, gather of K and V), build K and V CodeBooks for every shallow layer
(magnitudes, similarity, greedy cover, numbering, gather of the centres).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl reference]

Prints one JSON line.  With N > 1 (under torchrun) every rank compresses its own prompt: the units
of this pass are independent, so more GPUs means more prompts and no data-path collective.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2507_06517_b200 import synth

METRIC = "prompt tokens compressed/s (all layers)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of the similarity kernel per unit (one head's K or V of one
# layer), by sequence length, from the ncu capture summarised under profiles/ (8 units per launch there;
# traffic grows in proportion to the units of a launch).  Lengths without a capture report null.
SIMILARITY_TRAFFIC_BYTES_PER_UNIT = {16384: 19.7e6}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (profiling on a small case)")
    ap.add_argument("--shallow", type=int, default=None, help="override the number of CodeBook layers")
    ap.add_argument("--literal", action="store_true",
                    help="the paper's own composition: every layer evicts, then builds CodeBooks of what it kept")
    ap.add_argument("--repeat", action="store_true",
                    help="with --literal: unfold GQA, every query head selects its own tokens (Section 3.3)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-chunk", type=int, default=4, help="CodeBook layers per upload/compute/download group")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload_config(wl, extra=None):
    cfg = {"workload": f"{wl.name}: B{wl.batch} x {wl.n_layers} layers ({wl.n_shallow} CodeBook + "
                       f"{wl.n_layers - wl.n_shallow} evict), {wl.n_q_heads}/{wl.n_kv_heads} heads, d{wl.head_dim}, "
                       f"N={'/'.join(map(str, wl.seq_lens)) if wl.packed else wl.max_len}, {wl.dtype}, w{wl.window}",
           "tokens_per_step": wl.total_tokens,
           "l2": "inputs larger than L2 (K and V of all layers are read once per step)"}
    if extra:
        cfg.update(extra)
    return cfg


# ---- CPU baseline: the checker, as it stands, on a bounded sample ------------------------------

def oracle_sample_seconds(wl):
    """Times the CPU checker on (shallow layer 0, head 0: K and V CodeBooks) and on one deep layer
    (all heads) of sequence 0, and scales by unit counts to one whole step."""
    from oracle import spindlekv_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([int(x.get("num_threads", 1)) for x in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    ns, nd = wl.n_shallow, wl.n_layers - wl.n_shallow
    units = wl.batch * wl.n_kv_heads
    total = 0.0
    parts = []
    scale_len = wl.total_tokens / (wl.seq_lens[0])  # sequences other than 0: scaled by length
    if ns:
        k, v = synth.unit_kv(wl, 0, 0, 0)
        t0 = time.perf_counter()
        O.codebook_shallow(k.astype(np.float64), wl.theta_k)
        t1 = time.perf_counter()
        O.codebook_shallow(v.astype(np.float64), wl.theta_v)
        t2 = time.perf_counter()
        # cost grows with the square of the length; other sequences are scaled accordingly
        sq = sum(float(l) ** 2 for l in wl.seq_lens) / float(wl.seq_lens[0]) ** 2
        total += ((t1 - t0) + (t2 - t1)) * ns * wl.n_kv_heads * sq
        parts.append(f"layer 0 head 0 K+V CodeBooks ({t2 - t0:.1f} s)")
    if nd:
        lam = ns
        ks = np.stack([synth.unit_kv(wl, lam, 0, j)[0] for j in range(wl.n_kv_heads)])
        q = synth.window_queries(wl, lam, 0, list(ks))
        _, _, kplan = O.plan_layers(wl.n_layers, ns, wl.seq_lens, wl.window, wl.beta,
                                    reserve_ratio=wl.budget_frac, budget_tokens=wl.budget_tokens)
        t0 = time.perf_counter()
        res = O.evict_deep(q.astype(np.float64), ks.astype(np.float64), int(kplan[lam, 0]))
        for j in range(wl.n_kv_heads):
            O.gather_rows(ks[j], res["keep"][j])
        t1 = time.perf_counter()
        total += (t1 - t0) * nd * scale_len
        parts.append(f"layer {lam} all heads eviction ({t1 - t0:.1f} s)")
    return total, cores, "extrapolated by unit count from: " + "; ".join(parts)


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    sample = ""
    cores = 1
    for i in range(args.warmup + args.steps):
        t, cores, sample = oracle_sample_seconds(wl)
        if i >= args.warmup:
            times.append(t)
        if sum(times) > 0 and (time.perf_counter() - T_START) > 240:
            break
    sec = statistics.median(times)
    val = wl.total_tokens / sec
    line = {"metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": len(times),
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": workload_config(wl),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- clocks ---------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows = []
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for t, line in self.rows:
            if t < t0 or t > t1 + 0.2:
                continue
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---- native arm -------------------------------------------------------------------------------------

def host_inputs(wl):
    """Pinned host tensors K, V [m, ...] and Q [deep layers, B, H_q, w, d] in the storage dtype."""
    from concurrent.futures import ThreadPoolExecutor
    dt = torch.float32 if wl.dtype == "f32" else torch.bfloat16
    ns = wl.n_shallow

    def one(lam):
        K, V, Q = synth.layer_arrays(wl, lam, need_q=lam >= ns)
        return (torch.from_numpy(K).to(dt), torch.from_numpy(V).to(dt), None if Q is None else torch.from_numpy(Q).to(dt))

    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        layers = list(ex.map(one, range(wl.n_layers)))
    K = torch.stack([x[0] for x in layers]).pin_memory()
    V = torch.stack([x[1] for x in layers]).pin_memory()
    Q = torch.stack([x[2] for x in layers[ns:]]).pin_memory() if wl.n_layers > ns else None
    return K, V, Q


def run_literal(args, wl):
    """Every layer evicts under the pyramid over all layers, then builds K and V CodeBooks of the kept
    tokens (Section 3 as written).  Single GPU; reports throughput and the reserve ratios of Eq. (15)."""
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVLiteralPass, SpindleKVRepeatPass
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the reduction pass has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = wl.replace(n_shallow=0)   # window queries for every layer
    hK, hV, hQ = host_inputs(wl)
    cfg = B.Config(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                   window=wl.window, n_shallow=-1, beta=wl.beta, theta_k=wl.theta_k, theta_v=wl.theta_v,
                   budget_tokens=wl.budget_tokens if wl.budget_tokens is not None else -1.0,
                   reserve_ratio=wl.budget_frac if wl.budget_frac is not None else -1.0)
    p = (SpindleKVRepeatPass if args.repeat else SpindleKVLiteralPass)(cfg, wl.seq_lens, hK.dtype, device=dev)
    dK, dV, dQ = hK.to(dev), hV.to(dev), hQ.to(dev)
    for _ in range(max(args.warmup, 3)):
        p.run(dK, dV, dQ)
    st = p.device_status()
    if st["evict"][0] or st["codebook"][0]:
        raise RuntimeError(f"device status {st}")
    B.spindlekv_launch_count(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record()
    for _ in range(args.steps):
        p.run(dK, dV, dQ)
    ev1.record()
    torch.cuda.synchronize(dev)
    ms = ev0.elapsed_time(ev1)
    launches = B.spindlekv_launch_count(True)
    nk, nv = p.cb["K"]["n_entries"].cpu().numpy(), p.cb["V"]["n_entries"].cpu().numpy()
    kept = p.kept_host[:, 0].astype(np.float64)       # tokens kept per head (per query head when unfolded)
    heads = wl.n_q_heads if args.repeat else wl.n_kv_heads   # Eq. (15): h_g = h after a repeat
    r1 = kept / wl.max_len
    r2 = (nk[:, 0].sum(axis=1) + nv[:, 0].sum(axis=1)) / (2.0 * heads * kept)
    line = {"metric": METRIC + (", composition as written, GQA unfolded" if args.repeat else ", composition as written"), "value": wl.total_tokens * args.steps / (ms * 1e-3),
            "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": workload_config(wl, {"composition": "every layer: evict (pyramid over all layers), then CodeBooks of the kept tokens"}),
            "gpu_launches": int(launches),
            "reserve_ratio": {"r1_mean": float(r1.mean()), "r2_mean": float(r2.mean()), "r1_r2_mean": float((r1 * r2).mean()),
                              "kept_first_last": [int(kept[0]), int(kept[-1])]}}
    print(json.dumps(line))


def run_native(args, wl):
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the reduction pass has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # every rank compresses its own prompt (different seed)
    from paper_2507_06517_b200 import sharding
    wl = sharding.rank_workload(wl, rank)
    dev = torch.device("cuda", local_rank)
    cfg = B.Config(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                   window=wl.window, n_shallow=wl.n_shallow, beta=wl.beta, theta_k=wl.theta_k, theta_v=wl.theta_v,
                   budget_tokens=wl.budget_tokens if wl.budget_tokens is not None else -1.0,
                   reserve_ratio=wl.budget_frac if wl.budget_frac is not None else -1.0)
    hK, hV, hQ = host_inputs(wl)
    dtype = hK.dtype
    p = SpindleKVPass(cfg, wl.seq_lens, dtype, device=dev)
    dK = torch.empty_like(hK, device=dev)
    dV = torch.empty_like(hV, device=dev)
    dQ = torch.empty_like(hQ, device=dev) if hQ is not None else None

    def upload():
        dK.copy_(hK, non_blocking=True)
        dV.copy_(hV, non_blocking=True)
        if dQ is not None:
            dQ.copy_(hQ, non_blocking=True)

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, steps):
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            fn()
        ev1.record()
        barrier()
        tokens, ms = sharding.aggregate(wl.total_tokens, ev0.elapsed_time(ev1), dist, dev)
        timed.tokens = tokens
        return ms

    upload()
    step = lambda: p.run(dK, dV, dQ)
    for _ in range(max(args.warmup, 3)):
        step()
    st = p.device_status()
    for k, v in st.items():
        if v[0] != 0:
            raise RuntimeError(f"device status {v} in {k}")
    sampler = ClockSampler(local_rank) if rank == 0 else None
    B.spindlekv_launch_count(True)
    t0 = time.perf_counter()
    ms = timed(step, args.steps)
    t1 = time.perf_counter()
    job_tokens = timed.tokens
    launches = B.spindlekv_launch_count(True)
    clocks = sampler.stop(t0, t1) if sampler else None

    e2e = None
    if not args.no_e2e:
        # the same pass through the host-buffer call: K, V, Q start in pinned host memory and every result
        # (index maps, counts, magnitudes, kept rows, CodeBook rows) ends there, each step
        p2 = SpindleKVPass(cfg, wl.seq_lens, dtype, device=dev, layers_per_codebook_call=args.e2e_chunk)
        host_out = p2.host_outputs()
        h2d = sum(t.numel() * t.element_size() for t in (hK, hV) + ((hQ,) if hQ is not None else ()))
        d2h = sum(t.numel() * t.element_size() for t in host_out.values())
        step_e2e = lambda: p2.run_from_host(hK, hV, hQ, host_out)
        step_e2e()
        torch.cuda.synchronize(dev)
        for g in ("K", "V") if p.n_shallow else ():
            for k in ("ref", "n_entries"):
                if not torch.equal(host_out[f"{g}.{k}"], p.cb[g][k].cpu()):
                    raise RuntimeError(f"host-fed pass disagrees with the resident pass on {g}.{k}")
        if p.n_deep and not torch.equal(host_out["keep_cnt"], p.keep_cnt.cpu()):
            raise RuntimeError("host-fed pass disagrees with the resident pass on keep_cnt")
        ms_e2e = timed(step_e2e, args.steps)
        e2e = {"value": sharding.throughput(timed.tokens, args.steps, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps,
               "codebook_layers_per_group": args.e2e_chunk}
        del p2

    # per-kernel times: one more pass with event pairs around every launch
    B.spindlekv_timing_enable(True)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize(dev)
    kt = B.spindlekv_timing_read()
    B.spindlekv_timing_enable(False)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    pk, pk_src = peaks()
    total_ms = sum(v[0] for v in kt.values()) or 1.0
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps,
                   "share": v[0] / total_ms} for k, v in kt.items() if v[1]}
    # algorithmic bytes per step of the bandwidth-bound kernels (what must move at least once) against
    # the measured HBM copy rate
    e = 4 if wl.dtype == "f32" else 2
    tok, Hk, d = wl.total_tokens, wl.n_kv_heads, wl.head_dim
    nd, ns = wl.n_layers - wl.n_shallow, wl.n_shallow
    alg = {}
    if nd:
        kept = int(p.keep_cnt.sum().item())
        alg["window_score"] = nd * (tok * Hk * d * e + wl.batch * wl.n_q_heads * wl.window * d * e + 4 * Hk * tok)
        alg["topk"] = nd * Hk * 4 * tok + 4 * kept
        alg["gather"] = 2 * 2 * kept * d * e
    if ns:
        entries = sum(int(p.cb[g]["n_entries"].sum().item()) for g in ("K", "V"))
        alg["norms"] = 2 * ns * (tok * Hk * d * e + 4 * Hk * tok)
        alg["gather"] = alg.get("gather", 0) + 2 * entries * d * e
    for k, nbytes in alg.items():
        if k in kernels and kernels[k]["ms_per_step"] > 0:
            gbs = nbytes / (kernels[k]["ms_per_step"] * 1e-3) / 1e9
            kernels[k].update({"bound": "hbm", "algorithmic_bytes": nbytes, "achieved_gbs": gbs,
                               "frac_of_hbm_peak": gbs / pk["hbm_gbs"]})
    if nd and "window_score" in kernels and kernels["window_score"]["ms_per_step"] > 0 and wl.dtype == "bf16":
        # the window-score kernel takes one exponential per (query row, key) in each of its two passes; the
        # special-function units deliver 16 per clock and SM (148 SMs, the SM clock sampled during the run)
        h_n = wl.n_q_heads // wl.n_kv_heads
        exps = 2.0 * h_n * wl.window * tok * Hk * nd
        mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        peak = 16.0 * 148 * mhz * 1e6
        rate = exps / (kernels["window_score"]["ms_per_step"] * 1e-3)
        kernels["window_score"]["exp_unit"] = {"exponentials_per_step": exps, "achieved_per_s": rate,
                                               "peak_per_s": peak, "frac": rate / peak, "sm_mhz": mhz}
    roof = None
    if p.n_shallow and kt["similarity"][1]:
        sim_ms, sim_n = kt["similarity"]
        units_per_launch = 2 * wl.n_shallow * wl.n_kv_heads * wl.batch / (sim_n / args.steps)
        flops_per_step = sum(float(l) * (l - 1) * wl.head_dim for l in wl.seq_lens) * 2 * wl.n_shallow * wl.n_kv_heads
        achieved = flops_per_step * args.steps / (sim_ms * 1e-3) / 1e12
        peak = pk["bf16_tflops_sustained"] if wl.dtype == "bf16" else pk["bf16_tflops_sustained"] / 32.0
        traffic = None
        if not wl.packed and wl.max_len in SIMILARITY_TRAFFIC_BYTES_PER_UNIT and wl.head_dim == 128:
            traffic = SIMILARITY_TRAFFIC_BYTES_PER_UNIT[wl.max_len] * units_per_launch
        roof = {"kernel": "similarity (Eq. 4, 9)", "bound": "tensor", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": traffic, "peak_source": pk_src,
                "avg_launch_ms": sim_ms / sim_n, "algorithmic_flops_per_launch": flops_per_step * args.steps / sim_n}
    line = {"metric": METRIC, "value": sharding.throughput(job_tokens, args.steps, ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
            "data": "synthetic", "config": workload_config(wl, {"parallelism": f"replicas x{world}"}),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roof, "kernels": kernels,
            "greedy_rounds": st.get("codebook", (0, [0]))[1][0]}
    if not args.no_cpu_baseline and world == 1:
        sec, cores, sample = oracle_sample_seconds(wl)
        line["cpu_baseline"] = {"value": wl.total_tokens / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": sample}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


T_START = time.perf_counter()

if __name__ == "__main__":
    a = parse_args()
    w = synth.workload(a.workload)
    if a.layers is not None:
        w = w.replace(n_layers=a.layers, n_shallow=a.shallow if a.shallow is not None else a.layers // 2,
                      name=f"{w.name}[{a.layers} layers]")
    if a.impl == "reference":
        run_reference(a, w)
    elif a.literal:
        run_literal(a, w)
    else:
        run_native(a, w)
