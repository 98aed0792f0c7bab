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
SIMILARITY_TRAFFIC_BYTES_PER_UNIT = {16384: 5.27e6}


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
    ap.add_argument("--decode", action="store_true",
                    help="one decode step of attention over the replaced cache of every layer (Eq. 14 with RoPE re-applied)")
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

def oracle_sample_seconds(wl, gpu=None):
    """Times the CPU checker on the K and V CodeBooks of two heads of shallow layer 0 and on one deep layer
    (all heads) of sequence 0, and scales by unit counts to one whole step.

    ``gpu`` (optional, only looked at outside the timed sections): the GPU's adjacency of the same CodeBook units
    and its kept positions of the same deep layer; when given, the decisions that fall inside the 1e-4 margin
    are counted against the checker's and everything outside the margin must agree.
    """
    from oracle import spindlekv_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([int(x.get("num_threads", 1)) for x in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    ns, nd = wl.n_shallow, wl.n_layers - wl.n_shallow
    total = 0.0
    parts = []
    margins = {"rel_margin": 1e-4}
    scale_len = wl.total_tokens / (wl.seq_lens[0])  # sequences other than 0: scaled by length
    if ns:
        heads = list(range(min(2, wl.n_kv_heads)))
        spent = 0.0
        near = {"K": 0, "V": 0}
        flips = {"K": 0, "V": 0}
        pairs = 0
        for j in heads:
            k, v = synth.unit_kv(wl, 0, 0, j)
            for name, gamma, theta in (("K", k, wl.theta_k), ("V", v, wl.theta_v)):
                t0 = time.perf_counter()
                r = O.codebook_shallow(gamma.astype(np.float64), theta)
                spent += time.perf_counter() - t0
                m = np.triu(O.threshold_margin_mask(r["S"], theta, 1e-4), k=1)
                near[name] += int(m.sum())
                pairs += gamma.shape[0] * (gamma.shape[0] - 1) // 2
                if gpu is not None:
                    diff = np.triu(gpu["adj"][(name, j)] != r["G"], k=1)
                    if np.any(diff & ~m):
                        raise RuntimeError(f"adjacency of layer 0 head {j} {name} differs from the checker outside the 1e-4 margin")
                    flips[name] += int(diff.sum())
        # cost grows with the square of the length; other sequences are scaled accordingly
        sq = sum(float(l) ** 2 for l in wl.seq_lens) / float(wl.seq_lens[0]) ** 2
        total += spent / len(heads) * ns * wl.n_kv_heads * sq
        parts.append(f"layer 0 heads {heads} K+V CodeBooks ({spent:.1f} s)")
        margins["similarity"] = {"units": [f"layer 0 head {j}" for j in heads], "pairs_per_gamma": pairs // 2,
                                 "pairs_within_margin_of_theta": near,
                                 "decided_differently_from_checker": flips if gpu is not None else None}
    if nd:
        lam = ns
        ks = np.stack([synth.unit_kv(wl, lam, 0, j)[0] for j in range(wl.n_kv_heads)])
        q = synth.window_queries(wl, lam, 0, list(ks))
        _, _, kplan = O.plan_layers(wl.n_layers, ns, wl.seq_lens, wl.window, wl.beta,
                                    reserve_ratio=wl.budget_frac, budget_tokens=wl.budget_tokens)
        kk = int(kplan[lam, 0])
        t0 = time.perf_counter()
        res = O.evict_deep(q.astype(np.float64), ks.astype(np.float64), kk)
        for j in range(wl.n_kv_heads):
            O.gather_rows(ks[j], res["keep"][j])
        t1 = time.perf_counter()
        total += (t1 - t0) * nd * scale_len
        parts.append(f"layer {lam} all heads eviction ({t1 - t0:.1f} s)")
        near_k, differ = 0, 0
        for j in range(wl.n_kv_heads):
            m = O.topk_margin_mask(res["scores"][j], kk, 1e-4)
            near_k += int(m.sum())
            if gpu is not None:
                d = np.setxor1d(gpu["keep"][j][:kk], res["keep"][j][:kk])
                if not np.all(m[d]):
                    raise RuntimeError(f"kept set of layer {lam} head {j} differs from the checker outside the 1e-4 margin")
                differ += int(d.size)
        margins["top_k"] = {"unit": f"layer {lam}, sequence 0, {wl.n_kv_heads} heads", "k": kk,
                            "positions_within_margin_of_kth_score": near_k,
                            "kept_differently_from_checker": differ if gpu is not None else None}
    return total, cores, "extrapolated by unit count from: " + "; ".join(parts), margins


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    sample = ""
    cores = 1
    for i in range(args.warmup + args.steps):
        t, cores, sample, _ = oracle_sample_seconds(wl)
        if i >= args.warmup:
            times.append(t)
        if sum(times) > 0 and (time.perf_counter() - T_START) > 240:
            break
    sec = statistics.median(times)
    val = wl.total_tokens / sec
    line = {"metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": len(times),
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": workload_config(wl, {"parallelism": f"replicas x{args.gpus}"}),
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

    def wait_until_sampling(self, timeout=5.0):
        """Blocks until the first samples have arrived (the tool needs a moment to start), so that a short timed
        region is not over before the first one."""
        t_end = time.perf_counter() + timeout
        while self.proc is not None and len(self.rows) < 2 and time.perf_counter() < t_end:
            time.sleep(0.02)

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


def recorded(fn, dev):
    """``fn`` as a replay of its CUDA graph (one launch from the host per step) and the number of kernels a replay
    stands for; ``fn`` itself and 0 where recording is not possible."""
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import record_graph
    B.spindlekv_launch_count(True)
    try:
        graph = record_graph(fn, dev)
        return graph.replay, B.spindlekv_launch_count(True) // 2    # the recording runs fn twice
    except Exception as exc:   # noqa: BLE001
        print(f"[bench] CUDA graph capture failed ({exc}); direct calls", file=sys.stderr)
        return fn, 0


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
    step, per_replay = recorded(lambda: p.run(dK, dV, dQ), dev)
    for _ in range(max(args.warmup, 3)):
        step()
    st = p.device_status()
    if any(v[0] for v in st.values()):
        raise RuntimeError(f"device status {st}")
    B.spindlekv_launch_count(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize(dev)
    ms = ev0.elapsed_time(ev1)
    launches = B.spindlekv_launch_count(True) + per_replay * args.steps
    nk, nv = p.cb["K"]["n_entries"].cpu().numpy(), p.cb["V"]["n_entries"].cpu().numpy()
    kept = p.kept_host[:, 0].astype(np.float64)       # tokens kept per head (per query head when unfolded)
    heads = wl.n_q_heads if args.repeat else wl.n_kv_heads   # Eq. (15): h_g = h after a repeat
    # Eq. (15) per layer, evaluated by the library.  After a repeat h is the number of query heads: the CodeBooks of a
    # KV head then stand for all its query heads, whose slots in the per-head arrays beyond the first stay empty.
    pad = np.zeros(heads - wl.n_kv_heads, dtype=np.int32)
    rr = [B.spindlekv_reserve_ratio(wl.max_len, int(kept[lam]), np.concatenate([nk[lam, 0], pad]),
                                    np.concatenate([nv[lam, 0], pad])) for lam in range(wl.n_layers)]
    r1 = np.array([x[0] for x in rr])
    r2 = np.array([x[1] for x in rr])
    line = {"metric": METRIC + (", composition as written, GQA unfolded" if args.repeat else ", composition as written"), "value": wl.total_tokens * args.steps / (ms * 1e-3),
            "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": workload_config(wl, {"composition": "every layer: evict (pyramid over all layers), then CodeBooks of the kept tokens"}),
            "gpu_launches": int(launches),
            "reserve_ratio": {"r1_mean": float(r1.mean()), "r2_mean": float(r2.mean()), "r1_r2_mean": float((r1 * r2).mean()),
                              "kept_first_last": [int(kept[0]), int(kept[-1])]}}
    print(json.dumps(line))


def run_decode(args, wl):
    """CodeBooks of every layer (all tokens), then decode steps: the queries of one new token attend to the replaced
    cache of all layers.  Reports the time of a step and the bytes it has to read (CodeBook rows once, reference and
    magnitude per token) beside the bytes of the dense cache it stands for."""
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVDecodeAttention, SpindleKVPass
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the reduction pass has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = wl.replace(n_shallow=wl.n_layers, budget_tokens=None, budget_frac=1.0)
    hK, hV, _ = host_inputs(wl)
    cfg = B.Config(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                   window=wl.window, n_shallow=wl.n_layers, beta=wl.beta, theta_k=wl.theta_k, theta_v=wl.theta_v, reserve_ratio=1.0)
    p = SpindleKVPass(cfg, wl.seq_lens, hK.dtype, device=dev, layers_per_codebook_call=min(8, wl.n_layers))
    p.run(hK.to(dev), hV.to(dev), None)
    if p.device_status()["codebook"][0]:
        raise RuntimeError("device status in the CodeBook pass")
    n, d, e = wl.max_len, wl.head_dim, hK.element_size()
    att = SpindleKVDecodeAttention(p.cb_batch if p.cb_layers_per_call == wl.n_layers else B.Batch(wl.n_layers, wl.batch, n, wl.batch * n),
                                   wl.n_q_heads, wl.n_kv_heads, d, n + 64)
    g = torch.Generator(device="cpu").manual_seed(wl.seed)
    q = torch.randn((wl.n_layers, wl.batch, wl.n_q_heads, 1, d), generator=g).to(hK.dtype).to(dev)
    pos_q = torch.full((wl.batch,), n, dtype=torch.int32, device=dev)
    step, per_replay = recorded(lambda: att.run(q, pos_q, p.cb["K"], p.cb["V"]), dev)
    for _ in range(max(args.warmup, 3)):
        step()
    B.spindlekv_launch_count(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize(dev)
    ms = ev0.elapsed_time(ev1) / args.steps
    launches = B.spindlekv_launch_count(True) + per_replay * args.steps
    entries = int(p.cb["K"]["n_entries"].sum().item()) + int(p.cb["V"]["n_entries"].sum().item())
    units = wl.n_layers * wl.batch * wl.n_kv_heads
    alg = entries * d * e + units * n * 16                  # CodeBook rows once; reference and magnitude of K and of V per token
    dense = units * n * 2 * d * e
    pk, pk_src = peaks()
    line = {"metric": "decode steps/s over the replaced cache of all layers (Eq. 14, RoPE re-applied)", "value": 1e3 / ms, "unit": "steps/s",
            "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": workload_config(wl, {"cached_tokens_per_head": n, "query_heads_per_kv_head": wl.group}),
            "gpu_launches": int(launches),
            "roofline": {"kernel": "decode attention over CodeBooks", "bound": "hbm", "achieved": alg / (ms * 1e-3) / 1e9,
                         "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": alg / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], "traffic": None,
                         "peak_source": pk_src, "algorithmic_bytes": alg, "dense_cache_bytes": dense,
                         "codebook_entries_over_tokens": entries / (2.0 * units * n)}}
    print(json.dumps(line))


def sampled_gpu_decisions(wl, p, dK, dV, dtype, dev):
    """The GPU's adjacency of the CodeBook units and its kept positions of the evicting layer that the CPU-baseline
    leg runs the checker on (outside every timed region)."""
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200.pipeline import SpindleKVPass
    out = {"adj": {}, "keep": None}
    ns = wl.n_shallow
    if ns:
        l = wl.seq_lens[0]
        one = B.Config(n_layers=1, n_q_heads=1, n_kv_heads=1, head_dim=wl.head_dim, window=1, n_shallow=1,
                       budget_tokens=float(l), theta_k=wl.theta_k, theta_v=wl.theta_v)
        q = SpindleKVPass(one, [l], dtype, device=dev, keep_adjacency=True)
        for j in range(min(2, wl.n_kv_heads)):
            for name, src in (("K", dK), ("V", dV)):
                rows = (src[0, :l, j] if wl.packed else src[0, 0, j]).contiguous().reshape(1, 1, 1, l, wl.head_dim)
                q.codebook(rows, name)
                if q.device_status()["codebook"][0] != 0:
                    raise RuntimeError("device status in the sampled CodeBook unit")
                words = q.adj[0, :l].cpu().numpy().view(np.uint32)
                bits = np.unpackbits(words.view(np.uint8), axis=1, bitorder="little")[:, :l].astype(bool)
                out["adj"][(name, j)] = bits
        del q
    if wl.n_layers > ns:
        out["keep"] = p.keep_idx[0, :, : wl.seq_lens[0]].cpu().numpy()
    return out


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
    run_direct = lambda: p.run(dK, dV, dQ)
    # the timed steps replay one recorded pass (a CUDA graph: one launch from the host per step); direct calls where
    # recording is not possible, and for the per-kernel pass further down
    step, launches_per_replay = recorded(run_direct, dev)
    graph = step if step is not run_direct else None
    for _ in range(max(args.warmup, 3)):
        step()
    st = p.device_status()
    for k, v in st.items():
        if v[0] != 0:
            raise RuntimeError(f"device status {v} in {k}")
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.wait_until_sampling()
        for _ in range(3):   # the part is under load again when the timed region starts
            step()
    B.spindlekv_launch_count(True)
    t0 = time.perf_counter()
    ms = timed(step, args.steps)
    t1 = time.perf_counter()
    job_tokens = timed.tokens
    launches = B.spindlekv_launch_count(True) + launches_per_replay * args.steps
    clocks = sampler.stop(t0, t1) if sampler else None

    # the same steps once more, each with its own event pair: the median beside the mean
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in evs:
        a.record()
        step()
        b.record()
    barrier()
    per_step = sorted(a.elapsed_time(b) for a, b in evs)
    ms_median = sharding.aggregate(wl.total_tokens, statistics.median(per_step), dist, dev)[1]

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

    # per-kernel times: one more pass with event pairs around every launch, the three calls one after the other on
    # one stream (in the timed steps above they run side by side on three streams, where a kernel's span holds its
    # neighbours' time too)
    side = p.side_by_side
    p.side_by_side = False
    B.spindlekv_timing_enable(True)
    for _ in range(args.steps):
        run_direct()
    torch.cuda.synchronize(dev)
    kt = B.spindlekv_timing_read()
    B.spindlekv_timing_enable(False)
    p.side_by_side = side

    # counters of the CodeBook graph stage, per Gamma: the status block of a call holds its rounds, the units that went
    # through the bit matrix and the neighbour-list entries built from candidate records
    graph = {}
    if p.n_shallow:
        for g, src in (("K", dK), ("V", dV)):
            p.codebook(src[:p.n_shallow], g)
            stat, det = p.device_status()["codebook"]
            if stat != 0:
                raise RuntimeError(f"device status {stat} in the {g} CodeBook call")
            graph[g] = {"greedy_rounds": det[0], "units_through_bit_matrix": det[2], "list_entries": det[3]}

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
    if ns and graph:
        # Graph stage, bytes that must move at least once per step (K and V calls together).  List building: the
        # candidate records (8 bytes per similar pair, read), the lists (4 bytes per entry, written), and per token
        # degree, list start and length, pick degree and live bit (16 bytes, written).  Greedy cover (keys and
        # neighbourhood maxima live in shared memory): every list entry read once, per-token degree, list start and
        # length read, owner and pick degree written (20 bytes).  Numbering: pick degree, owner, rank, reference and
        # centre position per token (20 bytes).
        rows = 2 * ns * Hk * tok
        ent = sum(v["list_entries"] for v in graph.values())
        for name, nbytes in (("degree", ent // 2 * 8 + ent * 4 + rows * 16), ("greedy", ent * 4 + rows * 20),
                             ("finalise", rows * 20)):
            if name in kernels and kernels[name]["ms_per_step"] > 0:
                gbs = nbytes / (kernels[name]["ms_per_step"] * 1e-3) / 1e9
                kernels[name].update({"bound": "hbm (in fact: latency of dependent gathers; see profiles/)",
                                      "algorithmic_bytes": nbytes, "achieved_gbs": gbs, "frac_of_hbm_peak": gbs / pk["hbm_gbs"]})
        kernels["greedy"]["rounds"] = {g: v["greedy_rounds"] for g, v in graph.items()}
        kernels["degree"]["units_through_bit_matrix"] = {g: v["units_through_bit_matrix"] for g, v in graph.items()}
        kernels["degree"]["list_entries"] = {g: v["list_entries"] for g, v in graph.items()}
    roof = None
    if p.n_shallow and kt["similarity"][1]:
        sim_ms, sim_n = kt["similarity"]
        units_per_launch = 2 * wl.n_shallow * wl.n_kv_heads * wl.batch / (sim_n / args.steps)
        flops_per_step = sum(float(l) * (l - 1) * wl.head_dim for l in wl.seq_lens) * 2 * wl.n_shallow * wl.n_kv_heads
        achieved = flops_per_step * args.steps / (sim_ms * 1e-3) / 1e12
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        if wl.dtype == "bf16":
            bound, peak, peak_name = "tensor", pk["bf16_tflops_sustained"], "cuBLAS bf16 GEMM, sustained loop (MEASURED_PEAKS.json)"
        else:
            # fp32 inputs take the CUDA-core kernel: 128 fused multiply-adds per clock and SM, 148 SMs, sampled clock
            bound, peak, peak_name = "alu", 2.0 * 128 * 148 * mhz * 1e6 / 1e12, "fp32 FMA rate at the sampled SM clock"
        traffic = None
        if not wl.packed and wl.max_len in SIMILARITY_TRAFFIC_BYTES_PER_UNIT and wl.head_dim == 128:
            traffic = SIMILARITY_TRAFFIC_BYTES_PER_UNIT[wl.max_len] * units_per_launch
        roof = {"kernel": "similarity (Eq. 4, 9)", "bound": bound, "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": traffic, "peak_source": pk_src, "peak_is": peak_name,
                "avg_launch_ms": sim_ms / sim_n, "algorithmic_flops_per_launch": flops_per_step * args.steps / sim_n}
        if wl.dtype == "bf16":
            # the same achieved rate against the other denominators one may want: the cuBLAS burst figure, and the
            # tensor pipe itself at the clock sampled during the run (nominal 2250 TFLOP/s dense bf16 at 1965 MHz)
            roof["frac_of_cublas_sustained"] = achieved / pk["bf16_tflops_sustained"]
            roof["frac_of_cublas_burst"] = achieved / pk["bf16_tflops"]
            roof["frac_of_pipe_at_sampled_clock"] = achieved / (2250.0 * mhz / 1965.0)
            roof["executed_over_useful"] = 9.0 / 8.0   # one K-step in nine carries the threshold
    line = {"metric": METRIC, "value": sharding.throughput(job_tokens, args.steps, ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "ms_per_step_median": ms_median,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
            "data": "synthetic",
            "config": workload_config(wl, {"parallelism": f"replicas x{world}",
                                           "streams": "K CodeBooks, V CodeBooks and eviction side by side on three streams; "
                                                      "per-kernel times from a serial pass",
                                           "cuda_graph": graph is not None}),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roof, "kernels": kernels,
            "greedy_rounds": st.get("codebook", (0, [0]))[1][0]}
    if not args.no_cpu_baseline and world == 1:
        sec, cores, sample, margins = oracle_sample_seconds(wl, sampled_gpu_decisions(wl, p, dK, dV, dtype, dev))
        line["cpu_baseline"] = {"value": wl.total_tokens / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": sample}
        line["near_threshold"] = margins
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
    elif a.decode:
        run_decode(a, w)
    elif a.literal:
        run_literal(a, w)
    else:
        run_native(a, w)
