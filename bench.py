#!/usr/bin/env python
"""Benchmark of composed-cache query prefill (KV Packet serving path) on B200.

A *step* is one pass of the whole hot path over one batch: ``kvp_assemble`` (plan upload + staging
gather) followed by ``kvp_query_prefill`` for every layer, back to back on one stream.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

prints ONE JSON line.  ``value`` = query tokens/s of the whole job (batch * q_len tokens through the
full layer stack per step), inputs resident in HBM.  ``e2e`` = the same with the step's Q/K_new/V_new
coming from pinned host buffers and the outputs read back, copies inside the timed region.
``roofline`` is for the dominant kernel (the tcgen05 attention kernel), its duration measured live
with CUDA events on the launching stream; the fraction is given against the measured burst and sustained
bf16 GEMM peaks and the nominal one, with the rule that picks the headline.  ``extra_points`` add the
memory-bound short-query shape, the gather kernel in materialise mode, a decode step (one token per
request), one layer of config 4, config 2, a pruned-packet layer and host-resident packets, each with the
clock record of its own timed region.  ``cpu_baseline`` is the fp64 oracle on the host cores on a bounded
sample (three layers, about 10 s).  ``--impl reference`` times a smaller sample of the same kind once per step.  ``--shard prefix`` is the second
multi-GPU mode: the packets of one long-context batch split over the ranks, one all-gather of partial
results per layer.  ``--shard heads`` is the third: the kv heads of one batch split over the ranks, no exchange.

Workloads (seeded, synthetic, shaped like the paper's Llama-3.1-8B / Qwen2.5-7B RAG requests):
config3 (default; Llama-3.1-8B 32-layer stack, 10 x 1024-token packets, 128 query tokens, batch 4),
config2, config4, config5:<packets>:<q_len>:<batch>.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# NVIDIA's nominal B200 figures (dense bf16; HBM3e), for the "of nominal" fractions
NOMINAL_TFLOPS, NOMINAL_GBS, N_SMS = 2250.0, 8000.0, 148


def tensor_fractions(tflops: float, peaks, region_s: float, clocks):
    """One achieved bf16 rate against every denominator, and the headline fraction by a stated rule: the burst
    GEMM peak when the timed region is shorter than one second or the SM clock sampled during it stayed at
    >= 0.9 of its maximum (the conditions the burst peak was measured under), the sustained peak otherwise."""
    sm = (clocks or {}).get("sm_mhz")
    mx = (clocks or {}).get("sm_max_mhz")
    burst = region_s < 1.0 or (sm is not None and mx and sm >= 0.9 * mx)
    out = {"frac_burst": tflops / peaks["bf16_tflops"], "frac_sustained": tflops / peaks["bf16_tflops_sustained"],
           "frac_nominal": tflops / NOMINAL_TFLOPS,
           "peak_burst": peaks["bf16_tflops"], "peak_sustained": peaks["bf16_tflops_sustained"], "peak_nominal": NOMINAL_TFLOPS,
           "headline_peak": "burst" if burst else "sustained",
           "headline_rule": "burst if timed region < 1 s or median SM clock >= 0.9 max, else sustained",
           "rule_inputs": {"timed_region_s": region_s, "sm_mhz_median": sm, "sm_max_mhz": mx}}
    if sm:
        # clock-normalised: flop per SM cycle (the tensor pipe's ceiling is 8192 dense bf16 flop per SM cycle)
        out["flop_per_sm_cycle"] = tflops * 1e12 / (sm * 1e6 * N_SMS)
    return out, (peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"])


def make_spec(name: str, seed: int):
    from paper_2604_13226_b200 import inputs as gen
    if name == "config3":
        return gen.spec_config3(seed=seed)
    if name.startswith("config3:"):                  # the same requests over fewer layers (small profiler captures)
        s = gen.spec_config3(seed=seed, n_layers=int(name.split(":")[1]))
        s.name = name.replace(":", "_layers")
        return s
    if name == "config4":
        return gen.spec_config4(seed=seed)
    if name == "config4_layer":                      # one layer of the Qwen2.5-7B stack: same requests, same raggedness
        s = gen.spec_config4(seed=seed, n_layers=1)
        s.name = "config4_layer"
        return s
    if name == "config2":
        s = gen.spec_config3(seed=seed, n_layers=1, batch=1, pool=5, per_item=5, doc_len=512, q_len=64)
        s.name = "config2"
        return s
    if name.startswith("config5"):
        _, n, q, b = name.split(":")
        return gen.spec_config5(int(n), int(q), int(b), seed=seed)
    raise SystemExit(f"unknown workload {name}")


def algorithmic_work(spec):
    """Per layer: flops = 4 d Hq Lq (P + (Lq+1)/2) per request; bytes = prefix K,V once + Q, O, K_new,
    V_new read once and the appended rows written once (every byte the step must move, moved once)."""
    s = spec.shape
    d, Hq, Hkv, e, Lq = s.head_dim, s.n_q_heads, s.n_kv_heads, s.elem_bytes, spec.q_len
    flops = bytes_ = 0.0
    for b in range(spec.batch):
        P = spec.prefix_len(b)
        flops += 4.0 * d * Hq * Lq * (P + (Lq + 1) / 2.0)
        bytes_ += 2.0 * Hkv * d * e * P + (2.0 * Hq + 4.0 * Hkv) * d * e * Lq
    return flops, bytes_


# ---------------------------------------------------------------------------------------------------
# multi-GPU: requests are sharded across ranks (every rank composes and prefills its own batch); the only
# exchange is the barrier and the max-over-ranks of the timings
# ---------------------------------------------------------------------------------------------------

def rank_spec(workload: str, seed: int, rank: int):
    """The batch rank `rank` works on: same shape, its own seeded draw of packets and requests (weak scaling)."""
    return make_spec(workload, seed + 17 * rank)


def max_over_ranks(values, world: int, device=None):
    """Element-wise maximum of `values` (list of floats) over all ranks of the default process group."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def head_spec(workload: str, seed: int, rank: int, world: int):
    """`--shard heads`: rank `rank` holds kv heads [rank Hkv / world, (rank + 1) Hkv / world) of every packet of the
    SAME batch, and the query heads that read them (strong scaling; attention is independent per kv head, so there is
    no exchange inside the path - the ranks' outputs are the head slices of the output)."""
    from paper_2604_13226_b200 import inputs as gen
    return gen.shard_heads_spec(make_spec(workload, seed), rank, world)


def job_tokens_per_s(spec, world: int, ms_step: float, shard: str = "requests") -> float:
    """Whole-job rate: with requests sharded every rank pushes its own batch * q_len query tokens through the stack
    per step; with heads sharded all ranks work on the same batch * q_len tokens."""
    return spec.batch * spec.q_len * (world if shard == "requests" else 1) / (ms_step * 1e-3)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples, every 20 ms, taken for as long as the sampler runs; every
    sample carries nvidia-smi's own timestamp, so any timed region gets the record of exactly its samples."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_ms: int = 20):
        self.index, self.period_ms = index, period_ms
        self.proc = None
        self.samples = []                      # (epoch seconds, sm MHz, max MHz, watts, set of active reasons)
        self._thread = None

    def _read(self):
        import datetime
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                t = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.samples.append((t, float(f[1]), float(f[2]), float(f[3]),
                                     {n for n, v in zip(self.NAMES, f[4:8]) if v.lower().startswith("active")}))
            except ValueError:
                continue

    def start(self):
        import threading
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
            self._thread = threading.Thread(target=self._read, daemon=True)
            self._thread.start()
        except Exception:
            self.proc = None

    @staticmethod
    def now() -> float:
        return time.time()

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        if self._thread is not None:
            self._thread.join(timeout=5)

    def window(self, t0: float, t1: float):
        """Record of the samples stamped inside [t0, t1] (widened to the nearest sample on either side when the
        region is shorter than the sampling period)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(3 * self.period_ms / 1000.0)           # let the samples of the region's end arrive
        inside = [x for x in self.samples if t0 <= x[0] <= t1]
        if len(inside) < 2:
            mid = 0.5 * (t0 + t1)
            inside = sorted(self.samples, key=lambda x: abs(x[0] - mid))[:2]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"], "samples": 0}
        reasons = set()
        for x in inside:
            reasons |= x[4]
        return {"sm_mhz": statistics.median(x[1] for x in inside), "sm_mhz_min": min(x[1] for x in inside),
                "sm_max_mhz": max(x[2] for x in inside), "power_w_max": max(x[3] for x in inside),
                "reasons": sorted(reasons), "samples": len(inside), "period_ms": self.period_ms}


# ---------------------------------------------------------------------------------------------------
# oracle timing (cpu_baseline leg and the --impl reference arm)
# ---------------------------------------------------------------------------------------------------

ORACLE_TOKENS = 32          # query tokens per request the oracle is timed on (evenly spaced over the chunk)
BASELINE_TOKENS = 64        # the same for the `cpu_baseline` object, which also takes three layers (about 10 s of CPU work)


def oracle_sample(spec, wl, n_tokens: int = ORACLE_TOKENS, layers=(0,)):
    """Time the fp64 oracle, as it stands, on the given layers of every request: composition + re-basing of the whole
    prefix and the widening / concatenation of its inputs (a fixed cost per request and layer), then attention
    for every head of `n_tokens` query tokens spread evenly over the chunk (0 = all).  Only the attention time is
    scaled to the full chunk (work per row is the same to within q_len / prefix), and the mean over the sampled
    layers to the stack.  Returns the job-level rate it implies: query tokens/s through the full stack =
    batch*q_len / (L * mean_l sum_b t_b).  The reference arm times the default sample once per step; `cpu_baseline`
    times a larger one (first, middle and last layer, twice the tokens)."""
    from oracle import reference as orc
    from paper_2604_13226_b200 import inputs as gen
    s = spec.shape
    ad = wl.adapter_host()
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    toks = list(range(spec.q_len))
    if 0 < n_tokens < spec.q_len:
        toks = sorted({int(round(i * (spec.q_len - 1) / (n_tokens - 1))) for i in range(n_tokens)}) if n_tokens > 1 else [spec.q_len - 1]
    rows = [(h, i) for i in toks for h in range(s.n_q_heads)]
    layers = sorted({min(max(int(l), 0), s.n_layers - 1) for l in layers})
    t_total = t_fixed = t_att = 0.0
    digests = None
    for layer in layers:
        q, kn, vn = wl.query_layer(layer)
        # pull the bytes to the host before timing (the oracle's inputs are host arrays)
        cached = {}
        for it in spec.items:
            for pid, _ in it:
                if pid not in cached:
                    cached[pid] = wl.packet_layer(pid, layer)
        st = orc.Store(s.dtype)
        for pid, n in enumerate(spec.packet_lens):
            st.register_packet(n, 0, (lambda l_, pid=pid: cached[pid]))
        st.register_adapter(ad.n_header, 0, ad.n_trailer, 0,
                            (lambda l_, layer=layer: (ad.hk[layer], ad.hv[layer], ad.tk[layer], ad.tv[layer])))
        if digests is None:
            pids = sorted(cached)
            digests = {"algorithm": "blake2b-64 over the raw bytes, layer %d" % layer,
                       "q": gen.digest64(q), "k_new": gen.digest64(kn), "v_new": gen.digest64(vn),
                       "packets_k": gen.digest64(*[cached[p][0] for p in pids]),
                       "packets_v": gen.digest64(*[cached[p][1] for p in pids]),
                       "adapter": gen.digest64(ad.hk[layer], ad.hv[layer], ad.tk[layer], ad.tv[layer]), "packets": len(pids)}
        for b in range(spec.batch):
            t0 = time.perf_counter()
            plan = orc.compose(st, spec.items[b], spec.rebase)
            Kp, Vp, _ = orc.composed_kv(st, plan, layer, f, s.rope_pairing)
            Q = orc.widen(q[b], s.dtype)
            K = np.concatenate([Kp, orc.widen(kn[b], s.dtype)])
            V = np.concatenate([Vp, orc.widen(vn[b], s.dtype)])
            t1 = time.perf_counter()
            orc.attention_rows(K, V, Q, plan.prefix_len, 1.0 / np.sqrt(s.head_dim), rows)
            t2 = time.perf_counter()
            t_fixed += t1 - t0
            t_att += t2 - t1
            t_total += (t1 - t0) + (t2 - t1) / len(rows) * (spec.q_len * s.n_q_heads)
    tokens_per_s = spec.batch * spec.q_len / (s.n_layers * t_total / len(layers))
    return {"value": tokens_per_s, "unit": "tokens/s", "cores": orc.threads(), "kind": "oracle",
            "sample": f"layer{'s' if len(layers) > 1 else ''} {', '.join(str(l) for l in layers)} of all {spec.batch} requests: compose + "
                      f"re-base + widening of the prefix ({t_fixed:.2f} s) and attention rows of {len(toks)} of {spec.q_len} query "
                      f"tokens x {s.n_q_heads} heads ({t_att:.2f} s); attention scaled to {spec.q_len} tokens, the mean over the "
                      f"sampled layers to {s.n_layers} layers",
            "seconds": t_fixed + t_att, "input_digests": digests}


def baseline_sample(spec, wl):
    """The `cpu_baseline` object: the oracle on the first, middle and last layer, BASELINE_TOKENS query tokens each."""
    L = spec.shape.n_layers
    return oracle_sample(spec, wl, n_tokens=BASELINE_TOKENS, layers=(0, L // 2, L - 1))


def prefill_flags(spec) -> int:
    """Workloads with x8 outlier channels are run the way their parity test runs them: KVP_PRECISE_QK."""
    from paper_2604_13226_b200 import binding as kvp
    return kvp.PRECISE_QK if getattr(spec, "outlier_channels", 0) else 0


def workload_config(spec, materialize: bool, bytes_per_layer: float, shard: str = "requests", world: int = 1):
    """The `config` object of the JSON line: the workload, named the same way by both arms."""
    s = spec.shape
    sharding = "requests sharded across ranks, no collective"
    if shard == "heads":
        sharding = ("kv heads sharded across ranks (%d of %d kv heads and their %d query heads per GPU, the same batch on "
                    "every rank), no collective" % (s.n_kv_heads, s.n_kv_heads * world, s.n_q_heads))
    return {"workload": spec.name, "layers": s.n_layers, "q_heads": s.n_q_heads, "kv_heads": s.n_kv_heads,
            "head_dim": s.head_dim, "batch_per_gpu": spec.batch, "q_len": spec.q_len,
            "prefix_tokens": [spec.prefix_len(b) for b in range(spec.batch)], "rope_theta": s.rope_theta,
            "mode": "materialised cache" if materialize else "fused in place (adapters staged)",
            "qk": "precise (KVP_PRECISE_QK)" if prefill_flags(spec) else "plain",
            "l2": "inputs larger than L2: every layer reads %.0f MB of distinct K/V" % (bytes_per_layer / 1e6),
            "sharding": sharding}


# ---------------------------------------------------------------------------------------------------
# extra roofline points (memory-bound shape, gather kernel)
# ---------------------------------------------------------------------------------------------------

def flush_l2(torch, dev, buf=[None]):
    if buf[0] is None:
        buf[0] = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    buf[0].zero_()


def point_fractions(res, flops, bytes_, ms, peaks, clocks, region_s):
    """Rates of one timed kernel against the measured (burst / sustained) and nominal peaks."""
    tf = flops / ms / 1e9
    fr, _ = tensor_fractions(tf, peaks, region_s, clocks)
    res.update({"frac_tensor_burst": fr["frac_burst"], "frac_tensor_sustained": fr["frac_sustained"],
                "frac_tensor_nominal": fr["frac_nominal"], "flop_per_sm_cycle": fr.get("flop_per_sm_cycle"),
                "frac_hbm": bytes_ / ms / 1e6 / peaks["hbm_gbs"], "frac_hbm_nominal": bytes_ / ms / 1e6 / NOMINAL_GBS,
                "clocks": clocks})


def measure_point(spec_name: str, seed: int, iters: int, materialize: bool, peaks, device: int, sampler=None):
    """ms of one layer's attention kernel (CUDA events inside the library) and of the gather kernel."""
    import torch
    from paper_2604_13226_b200 import binding as kvp, inputs as gen
    from paper_2604_13226_b200.session import Session
    spec = make_spec(spec_name, seed)
    wl = gen.DeviceWorkload(spec, f"cuda:{device}")
    sess = Session(wl, materialize=materialize, device=device)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 1)
    dev = torch.device(f"cuda:{device}")
    qkv = sess.query_tensors(0)
    flags = prefill_flags(spec)
    att, gat = [], []
    t0 = ClockSampler.now()
    for it in range(iters + 3):
        flush_l2(torch, dev)
        sess.assemble()
        flush_l2(torch, dev)
        sess.prefill(0, flags, qkv=qkv, want_lse=False)
        torch.cuda.synchronize(dev)
        a, g = sess.ctx.kernel_times(0), sess.ctx.kernel_times(1)
        if it >= 3:
            att += a
            gat += g
    clocks = sampler.window(t0, ClockSampler.now()) if sampler is not None else None
    launch = sess.ctx.last_launch()
    assert sess.ctx.status_word() == 0
    flops, bytes_ = algorithmic_work(spec)
    s = spec.shape
    tok_bytes = 2.0 * s.n_kv_heads * s.head_dim * s.elem_bytes
    if materialize:
        moved = sum(spec.prefix_len(b) for b in range(spec.batch))
    else:
        moved = sum(spec.prefix_len(b) - sum(spec.packet_lens[p] for p, _ in spec.items[b]) for b in range(spec.batch))
    gather_bytes = 2.0 * moved * tok_bytes * s.n_layers           # read + write, all layers
    ms_a = statistics.median(att)
    ms_g = statistics.median(gat) if gat else None
    sess.close()
    del sess, wl
    torch.cuda.empty_cache()
    res = {"workload": spec.name, "attn_ms": ms_a, "attn_tflops": flops / ms_a / 1e9, "attn_gbs": bytes_ / ms_a / 1e6,
           "launch": launch, "l2": "flushed between iterations", "qk": "precise (KVP_PRECISE_QK)" if flags else "plain"}
    point_fractions(res, flops, bytes_, ms_a, peaks, clocks, ms_a * 1e-3)      # launches timed one at a time: burst conditions
    if ms_g:
        res.update({"gather_ms": ms_g, "gather_gbs": gather_bytes / ms_g / 1e6,
                    "gather_frac_hbm": gather_bytes / ms_g / 1e6 / peaks["hbm_gbs"], "gather_bytes": gather_bytes})
    return res


def measure_compressed_point(seed: int, iters: int, peaks, device: int, keep: float = 0.5, sampler=None):
    """One layer of the config-3 shape (4 requests x 10 x 1024-token packets, 128 query tokens) with every
    document pruned to about `keep` of its tokens, a different subset per kv head: attention kernel time,
    and the rates counted on the keys that are actually held."""
    import torch
    from paper_2604_13226_b200 import binding as kvp, inputs as gen
    from paper_2604_13226_b200.session import Session
    shape = gen.ModelShape(1, 32, 8, 128, "bf16", 500000.0, 0)
    items = [[(10 * b + i, 0) for i in range(10)] for b in range(4)]
    wl = gen.make_workload(shape, [1024] * 40, items, q_len=128, seed=seed, keep_rate=[keep] * 40)
    sess = Session(wl, device=device)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 1)
    dev = torch.device(f"cuda:{device}")
    sess.assemble()
    qkv = sess.query_tensors(0)
    att = []
    t0 = ClockSampler.now()
    for it in range(iters + 3):
        flush_l2(torch, dev)
        sess.prefill(0, qkv=qkv, want_lse=False)
        torch.cuda.synchronize(dev)
        a = sess.ctx.kernel_times(0)
        if it >= 3:
            att += a
    clocks = sampler.window(t0, ClockSampler.now()) if sampler is not None else None
    assert sess.ctx.status_word() == 0
    launch = sess.ctx.last_launch()
    d, g, Lq = shape.head_dim, shape.group, 128
    flops = bytes_ = 0.0
    held = total = 0
    for b in range(4):
        for hk in range(shape.n_kv_heads):
            keys = 10 * 32 + sum(len(wl.packets[pid].kept[0][hk]) for pid, _ in items[b])
            held += keys - 320
            total += 10 * 1024
            flops += 4.0 * d * g * Lq * (keys + (Lq + 1) / 2.0)
            bytes_ += 2.0 * d * 2 * keys
    ms = statistics.median(att)
    sess.close()
    del sess, wl
    torch.cuda.empty_cache()
    res = {"workload": "config3 shape, one layer, documents pruned per kv head", "kept_fraction": held / total, "attn_ms": ms,
           "attn_tflops_on_held_keys": flops / ms / 1e9, "attn_gbs_on_held_keys": bytes_ / ms / 1e6, "launch": launch,
           "l2": "flushed between iterations"}
    point_fractions(res, flops, bytes_, ms, peaks, clocks, ms * 1e-3)
    return res


def measure_host_packets_point(seed: int, iters: int, device: int, n_layers: int = 8):
    """Config-3 shape with `n_layers` layers and every packet waiting in pinned host memory: one request batch from
    `kvp_assemble` (which starts the host-to-pool copies, layer by layer) to the last layer's attention, against the
    same step with the packets resident and against the bare copy time.  The attention of layer l overlaps the copy
    of the layers after it; the link decides the total."""
    import torch
    from paper_2604_13226_b200 import inputs as gen
    from paper_2604_13226_b200.session import Session
    spec = gen.spec_config3(seed=seed, n_layers=n_layers)
    wl = gen.DeviceWorkload(spec, f"cuda:{device}")
    dev = torch.device(f"cuda:{device}")
    sess = Session(wl, device=device, host_packets=True)
    qkv = [sess.query_tensors(l) for l in range(n_layers)]
    n_packets = len(spec.packet_lens)
    used = sorted({pid for item in wl.items for pid, _ in item})          # only the packets a request names are copied
    h2d = sum(sess.host_kv[pid][0].numel() * sess.host_kv[pid][0].element_size() * 2 for pid in used)

    def step(evict):
        if evict:
            for pid in range(n_packets):
                sess.ctx.evict_packet(pid)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sess.assemble()
        for l in range(n_layers):
            sess.prefill(l, qkv=qkv[l], want_lse=False)
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1)

    step(True)
    cold = statistics.median(step(True) for _ in range(iters))
    warm = statistics.median(step(False) for _ in range(iters))
    # the bare transfer: the same pinned buffers to a device buffer of the same size
    sink = [(torch.empty_like(hk, device=dev), torch.empty_like(hv, device=dev)) for hk, hv in sess.host_kv[:4]]
    torch.cuda.synchronize(dev)
    ts = []
    for _ in range(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for (dk, dv), (hk, hv) in zip(sink, sess.host_kv[:4]):
            dk.copy_(hk, non_blocking=True)
            dv.copy_(hv, non_blocking=True)
        e1.record()
        torch.cuda.synchronize(dev)
        ts.append(e0.elapsed_time(e1))
    link_gbs = sum(hk.numel() * hk.element_size() * 2 for hk, _ in sess.host_kv[:4]) / statistics.median(ts) / 1e6
    assert sess.ctx.status_word() == 0
    sess.close()
    del sess, wl, sink
    torch.cuda.empty_cache()
    return {"workload": f"config3 shape, {n_layers} layers, packets in pinned host memory", "h2d_bytes": h2d,
            "assemble_to_last_layer_ms": cold, "h2d_gbs_inside_it": h2d / cold / 1e6, "plain_copy_gbs": link_gbs,
            "same_step_packets_resident_ms": warm}


# ---------------------------------------------------------------------------------------------------
# second scaling mode: prefix sharding (the packets of every request spread over the ranks)
# ---------------------------------------------------------------------------------------------------

def run_prefix_shard(args, rank: int, world: int, local_rank: int, peaks):
    """`--shard prefix`: strong scaling of one long-context batch.  Rank r holds packets [r n/N, (r+1) n/N) of every
    request (`kvp_assemble_at` re-bases them to their positions in the whole request), attends to them with
    KVP_PARTIAL (the last rank also takes the query's own keys), the partial (O, m, l) buffers are all-gathered into
    local memory over NCCL - the path's one exchange - and every rank merges them (`kvp_merge_partials`).  No kernel
    is given a peer's memory."""
    import torch
    from paper_2604_13226_b200 import binding as kvp, inputs as gen
    from paper_2604_13226_b200.session import Session
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    name = args.workload if args.workload.startswith("config5") else "config5:64:16:1"
    _, n, ql, b = name.split(":")
    n, ql, b = int(n), int(ql), int(b)
    if n % world:
        raise SystemExit(f"--shard prefix: {n} packets per request do not divide over {world} ranks")
    per_rank = n // world
    whole = gen.spec_config5(n, ql, b, seed=args.seed)
    # this rank's packets; with one request they are the whole workload's own bytes, else the rank's own draws
    spec = gen.shard_spec(whole, rank, world)[0] if b == 1 else gen.spec_config5(per_rank, ql, b, seed=args.seed + 17 * rank)
    doc = spec.packet_lens[0] + spec.n_header + spec.n_trailer
    pos_base = [rank * per_rank * doc] * b
    s = spec.shape
    wl = gen.DeviceWorkload(spec, f"cuda:{local_rank}")
    sess = Session(wl, device=local_rank)
    L = s.n_layers
    # the query is the same on every rank: drawn from the whole request's seed
    qkv = [gen.DeviceWorkload(whole, f"cuda:{local_rank}").query_device(l) for l in range(L)]
    part_bytes = sess.ctx.partial_bytes(b, ql)
    part = torch.empty(part_bytes, dtype=torch.uint8, device=dev)
    gathered = torch.empty(part_bytes * world, dtype=torch.uint8, device=dev) if world > 1 else part
    outs = [torch.empty_like(qkv[l][0]) for l in range(L)]
    flags = kvp.PARTIAL | (0 if rank == world - 1 else kvp.SKIP_QUERY_BLOCK)

    def layer(l, q, kn, vn, out):
        sess.ctx.query_prefill(sess.assembly_id, l, q, kn, vn, ql, part, None, flags)
        if world > 1:
            dist.all_gather_into_tensor(gathered, part)                        # NCCL, into this GPU's own memory
        sess.ctx.merge_partials(gathered, world, b, ql, out, None)

    def step():
        sess.assemble(pos_base=pos_base)
        for l in range(L):
            layer(l, *qkv[l], outs[l])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    launches_per_step = 1 + L * (sess.ctx.last_launch()["launches"] + 1)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 1)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)
    def timed(fn):
        """K steps, each bracketed by a barrier + synchronize and timed with its own event pair; L2 is flushed
        between them, outside the timed parts (a rank's share of the keys can be smaller than L2)."""
        total = 0.0
        for _ in range(args.steps):
            flush_l2(torch, dev)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            barrier()
            total += e0.elapsed_time(e1)
        return total

    t0 = ClockSampler.now()
    ms_total = timed(step)
    clocks = sampler.window(t0, ClockSampler.now()) if rank == 0 else None
    sampler.stop()
    attn_ms = sess.ctx.kernel_times(0)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 0)
    assert sess.ctx.status_word() == 0
    # end to end: the query chunk comes from pinned host memory and the output goes back, inside the timed region
    hq = [tuple(t.cpu().pin_memory() for t in qkv[l]) for l in range(L)]
    hout = [torch.empty_like(outs[l], device="cpu").pin_memory() for l in range(L)]
    dq = tuple(torch.empty_like(t) for t in qkv[0])
    dout = torch.empty_like(outs[0])

    def step_e2e():
        sess.assemble(pos_base=pos_base)
        for l in range(L):
            for dst, src in zip(dq, hq[l]):
                dst.copy_(src, non_blocking=True)
            layer(l, *dq, dout)
            hout[l].copy_(dout, non_blocking=True)

    for _ in range(3):
        step_e2e()
    ms_e2e = timed(step_e2e)
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], world, dev)
    h2d = sum(t.numel() * t.element_size() for t in hq[0]) * L
    d2h = hout[0].numel() * hout[0].element_size() * L
    sess.close()
    if rank == 0:
        ms_step = ms_total / args.steps
        flops, bytes_ = algorithmic_work(spec)                                 # this rank's share of the keys
        a_ms = statistics.mean(attn_ms) if attn_ms else None
        roof = None
        if a_ms:
            ach = bytes_ / a_ms / 1e6
            roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                    "frac_nominal": ach / NOMINAL_GBS, "peak_nominal": NOMINAL_GBS, "traffic": None, "peak_source": peaks["source"],
                    "kernel": "attn_sm100_kernel (one rank's keys)", "launches_timed": len(attn_ms), "avg_launch_ms": a_ms,
                    "algorithmic_bytes_per_launch": bytes_, "algorithmic_flops_per_launch": flops}
        cfg = workload_config(whole, False, bytes_)
        cfg.update({"sharding": "prefix: the packets of every request split over the ranks; per layer one all-gather of "
                                "(O, m, l) partials into local memory and a log-sum-exp merge",
                    "packets_per_rank": per_rank, "exchange_bytes_per_rank_per_layer": part_bytes,
                    "l2": "L2 flushed between steps, outside the timed parts (every step has its own event pair)"})
        print(json.dumps({
            "metric": "composed_cache_prefill_query_tokens_per_s", "value": b * ql / (ms_step * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
            "e2e": {"value": b * ql / (ms_e2e / args.steps * 1e-3), "unit": "tokens/s", "ms_per_step": ms_e2e / args.steps,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps, "roofline": roof, "clocks": clocks}))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------------
# main
# ---------------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config3")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-extras", action="store_true", help="skip the extra roofline points and the CPU baseline")
    ap.add_argument("--materialize", action="store_true", help="materialise the composed prefix instead of reading in place")
    ap.add_argument("--shard", default="requests", choices=["requests", "prefix", "heads"],
                    help="requests: every rank its own batch (weak scaling, the default); prefix: the packets of one "
                         "long-context batch (config5:<packets>:<q_len>:<batch>) split over the ranks (strong scaling); "
                         "heads: the kv heads of one batch split over the ranks, no exchange (strong scaling)")
    ap.add_argument("--sweep", action="store_true",
                    help="time the attention kernel over the config-5 grid (packets x q_len x batch) and print one JSON line per point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    peaks = load_peaks()

    import torch
    from paper_2604_13226_b200 import inputs as gen

    if args.sweep:
        if rank != 0:
            return
        assert torch.cuda.is_available(), "bench.py needs a CUDA device"
        sweep_sampler = ClockSampler(local_rank)
        sweep_sampler.start()
        for n in (2, 4, 8, 16, 32, 64):
            for ql in (16, 64, 256, 1024):
                for b in (1, 4, 16):
                    r = measure_point(f"config5:{n}:{ql}:{b}", args.seed, 5, False, peaks, local_rank, sweep_sampler)
                    r.pop("gather_ms", None); r.pop("gather_gbs", None); r.pop("gather_frac_hbm", None); r.pop("gather_bytes", None)
                    r.update({"packets": n, "q_len": ql, "batch": b, "bound": "tensor" if 4 * ql >= 247 else "hbm"})
                    print(json.dumps(r), flush=True)
        sweep_sampler.stop()
        return

    if args.impl == "reference":
        if rank != 0:
            return
        spec = make_spec(args.workload, args.seed)
        dev = "cuda:0" if torch.cuda.is_available() else None
        if dev is None:
            print(json.dumps({"impl": "reference", "unavailable": "the seeded workload generator needs a CUDA device"}))
            return
        wl = gen.DeviceWorkload(spec, dev)
        for _ in range(args.warmup):
            oracle_sample(spec, wl, n_tokens=1)
        t0 = time.perf_counter()
        vals = [oracle_sample(spec, wl) for _ in range(max(1, args.steps))]      # one bounded sample per step
        dt = time.perf_counter() - t0
        v = statistics.median(x["value"] for x in vals)
        cb = dict(vals[-1])
        cb["value"] = v
        _, bytes_ = algorithmic_work(spec)
        cfg = workload_config(spec, args.materialize, bytes_)                    # the same object the repo arm prints
        print(json.dumps({
            "impl": "reference", "metric": "composed_cache_prefill_query_tokens_per_s", "value": v, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": spec.batch * spec.q_len / v * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
            "cpu_baseline": cb, "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": dt,
            "note": "each step = a bounded sample of the workload run through the CPU oracle on the host cores"}))
        return

    if args.shard == "prefix":
        run_prefix_shard(args, rank, world, local_rank, peaks)
        return

    # ---- our arm ---------------------------------------------------------------------------------
    from paper_2604_13226_b200 import binding as kvp
    from paper_2604_13226_b200.session import Session
    kvp.lib()                                                    # fail loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    by_heads = args.shard == "heads"
    # weak scaling: every rank its own batch; or strong scaling over the kv heads of one batch
    spec = head_spec(args.workload, args.seed, rank, world) if by_heads else rank_spec(args.workload, args.seed, rank)
    s = spec.shape
    wl = gen.DeviceWorkload(spec, f"cuda:{local_rank}")
    sess = Session(wl, materialize=args.materialize, device=local_rank)
    L = s.n_layers
    qkv = [sess.query_tensors(l) for l in range(L)]
    outs = [torch.empty_like(qkv[l][0]) for l in range(L)]
    Lq = spec.q_len

    def step():
        sess.assemble()
        for l in range(L):
            q, kn, vn = qkv[l]
            sess.ctx.query_prefill(sess.assembly_id, l, q, kn, vn, Lq, outs[l], None, pf_flags)

    pf_flags = prefill_flags(spec)
    for _ in range(args.warmup):
        step()
    barrier()
    launches_per_step = 1 + L * sess.ctx.last_launch()["launches"]
    # every fifth attention (and gather) launch is bracketed by events: the period is coprime to the layer count, so
    # every layer is sampled, and the events cost the step less than bracketing every launch did (3 %)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 5)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_region0 = ClockSampler.now()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    clocks = sampler.window(t_region0, ClockSampler.now()) if rank == 0 else None
    ms_total = ev0.elapsed_time(ev1)
    attn_ms = sess.ctx.kernel_times(0)
    gather_ms = sess.ctx.kernel_times(1)
    sess.ctx.tune(kvp.TUNE_TIME_KERNELS, 0)
    status = sess.ctx.status_word()
    assert status == 0, f"device status word {status}"
    launch = sess.ctx.last_launch()

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ------------
    hq = [tuple(t.cpu().pin_memory() for t in qkv[l]) for l in range(L)]
    hout = [torch.empty_like(outs[l], device="cpu").pin_memory() for l in range(L)]
    # Two device buffers per tensor and three streams (host->device, compute, device->host): the copies of layer
    # l+1 and l-1 run while layer l computes, as a serving stack would drive the library through its stream argument.
    dq = [tuple(torch.empty_like(t) for t in qkv[0]) for _ in range(2)]
    dout = [torch.empty_like(outs[0]) for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in hq[0]) * L
    d2h = hout[0].numel() * hout[0].element_size() * L
    s_in, s_run, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_run = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def step_e2e():
        with torch.cuda.stream(s_run):
            sess.assemble()
        for l in range(L):
            k = l & 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_run[k])                     # the layer that last read this buffer is done
                for dst, src in zip(dq[k], hq[l]):
                    dst.copy_(src, non_blocking=True)
                ev_in[k].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[k])
                s_run.wait_event(ev_out[k])                    # its previous result has left the device
                sess.ctx.query_prefill(sess.assembly_id, l, dq[k][0], dq[k][1], dq[k][2], Lq, dout[k], None, pf_flags)
                ev_run[k].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[k])
                hout[l].copy_(dout[k], non_blocking=True)
                ev_out[k].record(s_out)

    def join():
        cur = torch.cuda.current_stream(dev)
        for st in (s_in, s_run, s_out):
            cur.wait_stream(st)

    def fork():
        cur = torch.cuda.current_stream(dev)
        for st in (s_in, s_run, s_out):
            st.wait_stream(cur)

    fork()
    for _ in range(3):
        step_e2e()
    join()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fork()
    for _ in range(args.steps):
        step_e2e()
    join()
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    # the results that came back are the ones the device-resident run produced
    assert torch.equal(hout[L - 1].to(dev), outs[L - 1]), "end-to-end output differs from the device-resident run"

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], world, dev)

    sess.close()
    del sess
    torch.cuda.empty_cache()

    if rank == 0:
        tokens = spec.batch * Lq * (1 if by_heads else world)
        ms_step = ms_total / args.steps
        value = job_tokens_per_s(spec, world, ms_step, args.shard)
        flops, bytes_ = algorithmic_work(spec)
        a_ms = statistics.mean(attn_ms) if attn_ms else None
        tensor_bound = s.group * Lq >= 247
        traffic = None
        tpath = os.path.join(ROOT, "profiles", "roofline_traffic.json")
        if os.path.exists(tpath):
            traffic = None if (by_heads and world > 1) else json.load(open(tpath)).get(spec.name)   # counters: all heads on one GPU
        if a_ms:
            if tensor_bound:
                ach = flops / a_ms / 1e9
                fr, peak = tensor_fractions(ach, peaks, ms_total * 1e-3, clocks)
                roof = {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                        "traffic": traffic, "peak_source": peaks["source"] + " (%s bf16 GEMM)" % fr["headline_peak"]}
                roof.update(fr)
            else:
                ach = bytes_ / a_ms / 1e6
                roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL_GBS, "peak_nominal": NOMINAL_GBS,
                        "traffic": traffic, "peak_source": peaks["source"]}
            roof.update({"kernel": "attn_sm100_kernel", "launches_timed": len(attn_ms), "avg_launch_ms": a_ms,
                         "algorithmic_flops_per_launch": flops, "algorithmic_bytes_per_launch": bytes_,
                         "attn_share_of_step": a_ms * L * args.steps / ms_total,     # every launch counted at the sampled mean
                         "gather_avg_ms": statistics.mean(gather_ms) if gather_ms else None})
        else:
            roof = None
        line = {
            "metric": "composed_cache_prefill_query_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "strong" if by_heads else "weak", "vs_baseline": None,
            "dtype": "bf16" if s.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": workload_config(spec, args.materialize, bytes_, args.shard, world),
            "prefix_tokens_per_s": sum(spec.prefix_len(b) for b in range(spec.batch)) * (1 if by_heads else world) / (ms_step * 1e-3),
            "e2e": {"value": tokens / (ms_e2e / args.steps * 1e-3), "unit": "tokens/s", "ms_per_step": ms_e2e / args.steps,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps, "launch": launch, "roofline": roof, "clocks": clocks,
        }
        if not args.no_extras and world == 1:
            extras = {}
            try:
                extras["hbm_bound_point"] = measure_point("config5:64:16:1", args.seed, 10, False, peaks, local_rank, sampler)
                extras["gather_materialise_point"] = measure_point("config5:16:64:1", args.seed, 10, True, peaks, local_rank, sampler)
                # the step after the prefill: one new token per request over 16 x 33,280-token composed caches
                extras["decode_point"] = measure_point("config5:16:1:16", args.seed, 10, False, peaks, local_rank, sampler)
                # one layer of the Qwen2.5-7B stack (28/4 heads, ragged prefixes, 256 query tokens, batch 8) and config 2
                extras["config4_layer"] = measure_point("config4_layer", args.seed, 10, False, peaks, local_rank, sampler)
                extras["config2"] = measure_point("config2", args.seed, 10, False, peaks, local_rank, sampler)
                extras["compressed_point"] = measure_compressed_point(args.seed, 10, peaks, local_rank, sampler=sampler)
                extras["host_packets_point"] = measure_host_packets_point(args.seed, 5, local_rank)
            except Exception as ex:                                   # extras never invalidate the main line
                extras["error"] = repr(ex)
            line["extra_points"] = extras
            wl2 = gen.DeviceWorkload(spec, f"cuda:{local_rank}")
            line["cpu_baseline"] = baseline_sample(spec, wl2)
        sampler.stop()
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
