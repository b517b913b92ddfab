#!/usr/bin/env python
"""Benchmark of the prefix-cached block-attention / greedy-accept hot path on B200.

One JSON line on stdout (rank 0).  A *step* is one pass of the whole hot path over one batch:
``agx_attn_prefixed_append`` (KV append + attention) for every layer pool of the workload, then one
``agx_accept_greedy`` over the verify blocks' logits.

Headline workload = "long context" (the largest of the five configurations): 4 sequences with a cached
context of 32768 tokens verifying q = 8 tokens each, plus one sequence prefilling a 2048-token suffix
over a 30720-token cached prefix, in one call; GQA 32/8, head_dim 128, bf16, page size 16 with shuffled
pages (1.3 GB of KV pools, far larger than L2); accept on bf16 logits [4 x 8, 128256].  ``value`` counts
query tokens per second (all block rows of the call / step time).  The other configurations (decode
verification, prefix-cached prefill, ragged mixed batch) are measured the same way and reported under
``workloads``, each with its roofline record, an end-to-end figure through the host-buffer entry
point, the CPU oracle timed beside it, median and minimum over the replays and the SM clock sampled
during its own timed region.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl agx|reference] [--no-extra]

N > 1 (under torchrun) runs one independent replica per GPU (the path shards by sequence with no
exchange step): weak scaling, value = all ranks' units / max-over-ranks time.
``--impl reference`` times the CPU oracle (the only reference there is) on a bounded sample.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "prefix-cached attn query tok/s"
UNIT = "query tok/s"
VOCAB = 128256
HKV, D = 8, 128
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0


# --------------------------------------------------------------------------- the configurations
def configs(W):
    """name -> (description, prefix lengths, block lengths, query heads, layer pools per step,
    indices of the verify sequences, pages shared by all sequences (tokens), seed)."""
    P4, q4 = W.c4_lengths()
    return {
        "c5_long_context": dict(
            text="long context (c5): 4 x (cached context 32768, verify q=8) + 1 x (cached prefix 30720, suffix prefill "
                 "q=2048) in one call, GQA 32/8, d=128, bf16, page 16 shuffled; accept on bf16 logits [4x8,128256]",
            P=[32768] * 4 + [30720], q=[8] * 4 + [2048], hq=32, layers=1, verify=[0, 1, 2, 3], shared=0, seed=5),
        "c2_decode_verify": dict(
            text="decode verification (c2): batch 1, cached context 4096, q=8, GQA 32/8, d=128, bf16, page 16 shuffled, "
                 "32 per-layer KV pools (553 MB) + accept on bf16 logits [8,128256]",
            P=[4096], q=[8], hq=32, layers=32, verify=[0], shared=0, seed=2),
        "c3_prefix_prefill": dict(
            text="prefix-cached prefill (c3): batch 1, cached prefix 3072 + uncached suffix q=512, GQA 24/8, d=128, bf16, "
                 "page 16 shuffled, 8 per-layer KV pools (235 MB)",
            P=[3072], q=[512], hq=24, layers=8, verify=[], shared=0, seed=3),
        "c4_ragged_mixed": dict(
            text="ragged mixed batch (c4): 16 sequences, cached lengths lognormal (median 4k, 2k-16k), 8 verify blocks "
                 "q in {1,2,4,8,16} + 8 suffix prefills q in 128..1024, first 2048 tokens' pages shared by all, "
                 "GQA 32/8, d=128, bf16; accept on the verify blocks' bf16 logits",
            P=[int(v) for v in P4], q=[int(v) for v in q4], hq=32, layers=1, verify=list(range(8)), shared=2048, seed=4),
    }


HEADLINE = "c5_long_context"


# --------------------------------------------------------------------------- peaks / clocks
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """One read-only ``nvidia-smi --query-gpu`` loop for the whole run; every sample is stamped on arrival, and a
    timed region is summarised from the samples that fell inside it."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_ms: int = 50):
        self.index, self.period_ms = index, period_ms
        self.proc = None
        self.samples = []   # (wall time, sm MHz, max MHz, [active reasons])

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
            t0 = time.time()
            while not self.samples and time.time() - t0 < 5.0:
                time.sleep(0.05)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm, mx = float(f[0]), float(f[1])
            except ValueError:
                continue
            self.samples.append((time.time(), sm, mx, [n for n, v in zip(self.NAMES, f[3:7]) if v.lower().startswith("active")]))

    def region(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        reasons = sorted({r for s in inside for r in s[3]})
        return {"sm_mhz": float(np.median([s[1] for s in inside])) if inside else None,
                "sm_max_mhz": max(s[2] for s in inside) if inside else None, "samples": len(inside), "reasons": reasons}

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()


# --------------------------------------------------------------------------- distributed helpers
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate_over_ranks(ms_local: float, units_local: float, backend_device=None):
    """Weak scaling over independent replicas: time = max over ranks, units = sum over ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, units_local
    dev = backend_device if backend_device is not None else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------- algorithmic work
def alg_bytes_attn(P, q, hq, hkv=HKV, d=D, esz=2, shared=0, first=True):
    """K and V of the visible tokens plus Q in and O out; pages shared by the batch count once (``first``)."""
    kv_tokens = (P + q) - (0 if first else shared)
    return 2 * hkv * d * esz * kv_tokens + 2 * q * hq * d * esz


def alg_flops_attn(P, q, hq, d=D):
    return 4 * d * hq * (q * P + q * (q + 1) // 2)


def roofline_record(bound, work, ms, peaks, extra=None):
    """bound 'hbm': work in bytes -> GB/s; 'tensor': work in flops -> TFLOP/s (against the sustained measured peak,
    since the kernels are timed inside long replayed graphs; the burst and nominal fractions ride along)."""
    if bound == "hbm":
        achieved = work / (ms * 1e-3) / 1e9
        rec = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
               "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (copy bandwidth)",
               "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS, "algorithmic_bytes": work}
    else:
        achieved = work / (ms * 1e-3) / 1e12
        rec = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
               "frac": achieved / peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " (sustained bf16 GEMM)",
               "frac_of_burst": achieved / peaks["bf16_tflops"], "burst_peak": peaks["bf16_tflops"],
               "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS, "algorithmic_flops": work}
    rec["us"] = ms * 1e3
    if extra:
        rec.update(extra)
    return rec


def ncu_traffic(summary_file: str, sources):
    """DRAM bytes per launch from a committed ncu summary (its ``traffic_bytes_per_launch:`` line), or None when the
    file is missing or the kernel sources changed after the counters were taken (``sources_sha256:`` line)."""
    path = os.path.join(ROOT, "profiles", summary_file)
    if not os.path.exists(path):
        return None, "no ncu summary committed"
    text = open(path).read()
    m = re.search(r"^traffic_bytes_per_launch:\s*([0-9]+)", text, re.M)
    h = re.search(r"^sources_sha256:\s*([0-9a-f]+)", text, re.M)
    if not m or not h:
        return None, "summary carries no machine-readable traffic line"
    if h.group(1) != sources_hash(sources):
        return None, "kernel sources changed since the counters were taken"
    return int(m.group(1)), f"profiles/{summary_file}"


def sources_hash(names):
    h = hashlib.sha256()
    for n in names:
        h.update(open(os.path.join(ROOT, "paper_2605_10380_b200", "csrc", n), "rb").read())
    return h.hexdigest()[:16]


TILE_SOURCES = ("agx_attn_tile.cu", "agx_sm100.cuh", "agx_internal.cuh")


# --------------------------------------------------------------------------- workload on the device
class LayeredVerify:
    """`layers` independent KV pools for one batch of sequences, plus logits for the accept step over the verify
    blocks (``verify`` = indices of the sequences whose blocks are draft groups)."""

    def __init__(self, torch, agx, W, P_list, q_list, hq, hkv, d, layers, vocab, seed, verify=None, shared=0,
                 planned_accept=None, early=True):
        self.torch, self.W, self.agx = torch, W, agx
        self.P = np.asarray(P_list, np.int32); self.Q = np.asarray(q_list, np.int32)
        self.hq, self.hkv, self.d, self.layers, self.vocab, self.shared = hq, hkv, d, layers, vocab, shared
        self.B = len(P_list)
        self.cu = W.cu_from_q(self.Q)
        self.total_q = int(self.cu[-1])
        g = torch.Generator(device="cuda"); g.manual_seed(seed)
        rng = np.random.default_rng(seed)
        table, self.num_pages = W.build_page_table(rng, self.P.astype(np.int64) + self.Q, shared, spare_pages=7)
        self.table_host = table
        self.page_table = torch.from_numpy(table).cuda()
        bf = torch.bfloat16
        rn = lambda *s: torch.randn(*s, generator=g, device="cuda", dtype=torch.float32).to(bf)
        self.k_pools = [rn(self.num_pages, hkv, 16, d) for _ in range(layers)]
        self.v_pools = [rn(self.num_pages, hkv, 16, d) for _ in range(layers)]
        self.q_block = [rn(self.total_q, hq, d) for _ in range(layers)]
        self.k_new = [rn(self.total_q, hkv, d) for _ in range(layers)]
        self.v_new = [rn(self.total_q, hkv, d) for _ in range(layers)]
        self.out = [torch.empty(self.total_q, hq, d, device="cuda", dtype=bf) for _ in range(layers)]
        self.prefix_dev = torch.from_numpy(self.P).cuda()
        self.cu_dev = torch.from_numpy(self.cu).cuda()
        self.h = agx.Handle(hq, hkv, d, "bf16")
        # every layer has its own pools and the cached prefixes were written by earlier steps: nothing in flight
        # writes the pages below the prefix length, so their loads may start before the dependency wait
        self.h.set_option(agx.AGX_OPT_EARLY_PREFIX_LOADS, 1 if early else 0)
        n = self.h.attn_workspace_bytes(self.P, self.Q)
        self.ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda") if n else None
        self.verify = list(verify) if verify is not None else []
        if vocab and self.verify:
            vq = self.Q[self.verify]
            aw = W.make_planted_accept("bench_accept", seed, "bf16", vocab, vq, self.P[self.verify], planned_accept=planned_accept)
            self.aw = aw
            self.logits = torch.from_numpy(aw.logits).cuda().view(bf)
            self.drafts = torch.from_numpy(aw.drafts if aw.drafts.size else np.zeros(1, np.int32)).cuda()
            self.acc = torch.zeros(len(self.verify), dtype=torch.int32, device="cuda")
            self.nxt = torch.zeros(len(self.verify), dtype=torch.int32, device="cuda")
            self.seq_lens = torch.from_numpy(self.P[self.verify].copy()).cuda()
            self.cu_verify = torch.from_numpy(aw.cu_q).cuda()
            self.acc_ws = torch.empty(self.h.accept_workspace_bytes(int(aw.cu_q[-1]), vocab), dtype=torch.uint8, device="cuda")
        else:
            self.aw = None

    def attn_layer(self, l):
        self.h.attn_prefixed(self.q_block[l], self.k_pools[l], self.v_pools[l], self.page_table, self.P, self.Q,
                             self.out[l], None, self.ws)
        return self.h.last_launch_count()

    def step(self, attn_only=False):
        n = 0
        for l in range(self.layers):
            if attn_only:
                n += self.attn_layer(l)
            else:   # the block's K/V rows are written by the attention kernel's CTAs before they read them
                self.h.attn_prefixed_append(self.q_block[l], self.k_new[l], self.v_new[l], self.k_pools[l], self.v_pools[l],
                                            self.page_table, self.P, self.Q, self.out[l], None, self.ws)
                n += self.h.last_launch_count()
        if not attn_only and self.aw is not None:
            # (the committed lengths simply keep advancing from replay to replay: their values feed nothing here)
            self.h.accept_greedy(self.logits, "bf16", self.vocab, self.drafts, self.cu_verify, self.acc, self.nxt, None,
                                 self.seq_lens, self.acc_ws)
            n += self.h.last_launch_count()
        return n

    def bytes_per_layer(self, idx=None):
        idx = range(self.B) if idx is None else idx
        return sum(alg_bytes_attn(int(self.P[s]), int(self.Q[s]), self.hq, self.hkv, self.d, shared=self.shared, first=(n == 0))
                   for n, s in enumerate(idx))

    def flops_per_layer(self, idx=None):
        idx = range(self.B) if idx is None else idx
        return sum(alg_flops_attn(int(self.P[s]), int(self.Q[s]), self.hq, self.d) for s in idx)


def capture(torch, fn):
    """Warm up (first calls configure kernels), then capture fn into a CUDA graph."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for _ in range(2):
            fn()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def time_graph(torch, g, steps, warmup, barrier=None):
    """Mean ms per replay over `steps` replays (events on the current stream, synchronised on both sides)."""
    for _ in range(warmup):
        g.replay()
    if barrier:
        barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    return e0.elapsed_time(e1) / steps


def replay_stats(torch, g, est_ms, blocks=100, warmup=5):
    """Median and minimum ms per replay over `blocks` timed blocks (at least 100 replays in all): an event between every
    two blocks of back-to-back replays (a block lasts about a millisecond, so the events' own cost does not show), no
    host synchronisation inside."""
    per = max(1, int(round(1.0 / max(est_ms, 1e-3))))
    for _ in range(warmup):
        g.replay()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(blocks + 1)]
    ev[0].record()
    for i in range(blocks):
        for _ in range(per):
            g.replay()
        ev[i + 1].record()
    torch.cuda.synchronize()
    t = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(blocks)]) / per
    return float(np.median(t)), float(t.min())


def timed_region(torch, g, min_seconds, est_ms, sampler, steps_min=100):
    """Replay `g` for at least `min_seconds` (so the clock sampler sees the region) and at least `steps_min` times."""
    steps = max(steps_min, int(min_seconds * 1e3 / max(est_ms, 1e-3)))
    t0 = time.time()
    ms = time_graph(torch, g, steps, 3)
    t1 = time.time()
    clocks = sampler.region(t0, t1) if sampler else None
    if clocks and clocks["sm_mhz"]:
        clocks["ms_x_sm_mhz"] = ms * clocks["sm_mhz"]
    return ms, steps, clocks


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_threads(n):
    """Limit the oracle's OpenMP team (the runtime it links is shared by the process)."""
    import ctypes
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def oracle_sample(lv, cfg, budget_s=4.0, threads=None):
    """The oracle, as it stands, on a bounded sample of the configuration, fed the very tensors the GPU ran on (first
    layer pool, copied to the host): whole verify blocks, and as many leading rows of the prefill blocks as the budget
    allows; cached prefixes in full."""
    import oracle
    torch, W = lv.torch, lv.W
    all_threads = oracle.num_threads()
    if threads:
        oracle_threads(threads)
    try:
        P, q, hq, verify = cfg["P"], cfg["q"], cfg["hq"], cfg["verify"]
        rate = 2.0e9 * (threads or all_threads)   # fp64 flop/s the oracle reaches, roughly: it only sizes the sample
        n_pre = max(1, len(P) - len(verify))
        plan = []
        for s in range(len(P)):
            rows = q[s]
            if s not in verify:
                rows = int(max(1, min(q[s], (budget_s * rate * 0.6 / n_pre) // alg_flops_attn(P[s], 1, hq))))
            plan.append(rows)
        host16 = lambda t: t.view(torch.uint16).cpu().numpy()
        kp, vp = host16(lv.k_pools[0]), host16(lv.v_pools[0])
        idx = np.concatenate([np.arange(lv.cu[s], lv.cu[s] + plan[s]) for s in range(len(P))])
        qb, kn, vn = host16(lv.q_block[0])[idx], host16(lv.k_new[0])[idx], host16(lv.v_new[0])[idx]
        cu = W.cu_from_q(plan)
        t0 = time.perf_counter()
        oracle.kv_append(kp, vp, kn, vn, "bf16", lv.table_host, lv.P, cu)
        oracle.attn_paged_batch(qb, kp, vp, lv.table_host, "bf16", lv.P, np.asarray(plan, np.int32), cu)
        rows_accept = 0
        if lv.aw is not None:
            aw = lv.aw
            oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
            rows_accept = int(aw.cu_q[-1])
        dt = time.perf_counter() - t0
        return {"value": float(sum(plan)) / dt, "unit": UNIT, "cores": threads or all_threads, "kind": "oracle", "seconds": dt,
                "sample": f"one layer call on the tensors the GPU ran on, prefill blocks cut to their first rows "
                          f"(block rows per sequence {plan}, cached prefixes in full; append + attention in fp64)"
                          + (f" + accept over [{rows_accept}, {VOCAB}] logits" if rows_accept else "")}
    finally:
        if threads:
            oracle_threads(all_threads)


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2605_10380_b200 import workloads as W
    import oracle
    cfg = configs(W)[HEADLINE]
    P, q, hq, verify = cfg["P"], cfg["q"], cfg["hq"], cfg["verify"]
    rows = [q[s] if s in verify else 8 for s in range(len(P))]   # the prefill block cut to its first 8 rows
    small = W.make_attn_workload("reference_sample", cfg["seed"], "bf16", hq, HKV, D, P, rows)
    aw = W.make_planted_accept("reference_accept", cfg["seed"], "bf16", VOCAB, [q[s] for s in verify], [P[s] for s in verify])
    kp, vp = small.k_pool.copy(), small.v_pool.copy()

    def step():
        oracle.kv_append(kp, vp, small.k_new, small.v_new, "bf16", small.page_table, small.prefix_len, small.cu_q)
        oracle.attn_paged_batch(small.q_block, kp, vp, small.page_table, "bf16", small.prefix_len, small.q_len, small.cu_q)
        oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)

    for _ in range(max(1, args.warmup)):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    tokens = float(sum(rows))
    value = args.steps * tokens / dt
    sample = (f"each step = one layer call of the workload (append + attention, fp64 oracle) with the 2048-row prefill block "
              f"cut to its first 8 rows (block rows {rows}, full cached contexts) + accept over [32, {VOCAB}] logits; "
              f"{tokens:.0f} query tokens per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg["text"], "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- one configuration, all figures
class HostStep:
    """The step through the host-buffer entry point: one agx_verify_step_host_enqueue per layer for the verify blocks
    (with the accept on the last layer) and one for the prefill blocks (attention only), then ONE stream synchronisation."""

    def __init__(self, torch, lv, cfg):
        self.torch, self.lv = torch, lv
        pin = lambda t: t.cpu().pin_memory()
        self.groups = []
        ver = [s for s in range(lv.B) if s in cfg["verify"]]
        pre = [s for s in range(lv.B) if s not in cfg["verify"]]
        self.h2d = self.d2h = 0
        for idx, with_accept in ((ver, True), (pre, False)):
            if not idx:
                continue
            rows = np.concatenate([np.arange(lv.cu[s], lv.cu[s + 1]) for s in idx])
            rows_t = torch.from_numpy(rows).cuda()
            P, Q = lv.P[idx].copy(), lv.Q[idx].copy()
            table = torch.from_numpy(np.ascontiguousarray(lv.table_host[idx])).cuda()
            g = dict(P=P, Q=Q, table=table, with_accept=with_accept,
                     hq=[pin(lv.q_block[l][rows_t]) for l in range(lv.layers)],
                     hk=[pin(lv.k_new[l][rows_t]) for l in range(lv.layers)],
                     hv=[pin(lv.v_new[l][rows_t]) for l in range(lv.layers)])
            g["out"] = [torch.empty_like(g["hq"][0]).pin_memory() for _ in range(lv.layers)]
            nb = len(idx)
            g["acc"] = torch.zeros(nb, dtype=torch.int32).pin_memory(); g["nxt"] = torch.zeros(nb, dtype=torch.int32).pin_memory()
            g["sl"] = torch.zeros(nb, dtype=torch.int32).pin_memory()
            vocab = lv.vocab if with_accept else 0
            if with_accept:
                g["logits"], g["drafts"] = pin(lv.logits), pin(lv.drafts)
            ws_n = lv.h.verify_step_host_workspace_bytes(P, Q, "bf16", lv.vocab, vocab)
            g["ws"] = torch.empty(ws_n, dtype=torch.uint8, device="cuda")
            esz, tq = 2, int(Q.sum())
            self.h2d += lv.layers * tq * (lv.hq + 2 * lv.hkv) * lv.d * esz
            self.d2h += lv.layers * tq * lv.hq * lv.d * esz
            if with_accept:
                self.h2d += tq * lv.vocab * esz + (tq - nb) * 4 + (2 * nb + 1) * 4
                self.d2h += 3 * nb * 4
            self.groups.append(g)

    def bind(self):
        """One pre-marshalled call per (layer, block kind); the attention-only variants serve the host-time figure."""
        lv = self.lv
        self.calls, self.calls_attn_only = [], []
        for l in range(lv.layers):
            last = l == lv.layers - 1
            for g in self.groups:
                for acc, dest in ((g["with_accept"] and last, self.calls), (False, self.calls_attn_only)):
                    dest.append(lv.h.verify_step_host_bind(
                        lv.k_pools[l], lv.v_pools[l], g["table"], g["P"], g["Q"], g["hq"][l], g["hk"][l], g["hv"][l],
                        g["logits"] if acc else None, "bf16", lv.vocab, lv.vocab if acc else 0, g["drafts"] if acc else None,
                        g["out"][l], g["acc"], g["nxt"], g["sl"], g["ws"]))

    def step(self):
        for call in self.calls:
            call()
        self.torch.cuda.current_stream().synchronize()   # one synchronisation per step: the host reads the results now

    def time(self, steps, warmup, barrier=None):
        self.bind()
        for _ in range(max(3, warmup)):
            self.step()
        if barrier:
            barrier()
        self.torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(steps):
            self.step()
        self.torch.cuda.synchronize()
        ms = (time.perf_counter() - t0) / steps * 1e3
        # host time of the enqueue calls alone (no synchronisation in between): what the CPU spends per call
        n_host = max(1, min(steps, 128 // max(1, len(self.calls_attn_only))))   # (short of the launch queue's depth)
        self.torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_host):
            for call in self.calls_attn_only:
                call()
        t_host = (time.perf_counter() - t0) / (n_host * len(self.calls_attn_only)) * 1e6
        self.torch.cuda.synchronize()
        return ms, t_host


def measure_config(torch, agx, W, name, cfg, peaks, sampler, args, barrier=None, rank=0, headline=False):
    lv = LayeredVerify(torch, agx, W, cfg["P"], cfg["q"], cfg["hq"], HKV, D, cfg["layers"], VOCAB, cfg["seed"] + rank,
                       verify=cfg["verify"], shared=cfg["shared"])
    launches = lv.step()
    torch.cuda.synchronize()
    assert lv.h.get_status() == 0
    tokens = float(lv.layers * lv.total_q)
    # ---- roofline parts: the attention call on each kind of block alone, against its own bound.  The bandwidth-bound
    #      verify blocks are timed first, before the long tensor-bound regions pull the board against its power cap.
    parts = {}
    ver = [s for s in range(lv.B) if s in cfg["verify"]]
    pre = [s for s in range(lv.B) if s not in cfg["verify"]]

    def measure_part(label, idx, bound):
        if not idx:
            return
        if len(idx) == lv.B:
            sub = lv
        else:
            # these blocks alone, over enough layer pools that the K/V pages come from HBM (300 MB or more in all) and that
            # one replay of the graph lasts about a millisecond (the gap between two graph launches, ~10 us, is not chained
            # the way the launches inside a graph are, and would otherwise count against a short call)
            P_, q_ = [cfg["P"][s] for s in idx], [cfg["q"][s] for s in idx]
            kv_mb = sum(a + b for a, b in zip(P_, q_)) * 4096 / 2 ** 20
            t_guess = max(kv_mb * 2 ** 20 / 5e12, sum(alg_flops_attn(a, b, cfg["hq"]) for a, b in zip(P_, q_)) / 1e15) + 10e-6
            n_layers = int(max(-(-300 // max(1.0, kv_mb)), min(8, -(-1e-3 // t_guess))))
            n_layers = int(max(1, min(n_layers, 8, (6 << 10) // max(1.0, 2 * kv_mb))))
            sub = LayeredVerify(torch, agx, W, P_, q_, cfg["hq"], HKV, D, n_layers, 0, cfg["seed"] + 17, shared=cfg["shared"])
        g = capture(torch, lambda: sub.step(attn_only=True))
        e = time_graph(torch, g, 3, 2)
        t_ms, _, ck = timed_region(torch, g, 0.5, e, sampler)
        t_ms /= sub.layers
        m2, n2 = replay_stats(torch, g, e)
        work = sub.bytes_per_layer() if bound == "hbm" else sub.flops_per_layer()
        parts[label] = roofline_record(bound, work, t_ms, peaks, {
            "median_us": m2 / sub.layers * 1e3, "min_us": n2 / sub.layers * 1e3, "clocks": ck,
            "launches_per_call": sub.attn_layer(0), "sequences": len(idx),
            "timed": "one agx_attn_prefixed call on these blocks alone, captured in a CUDA graph"
                     + (f" ({sub.layers} layer pools back to back)" if sub.layers > 1 else "")})
        del g
        torch.cuda.empty_cache()

    measure_part("verify_blocks", ver, "hbm")
    # ---- the whole step
    g_full = capture(torch, lv.step)
    est = time_graph(torch, g_full, 3, 2)
    if headline:
        t0 = time.time()
        ms = time_graph(torch, g_full, args.steps, args.warmup, barrier)
        clocks = sampler.region(t0, time.time()) if sampler else None
        steps = args.steps
        if clocks is not None and clocks["samples"] == 0:   # a region too short for the sampler: run it on, the K steps above stand
            _, _, clocks = timed_region(torch, g_full, 1.0, est, sampler)
            if clocks is not None:
                clocks["note"] = "the K timed steps ended before a sample fell inside; clocks from a 1 s continuation of the same replays"
    else:
        ms, steps, clocks = timed_region(torch, g_full, 1.0, est, sampler)
    med, mn = replay_stats(torch, g_full, est)
    rec = {"workload": cfg["text"], "ms_per_step": ms, "steps": steps, "median_ms": med, "min_ms": mn,
           "query_tok_per_step": tokens, "value": tokens / (ms * 1e-3), "unit": UNIT, "gpu_launches": launches, "clocks": clocks}
    measure_part("prefill_blocks", pre, "tensor")
    # whole attention call against max(sum flops / tensor peak, sum bytes / HBM peak)
    g = capture(torch, lambda: lv.step(attn_only=True))
    e = time_graph(torch, g, 3, 2)
    t_ms, _, _ = timed_region(torch, g, 0.5, e, sampler)
    t_ms /= lv.layers
    by, fl = lv.bytes_per_layer(), lv.flops_per_layer()
    t_roof_ms = max(fl / (peaks["bf16_tflops_sustained"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e3
    parts["whole_call"] = {"us": t_ms * 1e3, "algorithmic_bytes": by, "algorithmic_flops": fl,
                           "roofline_us": t_roof_ms * 1e3, "frac": t_roof_ms / t_ms,
                           "note": "max(sum of flops / sustained bf16 peak, sum of bytes / copy bandwidth) over the time of the one call; "
                                   "pages shared by the batch counted once"}
    del g
    rec["roofline"] = parts
    # ---- end to end through the host-buffer entry point
    hs = HostStep(torch, lv, cfg)
    e2e_steps = max(5, min(200, int(0.5e3 / max(est, 0.05))))
    e2e_ms, host_us = hs.time(e2e_steps, 3, barrier)
    rec["e2e"] = {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": hs.h2d,
                  "d2h_bytes_per_step": hs.d2h, "host_enqueue_us_per_call": host_us,
                  "calls_per_step": lv.layers * len(hs.groups),
                  "path": "agx_verify_step_host_enqueue per layer and block kind (pinned host q/k_new/v_new/logits in, "
                          "out and accept results back), one stream synchronisation per step"}
    if lv.aw is not None:
        rec["accept_lengths"] = {"planned": "uniform over 0..k per sequence",
                                 "histogram": np.bincount(lv.aw.planned_accept, minlength=int(lv.Q[cfg["verify"]].max())).tolist()}
    del hs
    return rec, lv


# --------------------------------------------------------------------------- extra workloads (N = 1)
def extra_workloads(torch, agx, W, peaks, sampler):
    out = {}

    def guarded(name):
        def deco(fn):
            try:
                out[name] = fn()
            except Exception as e:  # keep the headline line alive
                out[name] = {"error": repr(e)}
            torch.cuda.empty_cache()
        return deco

    @guarded("batched_verify_16x8192")
    def _():   # serving-style batch (the paper's own setting is batch 1): 16 x (P = 8192, q = 8), 537 MB of KV per call
        lv = LayeredVerify(torch, agx, W, [8192] * 16, [8] * 16, 32, HKV, D, 3, 0, 6)
        g = capture(torch, lambda: lv.step(attn_only=True))
        ms, _, ck = timed_region(torch, g, 0.5, 0.3, sampler)
        return dict(roofline_record("hbm", lv.bytes_per_layer(), ms / 3, peaks), query_tok_per_s=128 / (ms / 3 * 1e-3), clocks=ck)

    @guarded("accept_step")
    def _():   # accept alone: one read of the logits; 64 distinct buffers rotated inside one graph so they come from HBM
        acc = {}
        for name, q_list, planned in (("c2_accept_8x128256", [8], None), ("c5_accept_32x128256", [8] * 4, None),
                                      ("batch_accept_256x128256", [8] * 32, None)):
            h = agx.Handle(32, 8, 128, "bf16")
            rows, B, V = sum(q_list), len(q_list), VOCAB
            nbuf = 64 if rows <= 32 else 8
            bufs = [torch.randn(rows, V, device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
            drafts = torch.randint(0, V, (max(rows - B, 1),), device="cuda", dtype=torch.int32)
            cu = torch.from_numpy(W.cu_from_q(q_list)).cuda()
            al = torch.zeros(B, dtype=torch.int32, device="cuda"); nt = torch.zeros(B, dtype=torch.int32, device="cuda")
            ws = torch.empty(h.accept_workspace_bytes(rows, V), dtype=torch.uint8, device="cuda")

            def run():
                for x in bufs:
                    h.accept_greedy(x, "bf16", V, drafts, cu, al, nt, None, None, ws)
            g = capture(torch, run)
            ms, _, _ = timed_region(torch, g, 0.3, 0.5, sampler)
            med, mn = replay_stats(torch, g, ms)
            by = rows * V * 2
            acc[name] = dict(roofline_record("hbm", by, ms / nbuf, peaks), median_us=med / nbuf * 1e3, min_us=mn / nbuf * 1e3)
            del bufs, g
            torch.cuda.empty_cache()
        return acc

    @guarded("accept_paper_shaped")
    def _():
        # draft groups of 4 (the paper's figure) accepted token by token with probability 0.25 (its Table 3: 48 of 194 and
        # 56 of 218 drafts accepted); 64 sequences, results bit-exact against the planted plan; reported, not gated
        rng = np.random.default_rng(25)
        B, k, V = 64, 4, VOCAB
        planned = np.array([int(np.argmax(np.append(rng.random(k) >= 0.25, True))) for _ in range(B)], dtype=np.int32)
        aw = W.make_planted_accept("paper_shaped", 26, "bf16", V, [k + 1] * B, [4096] * B, planned_accept=planned)
        h = agx.Handle(32, 8, 128, "bf16")
        logits = torch.from_numpy(aw.logits).cuda().view(torch.bfloat16)
        drafts = torch.from_numpy(aw.drafts).cuda(); cu = torch.from_numpy(aw.cu_q).cuda()
        al = torch.zeros(B, dtype=torch.int32, device="cuda"); nt = torch.zeros(B, dtype=torch.int32, device="cuda")
        ws = torch.empty(h.accept_workspace_bytes(B * (k + 1), V), dtype=torch.uint8, device="cuda")
        g = capture(torch, lambda: h.accept_greedy(logits, "bf16", V, drafts, cu, al, nt, None, None, ws))
        ms, _, _ = timed_region(torch, g, 0.3, 0.03, sampler)
        got = al.cpu().numpy()
        return {"sequences": B, "drafts_per_group": k, "per_token_acceptance": 0.25, "us": ms * 1e3,
                "accept_length_histogram": np.bincount(got, minlength=k + 1).tolist(),
                "accepted_drafts": int(got.sum()), "drafts": B * k, "matches_plan": bool(np.array_equal(got, planned)),
                "GB/s": B * (k + 1) * V * 2 / (ms * 1e-3) / 1e9, "paper": "48/194 and 56/218 drafts accepted (its Table 3)"}

    @guarded("kv_append_512_tokens")
    def _():   # KV append alone: the 512-token suffix of the prefill configuration (1 MB of K and of V, read + write)
        lv = LayeredVerify(torch, agx, W, [3072], [512], 24, HKV, D, 8, 0, 13)

        def run_append():
            for l in range(lv.layers):
                lv.h.kv_append(lv.k_pools[l], lv.v_pools[l], lv.k_new[l], lv.v_new[l], lv.page_table, lv.prefix_dev, lv.cu_dev)
        g = capture(torch, run_append)
        ms, _, _ = timed_region(torch, g, 0.2, 0.02, sampler)
        ms /= lv.layers
        by = 2 * 2 * 512 * 8 * 128 * 2
        return {"us": ms * 1e3, "GB/s": by / (ms * 1e-3) / 1e9}

    @guarded("multi_token_tax")
    def _():   # one attention call verifying q = 8 tokens against decoding q = 1 over the same context
        tax = {}   # (the paper measures 1.86x for q = 2 with its stock attention; the point of the small-q kernels is ~1.0)
        for P, B, layers in ((4096, 1, 32), (32768, 4, 1)):
            t = {}
            for q in (1, 8):
                lv = LayeredVerify(torch, agx, W, [P] * B, [q] * B, 32, HKV, D, layers, 0, 11)
                g = capture(torch, lambda: lv.step(attn_only=True))
                t[q] = timed_region(torch, g, 0.3, 0.3, sampler)[0] / layers
                del lv, g
                torch.cuda.empty_cache()
            tax[f"P{P}_batch{B}"] = {"us_q1": t[1] * 1e3, "us_q8": t[8] * 1e3, "ratio_q8_over_q1": t[8] / t[1]}
        return tax

    @guarded("mid_q_second_workload")
    def _():
        # the paper's second LLM call (its Sec. 3.2: input 88-90 % static): a suffix of 80-200 tokens over a cached prefix of
        # 0.7-1.5k tokens, q * G near the ridge between the bandwidth and the tensor roofline
        res = {}
        for P, q in ((700, 80), (1000, 128), (1500, 200)):
            lv = LayeredVerify(torch, agx, W, [P], [q], 32, HKV, D, 16, 0, 31)
            g = capture(torch, lambda: lv.step(attn_only=True))
            ms_g = timed_region(torch, g, 0.3, 0.3, sampler)[0]
            ms = ms_g / lv.layers
            med, mn = replay_stats(torch, g, ms_g)
            fl, by = lv.flops_per_layer(), lv.bytes_per_layer()
            t_roof = max(fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9))
            res[f"P{P}_q{q}"] = {"us": ms * 1e3, "median_us": med / lv.layers * 1e3, "min_us": mn / lv.layers * 1e3,
                                 "TFLOP/s": fl / (ms * 1e-3) / 1e12, "GB/s": by / (ms * 1e-3) / 1e9,
                                 "frac_of_burst_bf16": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                 "roofline_us": t_roof * 1e6, "launches_per_call": lv.attn_layer(0)}
            del lv, g
            torch.cuda.empty_cache()
        return res

    @guarded("ngram_and_prefix_reuse")
    def _():   # the steps around the hot path: n-gram draft table (Sec. 4.3) and prefix-reuse page traffic (Sec. 4.2)
        h = agx.Handle(32, 8, 128, "bf16")
        rng = np.random.default_rng(17)
        n_tok = 4096                                                   # a prompt-sized token stream over a 2k-token alphabet
        toks = torch.from_numpy(rng.integers(0, 2048, n_tok).astype(np.int32)).cuda()
        lut = torch.empty(agx.ngram_lut_bytes(n_tok), dtype=torch.uint8, device="cuda")
        nws = torch.empty(agx.ngram_workspace_bytes(n_tok), dtype=torch.uint8, device="cuda")
        g = capture(torch, lambda: h.ngram_build(toks, 3, lut, nws))
        t_build = time_graph(torch, g, 200, 5)
        ctx = toks[100:102].reshape(1, 2).contiguous()
        fill = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
        dr = torch.zeros((1, 4), dtype=torch.int32, device="cuda"); hd = torch.zeros(1, dtype=torch.int32, device="cuda")
        g2 = capture(torch, lambda: h.ngram_draft(lut, ctx, fill, 4, dr, hd))
        t_draft = time_graph(torch, g2, 200, 5)
        res = {"ngram_trigram_4096_tokens": {"build_us": t_build * 1e3, "draft_4_tokens_us": t_draft * 1e3,
                                             "paper_build_ms_on_its_cpu": 83.0}}
        # copy of one cut page per sequence (16 sequences); import of a 3072-token stored prefix from pinned host memory,
        # alone, and on a side stream while attention over resident pages runs on the main stream
        lv = LayeredVerify(torch, agx, W, [3072], [512], 24, HKV, D, 8, 0, 19)
        spare = lv.num_pages
        kp = torch.zeros((spare + 400, HKV, 16, D), dtype=torch.bfloat16, device="cuda"); vp = torch.zeros_like(kp)
        src = torch.arange(0, 16, dtype=torch.int32, device="cuda"); dst = torch.arange(100, 116, dtype=torch.int32, device="cuda")
        g3 = capture(torch, lambda: h.kv_copy_pages(kp, vp, src, dst))
        t_copy = time_graph(torch, g3, 200, 5)
        n_imp = 3072 // 16
        hk = torch.zeros((n_imp, HKV, 16, D), dtype=torch.bfloat16).pin_memory(); hv = torch.zeros_like(hk).pin_memory()
        dst_imp = torch.arange(spare, spare + n_imp, dtype=torch.int32, device="cuda")
        stg = torch.empty(h.kv_import_staging_bytes(n_imp), dtype=torch.uint8, device="cuda")
        side = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        n_rep = 20

        def imports(stream):
            for _ in range(n_rep):
                h.kv_import_pages(kp, vp, hk, hv, dst_imp, stg, stream=stream)

        def attention():
            for _ in range(n_rep):
                lv.step(attn_only=True)   # 8 prefill layers of the c3 shape: ~0.25 ms per step

        def timed(fn):
            for _ in range(2):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(main)
            fn()
            e1.record(main)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n_rep

        t_att = timed(attention)

        def both():
            side.wait_stream(main)
            imports(side)
            attention()
            main.wait_stream(side)
        imp_bytes = 2 * n_imp * HKV * 16 * D * 2
        rec = {"copy_16_pages_us": t_copy * 1e3, "import_bytes": imp_bytes, "attention_8_layers_us": t_att * 1e3,
               "note": "import of a 3072-token stored prefix on a side stream while 8 prefill-attention layer calls (P=3072, "
                       "q=512) over resident pages run on the main stream, against the two back to back (the paper: KV load "
                       "is 5.8-11.7 % of prefill latency)"}
        for label, bits in (("kernel_reads_host_pages", 3), ("copy_engine_then_scatter", 2)):
            h.set_option(agx.AGX_OPT_ZERO_COPY, bits)
            t_imp = timed(lambda: imports(main))
            t_both = timed(both)
            rec[label] = {"import_alone_us": t_imp * 1e3, "import_GB/s": imp_bytes / (t_imp * 1e-3) / 1e9,
                          "import_beside_attention_us": t_both * 1e3, "import_then_attention_us": (t_imp + t_att) * 1e3,
                          "hidden_fraction_of_import": max(0.0, min(1.0, (t_imp + t_att - t_both) / t_imp))}
        h.set_option(agx.AGX_OPT_ZERO_COPY, 3)
        res["prefix_reuse_pages"] = rec
        return res

    return out


# --------------------------------------------------------------------------- main arm
def run_agx(args):
    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the agx path")
    torch.cuda.set_device(local_rank)
    barrier = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        barrier = lambda: dist.barrier()
    from paper_2605_10380_b200 import build as _build
    if rank == 0:
        _build.build()
    if barrier:
        barrier()
    from paper_2605_10380_b200 import agx
    from paper_2605_10380_b200 import workloads as W
    peaks = load_peaks()
    cfgs = configs(W)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    head, lv = measure_config(torch, agx, W, HEADLINE, cfgs[HEADLINE], peaks, sampler, args, barrier, rank, headline=True)
    ms_max, units_all = aggregate_over_ranks(head["ms_per_step"], head["query_tok_per_step"], torch.device("cuda", local_rank))
    e2e_ms_max, _ = aggregate_over_ranks(head["e2e"]["ms_per_step"], head["query_tok_per_step"], torch.device("cuda", local_rank))
    if rank != 0:
        return
    dom = dict(head["roofline"]["prefill_blocks"])   # the dominant kernel of the step: the 256-row tensor-core schedule
    traffic, traffic_src = ncu_traffic("attn_tile_bf16_c5_long_context_prefill.txt", TILE_SOURCES)
    dom.update({"traffic": traffic, "traffic_source": traffic_src,
                "kernel": "attn_tile_bf16_kernel<false> (+ attn_combine_kernel where the planner splits the KV axis): the "
                          "agx_attn_prefixed call on the 2048-row prefill block",
                "us_per_launch": dom["us"], "share_of_step": dom["us"] * 1e-3 / head["ms_per_step"]})
    line = {
        "metric": METRIC, "value": units_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfgs[HEADLINE]["text"],
                   "step": "1 x agx_attn_prefixed_append (KV append + attention, 5 sequences, 2080 block rows) + "
                           "1 x agx_accept_greedy ([32, 128256] logits), one CUDA graph",
                   "l2": "inputs larger than L2: 1.3 GB of KV pools, each page read once per step",
                   "options": "AGX_OPT_EARLY_PREFIX_LOADS on (cached prefixes are not written by launches in flight)",
                   "parallelism": f"{world} independent replica(s), no collective"},
        "gpu_launches": head["gpu_launches"], "median_ms": head["median_ms"], "min_ms": head["min_ms"],
        "e2e": dict(head["e2e"], value=units_all / (e2e_ms_max * 1e-3), ms_per_step=e2e_ms_max),
        "roofline": dom, "clocks": head["clocks"],
    }
    if world == 1:
        line["cpu_baseline"] = oracle_sample(lv, cfgs[HEADLINE], budget_s=6.0)
        del lv
        torch.cuda.empty_cache()
        work = {HEADLINE: {k: head[k] for k in ("roofline", "accept_lengths") if k in head}}
        if not args.no_extra:
            for name, cfg in cfgs.items():
                if name == HEADLINE:
                    continue
                try:
                    rec, lv = measure_config(torch, agx, W, name, cfg, peaks, sampler, args)
                    rec["cpu_baseline"] = oracle_sample(lv, cfg, budget_s=3.0)
                    if name in ("c2_decode_verify", "c3_prefix_prefill"):
                        rec["cpu_baseline_single_thread"] = oracle_sample(lv, cfg, budget_s=3.0, threads=1)
                    work[name] = rec
                    del lv
                except Exception as e:
                    work[name] = {"error": repr(e)}
                torch.cuda.empty_cache()
            try:
                work["c1_tiny_verify_oracle_single_thread"] = oracle_c1(W)
            except Exception as e:
                work["c1_tiny_verify_oracle_single_thread"] = {"error": repr(e)}
            work.update(extra_workloads(torch, agx, W, peaks, sampler))
        line["workloads"] = work
    if sampler:
        sampler.stop()
    print(json.dumps(line))


def oracle_c1(W):
    """The tiny fp32 configuration through the oracle, single-threaded (reported only)."""
    import oracle
    w = W.c1_tiny_verify()
    all_threads = oracle.num_threads()
    oracle_threads(1)
    try:
        kp, vp = w.k_pool.copy(), w.v_pool.copy()
        n, t0 = 200, time.perf_counter()
        for _ in range(n):
            oracle.kv_append(kp, vp, w.k_new, w.v_new, w.dtype, w.page_table, w.prefix_len, w.cu_q)
            oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, w.dtype, w.prefix_len, w.q_len, w.cu_q)
        dt = (time.perf_counter() - t0) / n
        return {"value": 4 / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "us_per_call": dt * 1e6}
    finally:
        oracle_threads(all_threads)


ONLY = {  # name: (P list, q list, Hq, layers)
    "c2": ([4096], [8], 32, 4),
    "c2q1": ([4096], [1], 32, 4),
    "c3": ([3072], [512], 24, 1),
    "c4v": None, "c4p": None,   # the verify / prefill half of the ragged mixed batch (filled in at run time)
    "c5v": ([32768] * 4, [8] * 4, 32, 1),
    "c5p": ([30720], [2048], 32, 1),
    "c5p_small": ([7680], [1024], 32, 1),
    "b4": ([4096] * 4, [8] * 4, 32, 2),     # four verify blocks: KV splits merged inside thread-block clusters
    "m80": ([700], [80], 32, 2), "m128": ([1000], [128], 32, 2), "m200": ([1500], [200], 32, 2),
    "accept8": None, "append512": None, "ngram": None,   # the other kernels of the library
    "step": None,                                         # the headline step itself, eagerly: the launch list of one step
}


def run_only(args):
    """Profiling aid: eager (no graph) calls of ONE workload, a few launches, one line out."""
    import torch
    torch.cuda.set_device(0)
    from paper_2605_10380_b200 import agx
    from paper_2605_10380_b200 import workloads as W
    name = args.only
    if name == "step":
        cfg = configs(W)[HEADLINE]
        lv = LayeredVerify(torch, agx, W, cfg["P"], cfg["q"], cfg["hq"], HKV, D, cfg["layers"], VOCAB, cfg["seed"],
                           verify=cfg["verify"], shared=cfg["shared"])
        for _ in range(args.warmup):
            n = lv.step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            n = lv.step()
        e1.record()
        torch.cuda.synchronize()
        assert lv.h.get_status() == 0
        print(json.dumps({"only": name, "ms_per_step_eager": e0.elapsed_time(e1) / args.steps, "launches_per_step": n}))
        return
    if name in ("accept8", "append512", "ngram"):
        h = agx.Handle(32, 8, 128, "bf16")
        if name == "accept8":
            aw = W.make_planted_accept("only_accept", 9, "bf16", VOCAB, [8], [4096])
            logits = [torch.from_numpy(aw.logits).cuda().view(torch.bfloat16).clone() for _ in range(3)]
            drafts = torch.from_numpy(aw.drafts).cuda(); cu = torch.from_numpy(aw.cu_q).cuda()
            al = torch.zeros(1, dtype=torch.int32, device="cuda"); nt = torch.zeros(1, dtype=torch.int32, device="cuda")
            ws = torch.empty(h.accept_workspace_bytes(8, VOCAB), dtype=torch.uint8, device="cuda")
            fn = lambda i: h.accept_greedy(logits[i % 3], "bf16", VOCAB, drafts, cu, al, nt, None, None, ws)
        elif name == "append512":
            lv = LayeredVerify(torch, agx, W, [3072], [512], 24, HKV, D, 3, 0, 13)
            fn = lambda i: lv.h.kv_append(lv.k_pools[i % 3], lv.v_pools[i % 3], lv.k_new[i % 3], lv.v_new[i % 3], lv.page_table,
                                          lv.prefix_dev, lv.cu_dev)
        else:
            rng = np.random.default_rng(17)
            toks = torch.from_numpy(rng.integers(0, 2048, 4096).astype(np.int32)).cuda()
            lut = torch.empty(agx.ngram_lut_bytes(4096), dtype=torch.uint8, device="cuda")
            nws = torch.empty(agx.ngram_workspace_bytes(4096), dtype=torch.uint8, device="cuda")
            ctx = toks[100:102].reshape(1, 2).contiguous(); fill = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
            dr = torch.zeros((1, 4), dtype=torch.int32, device="cuda"); hd = torch.zeros(1, dtype=torch.int32, device="cuda")

            def fn(i):
                h.ngram_build(toks, 3, lut, nws)
                h.ngram_draft(lut, ctx, fill, 4, dr, hd)
        for i in range(args.warmup):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        assert h.get_status() == 0
        print(json.dumps({"only": name, "ms_per_call_eager": e0.elapsed_time(e1) / args.steps}))
        return
    if name in ("c4v", "c4p"):
        P4, q4 = W.c4_lengths()
        idx = range(8) if name == "c4v" else range(8, 16)
        P, q, hq, layers, shared = [int(P4[s]) for s in idx], [int(q4[s]) for s in idx], 32, 1, 2048
    else:
        (P, q, hq, layers), shared = ONLY[name], 0
    lv = LayeredVerify(torch, agx, W, P, q, hq, HKV, D, layers, 0, 7, shared=shared)
    for _ in range(args.warmup):
        for l in range(layers):
            lv.attn_layer(l)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        for l in range(layers):
            lv.attn_layer(l)
    e1.record()
    torch.cuda.synchronize()
    assert lv.h.get_status() == 0
    ms = e0.elapsed_time(e1) / (args.steps * layers)
    print(json.dumps({"only": name, "ms_per_call_eager": ms, "bytes": lv.bytes_per_layer(),
                      "flops": lv.flops_per_layer(), "GBps": lv.bytes_per_layer() / ms / 1e6,
                      "TFLOPs": lv.flops_per_layer() / ms / 1e9}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="agx", choices=["agx", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="headline workload only")
    ap.add_argument("--only", choices=sorted(ONLY), help="profiling aid: eager attention calls of one workload")
    args = ap.parse_args()
    if args.only:
        return run_only(args)
    if args.impl == "reference":
        if args.steps == 1000:
            args.steps = 10   # (the default is sized for the GPU arm: the oracle takes about a second per step)
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_agx(args)


if __name__ == "__main__":
    main()
