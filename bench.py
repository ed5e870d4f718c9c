#!/usr/bin/env python
"""Benchmark of the PureKV hot path on B200.

A step = one pass of the whole hot path over one synthetic batch: planning, ST-SpAttn prefill
of every layer (dense causal up to the CLIE layer), low-layer window scores, V-norm top-h
selection and K/V compaction of the compressed layers.  Default workload: the
VideoLLaMA2-shaped one (32 layers, 32/8 heads, head_dim 128, 2432 tokens, bf16).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--cfg 1] [--impl reference]

Prints ONE JSON line (rank 0).  `value` = prefill tokens/s of the whole job with inputs
resident in HBM; `e2e` = the same with inputs in pinned host memory and the compact cache read
back; `roofline` describes the dominant kernel (tensor-core prefill); `cpu_baseline` is the
fp64 oracle timed on this machine's host cores on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "st_spattn_prefill_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one ST-SpAttn launch of the tensor-core prefill
# kernel, from the ncu capture summarised under profiles/.  It is reported only while the kernel and planner
# sources are the ones the capture was taken from (sha1 of their text); otherwise the roofline's traffic is null.
NCU_TRAFFIC = {"cfg1_videollama2": {"bytes_per_launch": 31.0e6, "source_sha1": "6c7e587a4c974b32291d8bee206eaa2ce03d012b"}}
KERNEL_SOURCES = ("prefill_tc.cu", "tc_util.cuh", "plan.cu", "common.cuh", "prefill.cuh")


def kernel_source_sha1() -> str:
    import hashlib
    h = hashlib.sha1()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2510_25600_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic(workload: str):
    rec = NCU_TRAFFIC.get(workload)
    if rec and rec["bytes_per_launch"] is not None and rec["source_sha1"] == kernel_source_sha1():
        return rec["bytes_per_launch"]
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU while the timed region runs: NVML read-only queries
    from a thread every few milliseconds, or `nvidia-smi -lms` when the NVML binding is missing."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.sm, self.smax, self.reasons = [], [], set()
        self.proc = self.thread = self.nvml = None
        self._stop = threading.Event()

    def _physical_index(self) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [v.strip() for v in vis.split(",") if v.strip()]
            if self.index < len(ids) and ids[self.index].isdigit():
                return int(ids[self.index])
        return self.index

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.smax.append(float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)))
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self._physical_index()}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll_nvml(self):
        n = self.nvml
        bits = {"hw_slowdown": n.nvmlClocksEventReasonHwSlowdown, "hw_thermal_slowdown": n.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": n.nvmlClocksEventReasonSwThermalSlowdown, "sw_power_cap": n.nvmlClocksEventReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                r = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def _read_smi(self):
        for line in self.proc.stdout:
            r = [c.strip() for c in line.split(",")]
            try:
                self.sm.append(float(r[0]))
                self.smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(self.NAMES, r[3:7]):
                if v.lower().startswith("active"):
                    self.reasons.add(name)

    def stop(self):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["clock query unavailable"]}
        self.thread.join(timeout=2)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": max(self.smax) if self.smax else None,
                "samples": len(self.sm), "reasons": sorted(self.reasons),
                "source": "nvml" if self.nvml is not None else "nvidia-smi"}


# ---- multi-process plumbing: one process per GPU, replicas only (the path has no exchange step) -----------
def rank_env():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(x: float, device="cpu") -> float:
    """Max of a host scalar over all ranks (the slowest rank sets the job's time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(tokens_per_rank: int, world: int, seconds_per_step_max: float) -> float:
    """Whole-job tokens/s of `world` independent replicas that each process tokens_per_rank per step."""
    return world * tokens_per_rank / seconds_per_step_max


def oracle_sample(wl, layers_x, budget_s: float = 20.0):
    """Times the oracle on a bounded sample of the step; returns (tokens/s extrapolated to the whole step,
    cores, description).  Prefill: all heads of a row sample of one ST layer and of the dense layer; score,
    selection and compaction of one layer in full."""
    from oracle import purekv_oracle as po
    b = wl.batch
    cu = b.cu_seqlens
    t_tot = b.total_tokens
    rng = np.random.default_rng(wl.seed)
    cores = len(os.sched_getaffinity(0))
    x0 = layers_x[0]
    x1 = next((x for x in layers_x[1:] if "q" in x), x0)
    dense = type(wl.mask)(wl.mask.grid_h, wl.mask.grid_w, tile=wl.mask.tile, dense_causal=True)
    n_rows = min(t_tot, 256)
    rows = np.sort(rng.choice(t_tot, size=n_rows, replace=False))
    t = time.perf_counter()
    po.prefill(x1["q"], x1["k"], x1["v"], cu, b.n_prefix, b.n_frames, po.mask_params(wl.mask), rows=rows)
    t_st = (time.perf_counter() - t) * t_tot / n_rows
    t = time.perf_counter()
    po.prefill(x0["q"], x0["k"], x0["v"], cu, b.n_prefix, b.n_frames, po.mask_params(dense), rows=rows)
    t_dense = (time.perf_counter() - t) * t_tot / n_rows
    t = time.perf_counter()
    c = po.lowlayer_score(x0["q"], x0["k"], cu, wl.window)
    t_score = time.perf_counter() - t
    hk, ck = po.budgets(b.seq_lens, wl.window, wl.keep_ratio)
    t = time.perf_counter()
    s = po.vnorm_scores(c, x1["v"])
    idx, _ = po.select(s, cu, wl.window, hk, ck)
    po.compact(x1["k"], idx, cu, ck)
    po.compact(x1["v"], idx, cu, ck)
    t_comp = time.perf_counter() - t
    n_dense = max(wl.scored_layers) + 1
    n_st = wl.n_layers - n_dense
    total = n_dense * t_dense + n_st * t_st + len(wl.scored_layers) * t_score + len(wl.compacted_layers) * t_comp
    desc = (f"{n_rows} seeded rows x all {wl.n_q_heads} heads of one ST layer and one dense layer, full score / select / "
            f"compact of one layer; extrapolated to {n_dense} dense + {n_st} ST layers, {len(wl.scored_layers)} scored, "
            f"{len(wl.compacted_layers)} compacted")
    return t_tot / total, cores, desc, total


def run_reference(args, wl):
    """--impl reference: the oracle as it stands, on host cores, bounded sample per step."""
    if rank_env()[1] != 0:
        return
    from oracle import purekv_oracle as po
    from paper_2510_25600_b200 import inputs
    po.build()
    pool = ThreadPoolExecutor(len(os.sched_getaffinity(0)))
    layers_x = [inputs.make_qkv(wl, l, pool=pool) for l in range(min(2, wl.n_layers))]
    vals, tot = [], 0.0
    for i in range(args.warmup + args.steps):
        v, cores, desc, total = oracle_sample(wl, layers_x)
        if i >= args.warmup:
            vals.append(v)
            tot += total
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / max(1, args.steps),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "tokens": wl.batch.total_tokens, "layers": wl.n_layers},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """--sweep: the long-video workload (cfg 3) under masks of growing block density, and its compression at
    three keep ratios.  Prints one JSON line with a table; a companion to the default line, not a replacement."""
    import torch
    from paper_2510_25600_b200 import binding as P, inputs
    wl = inputs.workload(3)
    b = wl.batch
    peaks, peak_kind = load_peaks()
    pool = ThreadPoolExecutor(len(os.sched_getaffinity(0)))
    x = inputs.make_qkv(wl, 0, pool=pool)
    up = lambda n: torch.from_numpy(x[n + "_bits"].view(np.int16)).cuda().view(torch.bfloat16)
    q, k, v = up("q"), up("k"), up("v")
    db = P.Batch(b.seq_lens, b.n_prefix, b.n_frames)
    g = b.grid_h
    M = inputs.STMask
    masks = [("paper mask", wl.mask)]
    masks += [(f"whole-frame links, depth {d}", M(g, g, 1, -1, d, 1, -1, tile=128)) for d in (1, 2, 4, 8, 16)]
    masks += [(f"same cell of all earlier frames at stride {st}", M(g, g, 1, -1, -1, st, 0, tile=128)) for st in (10, 5, 3)]
    masks += [("spatial radius 4", M(g, g, 1, 4, 1, 1, 0, tile=128)), ("dense causal", M(g, g, tile=128, dense_causal=True))]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = torch.empty_like(q)

    def timed(fn, reps):
        out = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1))
        return float(np.median(out))

    rows = []
    peak = float(peaks["bf16_tflops"])
    for name, m in masks:
        plan = P.purekv_plan_build(db, P.st_params(m), P.BF16, wl.head_dim, wl.n_q_heads, wl.n_kv_heads)
        ws = torch.empty(max(16, plan.info.ws_bytes), dtype=torch.uint8, device="cuda")
        fn = lambda: P.purekv_st_sparse_prefill(q, k, v, db, plan, out=o, status=status, ws=ws)
        for _ in range(3):
            fn()
        ms = timed(fn, max(3, min(args.steps, 10)))
        info = plan.info
        tf = 4.0 * info.tile_q * info.tile_k * wl.head_dim * wl.n_q_heads * info.tiles_kept / ms / 1e9
        rows.append({"mask": name, "block_density": info.tiles_kept / info.tiles_causal, "ms": ms, "TFLOPs": tf,
                     "frac_of_burst_peak": tf / peak, "tokens_per_s": b.total_tokens / (ms * 1e-3)})
    P.purekv_poll_status(status)
    comp = []
    hbm = float(peaks["hbm_gbs"])
    kk, vv = k[None].contiguous(), v[None].contiguous()
    row = wl.n_kv_heads * wl.head_dim * 2
    for keep in (0.1, 0.2, 0.5):
        bud = P.Budget(db, wl.window, keep)
        c = P.purekv_lowlayer_score(q, k, db, wl.window)
        idx = P.purekv_select_topk(c, vv, db, bud)
        t_sel = timed(lambda: P.purekv_select_topk(c, vv, db, bud, idx_out=idx), 5)
        kc, vc = P.purekv_compact_kv(kk, vv, idx, db, bud)
        t_cmp = timed(lambda: P.purekv_compact_kv(kk, vv, idx, db, bud, k_out=kc, v_out=vc), 5)
        by = 4 * bud.total_kept * row + wl.n_kv_heads * bud.total_kept * 4
        # one decode step (one new query) over this layer's compact cache
        q_dec = q[-1:].contiguous()
        o_dec = torch.empty_like(q_dec)
        ws_dec = torch.empty(max(16, P.purekv_decode_ws_bytes(1, bud.total_kept, wl.n_q_heads, wl.n_kv_heads, wl.head_dim)),
                             dtype=torch.uint8, device="cuda")
        t_dec = timed(lambda: P.purekv_decode_attention(q_dec, kc[0], vc[0], bud, out=o_dec, ws=ws_dec), 5)
        comp.append({"keep_ratio": keep, "kept": bud.total_kept, "select_ms": t_sel, "compact_ms": t_cmp,
                     "compact_GBps": by / t_cmp / 1e6, "compact_frac_hbm": by / t_cmp / 1e6 / hbm,
                     "decode_ms": t_dec, "decode_GBps": 2 * bud.total_kept * row / t_dec / 1e6})
    t_score = timed(lambda: P.purekv_lowlayer_score(q, k, db, wl.window, c_out=c), 5)
    # the same scores in one pass from the dense layer's log-sum-exp (what the pipeline runs for this shape)
    dense = inputs.STMask(b.grid_h, b.grid_w, tile=wl.mask.tile, dense_causal=True)
    plan_d = P.purekv_plan_build(db, P.st_params(dense), P.BF16, wl.head_dim, wl.n_q_heads, wl.n_kv_heads)
    ws_d = torch.empty(max(16, plan_d.info.ws_bytes), dtype=torch.uint8, device="cuda")
    lse = torch.empty((wl.n_q_heads, b.total_tokens), dtype=torch.float32, device="cuda")
    P.purekv_st_sparse_prefill(q, k, v, db, plan_d, out=o, lse=lse, status=status, ws=ws_d)
    t_score_lse = timed(lambda: P.purekv_lowlayer_score_lse(q, k, lse, db, wl.window, c_out=c, status=status), 5)
    P.purekv_poll_status(status)
    # the decode step where it is bandwidth bound: many requests, each with a few thousand kept rows (synthetic cache)
    n_big, kept_big = 128, 4096

    class _Kept:
        h_cu_kept = np.arange(n_big + 1, dtype=np.int32) * kept_big
        cu_kept = torch.from_numpy(h_cu_kept.copy()).cuda()
    kc_big = torch.randn((n_big * kept_big, wl.n_kv_heads, wl.head_dim), device="cuda").to(torch.bfloat16)
    vc_big = torch.randn_like(kc_big)
    q_big = torch.randn((n_big, wl.n_q_heads, wl.head_dim), device="cuda").to(torch.bfloat16)
    o_big = torch.empty_like(q_big)
    ws_big = torch.empty(max(16, P.purekv_decode_ws_bytes(n_big, kept_big, wl.n_q_heads, wl.n_kv_heads, wl.head_dim)),
                         dtype=torch.uint8, device="cuda")
    t_big = timed(lambda: P.purekv_decode_attention(q_big, kc_big, vc_big, _Kept, out=o_big, ws=ws_big), 5)
    by_big = 2 * kc_big.numel() * 2 + 2 * q_big.numel() * 2
    decode_big = {"requests": n_big, "kept_per_request": kept_big, "heads": [wl.n_q_heads, wl.n_kv_heads], "ms": t_big,
                  "GBps": by_big / t_big / 1e6, "frac_hbm": by_big / t_big / 1e6 / hbm, "bytes": by_big}
    print(json.dumps({"sweep": wl.name, "tokens": b.total_tokens, "peak_TFLOPs": peak, "peak_kind": peak_kind + " burst (kernel timed alone)",
                      "prefill": rows, "score_ms": t_score, "score_one_pass_ms": t_score_lse,
                      "compression": comp, "decode_large_batch": decode_big,
                      "timing": "cold L2 (256 MiB fill before each call), median"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--cfg", type=int, default=1)
    ap.add_argument("--impl", default="purekv")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--print-kernel-hash", action="store_true", help="sha1 of the prefill kernel sources, then exit")
    ap.add_argument("--sweep", action="store_true", help="long-video workload: TFLOP/s against block density, compaction")
    args = ap.parse_args()
    if args.print_kernel_hash:
        print(kernel_source_sha1())
        return
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    if args.sweep:
        run_sweep(args)
        return
    from paper_2510_25600_b200 import inputs
    wl = inputs.workload(args.cfg)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2510_25600_b200 import binding as P
    from paper_2510_25600_b200.pipeline import PureKVPipeline

    world, rank, local = rank_env()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks, peak_kind = load_peaks()

    # ---- inputs: generated on the host from the seed, then resident in HBM -------------------------------
    b = wl.batch
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    kv_layers = max(wl.n_layers, wl.compacted_layers[-1] + 1)
    pipe = PureKVPipeline(b.seq_lens, b.n_prefix, b.n_frames, wl.mask, wl.n_layers, wl.n_q_heads, wl.n_kv_heads,
                          wl.head_dim, tdt, wl.scored_layers, wl.compacted_layers, wl.window, wl.keep_ratio, kv_layers)
    (hq, hk, hv), h_out = pipe.alloc_host_io()
    pool = ThreadPoolExecutor(len(os.sched_getaffinity(0)))
    keep_for_oracle = []
    for layer in range(kv_layers):
        x = inputs.make_qkv(wl, layer, which="qkv" if layer < wl.n_layers else "kv", pool=pool)
        key = "_bits" if wl.dtype == "bf16" else ""
        view = (lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)) if wl.dtype == "bf16" else torch.from_numpy
        if layer < wl.n_layers:
            hq[layer].copy_(view(x["q" + key]))
        hk[layer].copy_(view(x["k" + key]))
        hv[layer].copy_(view(x["v" + key]))
        if layer < 2:
            keep_for_oracle.append(x)
    d_in = tuple(t.cuda() for t in (hq, hk, hv))
    torch.cuda.synchronize()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing ---------------------------------------------------------------------------
    # per-launch events only in the warm-up passes (they tell dense from ST layers); in the timed region one event pair
    # per step spans the prefill launches, so consecutive launches still overlap their ramp and tail
    ev = lambda: torch.cuda.Event(enable_timing=True)
    events = [[(ev(), ev()) for _ in range(wl.n_layers)] for _ in range(args.warmup)]
    spans = [(ev(), ev()) for _ in range(args.steps)]
    for s in range(args.warmup):
        pipe.run_device(*d_in, events=events[s])
    pipe.check_status()
    sampler = ClockSampler(local)
    sampler.start()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        pipe.run_device(*d_in, span=spans[s])
    e1.record()
    sync_all()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    pipe.check_status()
    ms_step = max_over_ranks(ms_total, "cuda") / args.steps
    tokens = b.total_tokens
    value = job_throughput(tokens, world, ms_step * 1e-3)

    # ---- roofline of the dominant kernel (tensor-core prefill), from events around each launch -------------
    info_d, info_s = pipe.plan_dense.info, pipe.plan_st.info
    n_dense = pipe.clie + 1
    flops_tile = 4.0 * info_s.tile_q * info_s.tile_k * wl.head_dim * wl.n_q_heads
    flops_step = flops_tile * (n_dense * info_d.tiles_kept + (wl.n_layers - n_dense) * info_s.tiles_kept)
    k_ms = np.array([[p[0].elapsed_time(p[1]) for p in step] for step in events[1:]])     # [warm-up passes, layers]
    prefill_ms_step = float(np.mean([p[0].elapsed_time(p[1]) for p in spans]))          # timed region, all launches of a step
    achieved = flops_step / (prefill_ms_step * 1e-3) / 1e12
    peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    roofline = {"kernel": f"prefill_tc_kernel (128-key entries, skip granularity {info_s.tile_k})", "bound": "tensor", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak, "traffic": ncu_traffic(wl.name),
                "algorithmic_bytes_per_launch": b.total_tokens * wl.head_dim * 2 * (2 * wl.n_q_heads + 2 * wl.n_kv_heads),
                "peak_kind": f"{peak_kind} sustained cuBLAS bf16 (burst {peaks['bf16_tflops']}, nominal dense 2250)",
                "flops_per_step": flops_step, "launches_per_step": wl.n_layers, "avg_launch_ms": prefill_ms_step / wl.n_layers,
                "st_layer_ms_isolated": float(k_ms[:, n_dense:].mean()) if wl.n_layers > n_dense else None,
                "dense_layer_ms_isolated": float(k_ms[:, :n_dense].mean()),
                "tiles_kept_st": info_s.tiles_kept, "tiles_causal": info_s.tiles_causal,
                "useful_flops_per_step": 4.0 * wl.head_dim * wl.n_q_heads *
                (n_dense * info_d.pairs_kept + (wl.n_layers - n_dense) * info_s.pairs_kept)}

    # ---- per-step breakdown of the HBM-bound steps (separately timed, cold L2: inputs exceed L2) -----------
    def time_call(fn, reps=5):
        out = []
        for _ in range(reps):
            flush.zero_()
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            c.record()
            torch.cuda.synchronize()
            out.append(a.elapsed_time(c))
        return float(np.median(out))

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    q, k, v = d_in
    esz = 2 if wl.dtype == "bf16" else 4
    lo, hi = pipe.compacted[0], pipe.compacted[-1] + 1
    nc = hi - lo
    sl = pipe.scored[-1]
    if pipe.one_pass_scores:          # as the pipeline runs it: from the log-sum-exp the scored layer's prefill left
        t_score = time_call(lambda: P.purekv_lowlayer_score_lse(q[sl], k[sl], pipe.lse[len(pipe.scored) - 1], pipe.batch,
                                                                wl.window, c_out=pipe.c[0], status=pipe.status))
    else:
        t_score = time_call(lambda: P.purekv_lowlayer_score(q[sl], k[sl], pipe.batch, wl.window, c_out=pipe.c[0],
                                                            ws=pipe.score_ws))
    t_select = time_call(lambda: P.purekv_select_topk(pipe.c[len(pipe.scored) - 1], v[lo:hi], pipe.batch, pipe.budget,
                                                      idx_out=pipe.idx, ws=pipe.select_ws))
    t_compact = time_call(lambda: P.purekv_compact_kv(k[lo:hi], v[lo:hi], pipe.idx, pipe.batch, pipe.budget,
                                                      k_out=pipe.k_c, v_out=pipe.v_c))
    # what the compact cache is for: one decode step (one new query per request) over all compacted layers,
    # one call per layer; not part of the timed step or of `value`
    kept_max = int(np.diff(pipe.budget.h_cu_kept).max())
    q_dec = torch.randn((b.n_req, wl.n_q_heads, wl.head_dim), device="cuda").to(q.dtype)
    o_dec = torch.empty_like(q_dec)
    dec_need = P.purekv_decode_ws_bytes(b.n_req, kept_max, wl.n_q_heads, wl.n_kv_heads, wl.head_dim)
    dec_ws = torch.empty(max(16, dec_need), dtype=torch.uint8, device="cuda")

    def decode_all_layers():
        for layer in range(nc):
            P.purekv_decode_attention(q_dec, pipe.k_c[layer], pipe.v_c[layer], pipe.budget, out=o_dec, ws=dec_ws)
    decode_ok = wl.n_q_heads // wl.n_kv_heads <= 8 and wl.head_dim * (2 if wl.dtype == "bf16" else 4) == 256
    t_decode = time_call(decode_all_layers) if decode_ok else None
    t_plan = time.perf_counter()
    pipe.build_plans()
    t_plan = (time.perf_counter() - t_plan) * 1e3
    row = wl.n_kv_heads * wl.head_dim * esz
    kt = pipe.budget.total_kept
    bytes_score = tokens * row + min(wl.window, tokens) * wl.n_q_heads * wl.head_dim * esz * b.n_req + wl.n_kv_heads * tokens * 4
    bytes_select = nc * (tokens * row + wl.n_kv_heads * tokens * 4 + wl.n_kv_heads * kt * 4)
    bytes_compact = nc * (4 * kt * row + wl.n_kv_heads * kt * 4)
    hbm = float(peaks["hbm_gbs"])
    steps_detail = {
        "plan_build_ms": t_plan,
        "score": {"ms": t_score, "GBps": bytes_score / t_score / 1e6, "frac_hbm": bytes_score / t_score / 1e6 / hbm,
                  "kernel": "one pass, tcgen05, from the prefill's log-sum-exp" if pipe.one_pass_scores else "two passes",
                  "TFLOPs": (1 if pipe.one_pass_scores else 2) * 2.0 * wl.n_q_heads * min(wl.window, tokens) * tokens *
                  wl.head_dim / t_score / 1e9},
        "select": {"ms": t_select, "GBps": bytes_select / t_select / 1e6, "frac_hbm": bytes_select / t_select / 1e6 / hbm},
        "compact": {"ms": t_compact, "GBps": bytes_compact / t_compact / 1e6, "frac_hbm": bytes_compact / t_compact / 1e6 / hbm},
        "hbm_peak_GBps": hbm, "hbm_peak_kind": peak_kind, "timing": "cold L2 (256 MiB flush before each call), median of 5",
    }
    if t_decode is not None:
        bytes_decode = nc * (2 * kt * row + 2 * b.n_req * wl.n_q_heads * wl.head_dim * esz)
        steps_detail["decode_step_after"] = {
            "ms": t_decode, "launches": nc * (2 if dec_need else 1), "us_per_layer": 1e3 * t_decode / nc,
            "GBps": bytes_decode / t_decode / 1e6, "frac_hbm": bytes_decode / t_decode / 1e6 / hbm,
            "note": "one new query per request over the compact cache of every compacted layer, one call per layer; "
                    "outside the timed step"}

    # ---- end to end: pinned host inputs, compact cache read back ---------------------------------------------
    e2e = None
    if not args.no_e2e:
        n_e2e = max(3, min(args.steps, 10))
        pipe.run_host((hq, hk, hv), h_out, d_in)
        sync_all()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            pipe.run_host((hq, hk, hv), h_out, d_in)
        sync_all()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, "cuda")
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
        d2h = sum(t.numel() * t.element_size() for t in h_out)
        e2e = {"value": job_throughput(tokens, world, dt / n_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": 1e3 * dt / n_e2e}
    pipe.check_status()

    # ---- the oracle on this machine's host cores (rank 0, N = 1 only) ---------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import purekv_oracle as po
        po.build()
        v_cpu, cores, desc, _ = oracle_sample(wl, keep_for_oracle)
        cpu = {"value": v_cpu, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
                "config": {"workload": wl.name, "tokens": tokens, "layers": wl.n_layers, "heads": [wl.n_q_heads, wl.n_kv_heads],
                           "head_dim": wl.head_dim, "tile": wl.mask.tile, "window": wl.window, "keep_ratio": wl.keep_ratio,
                           "l2": "inputs larger than L2 (each layer reads its own Q/K/V; %.0f MB per step)" %
                                 (sum(t.numel() * t.element_size() for t in d_in) / 1e6),
                           "multi_gpu": "replicas only (the path has no exchange step)",
                           "step": "plan build + %d prefill layers + score + select + compact" % wl.n_layers},
                "clocks": clocks, "e2e": e2e, "gpu_launches": pipe.launches_per_step * args.steps,
                "roofline": roofline, "cpu_baseline": cpu, "steps_detail": steps_detail}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
