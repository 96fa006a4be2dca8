#!/usr/bin/env python
"""Benchmark of the FP8 ICL-attention hot path on B200.

One step = one pass of the whole path over one batch of synthetic input:
quantize Q_train, K, V (per-head absmax), quantize Q_test with the train-query
scale, then the fused train->train + test->train FP8 attention.  The metric is
tensor-core TFLOPS, 4*B*H*d*N*(N+M) FLOPs per step divided by the step time
(quantization included, as in the paper's latency tables).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no
exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

NOMINAL_FP8_OVER_BF16 = 2.0           # dense tensor peak ratio (4.5 / 2.25 PFLOP/s)
# exponentials per clock per SM: the 16-lane MUFU alone; with a share f of them on the FMA pipe
# the limit is 16 / (1 - f)
SOFTMAX_MUFU_PER_CLK_SM = 16.0


def fma_share_of_exponentials(w, sms: int) -> float:
    """Share of the FP8 kernel's exponentials that it evaluates by a polynomial on the FMA pipe:
    a quarter, or an eighth in the three-tile launches (d = 64, at least eight rounds of
    384-row blocks)."""
    blocks3 = w.B * w.H * (-(-w.n_train // 384) + -(-w.n_test // 384))
    return 0.125 if (w.d == 64 and blocks3 >= 8 * sms) else 0.25


def ncu_dram_traffic(workload: str):
    """DRAM bytes of one attention launch (dram__bytes_read.sum + dram__bytes_write.sum) from
    the ncu capture recorded under profiles/ for this workload, with the commit it was taken
    at; None where no capture exists."""
    path = os.path.join(ROOT, "profiles", f"icl_attention_fp8_{workload}_dram_traffic.txt")
    try:
        kv = {}
        with open(path) as f:
            for ln in f:
                if "=" in ln and not ln.lstrip().startswith("#"):
                    k, v = ln.split("=", 1)
                    kv[k.strip()] = v.strip()
        return {"bytes": float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"]),
                "captured_at_commit": kv.get("commit"), "launch": kv.get("launch")}
    except Exception:
        return None


FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return json.load(f), "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU while the timed region runs
    (one streaming ``nvidia-smi -lms 20`` child, read line by line)."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.sm, self.max_sm, self.reasons = [], 0.0, set()
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def run(self):
        if self.proc is None:
            return
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            try:
                self.sm.append(float(f[0]))
                self.max_sm = float(f[1])
            except (ValueError, IndexError):
                continue
            for name, val in zip(self.NAMES, f[2:]):
                if val.lower().startswith("active"):
                    self.reasons.add(name)

    def restart(self):
        """Forget the samples so far (the next ones belong to a new region)."""
        self.sm = []
        self.reasons = set()

    def snapshot(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.sm)), "sm_min_mhz": float(np.min(self.sm)),
                "sm_max_mhz": self.max_sm, "reasons": sorted(self.reasons), "samples": len(self.sm)}

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()          # our own child, by handle
            self.join(timeout=10)


def library_fp8_gemm_rate(seconds: float = 3.0, n: int = 8192):
    """Dense e4m3 GEMM rate of the vendor library on this GPU (TFLOP/s): best of 10 single
    calls and back-to-back calls for `seconds` under the power cap.  Context for the roofline
    only (what the tensor cores sustain on FP8 operands here); nothing on the timed path."""
    import time
    import torch
    a = (torch.randn(n, n, device="cuda") * 0.5).to(torch.float8_e4m3fn)
    b = (torch.randn(n, n, device="cuda") * 0.5).to(torch.float8_e4m3fn).t()
    one = torch.tensor(1.0, device="cuda")

    def gemm():
        return torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)

    for _ in range(3):
        gemm()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        gemm()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    calls, t0 = 0, time.time()
    e0.record()
    while time.time() - t0 < seconds:
        for _ in range(50):
            gemm()
        calls += 50
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    flop = 2.0 * n ** 3
    return flop / best / 1e9, flop * calls / e0.elapsed_time(e1) / 1e9


def oracle_sample(w, rows_per_head: int, seed: int = 0):
    """Time the CPU oracle, as it stands, on a bounded sample of workload ``w``:
    the full per-head quantization of K, V and both query tensors, then exact
    attention for ``rows_per_head`` train and test query rows per (b,h) against
    all train keys.  Returns (TFLOPS of the sampled attention rows, info)."""
    import oracle
    from paper_2609_13031_b200 import workloads as W
    oracle.build()
    g = W.generate(w)
    cores = oracle.hardware_threads()
    t0 = time.perf_counter()
    q8, sq = oracle.quantize(g["q_train"])
    k8, sk = oracle.quantize(g["k"])
    v8, sv = oracle.quantize(g["v"])
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq)
    t_quant = time.perf_counter() - t0
    rng = np.random.default_rng(seed)
    n_rows = 0
    t0 = time.perf_counter()
    for q, nq in ((q8, w.n_train), (t8, w.n_test)):
        if nq == 0:
            continue
        rows = np.unique(rng.integers(0, nq, size=min(rows_per_head, nq)))
        oracle.icl_attention_rows(q, k8, v8, rows, sq=sq, sk=sk, sv=sv)
        n_rows += rows.size * w.B * w.H
    t_attn = time.perf_counter() - t0
    flops = 4.0 * w.d * w.n_train * n_rows
    # quantization is charged in proportion to the sampled share of the query rows
    share = n_rows / float(w.B * w.H * (w.n_train + w.n_test))
    seconds = t_attn + t_quant * share
    info = {"cores": cores, "rows": int(n_rows), "seconds_attention": t_attn,
            "seconds_quantize_full": t_quant,
            "sample": f"{n_rows} query rows ({rows_per_head} train + {rows_per_head} test per head) "
                      f"against all {w.n_train} train keys of {w.name}, plus the sampled share of a "
                      f"full quantization pass"}
    return flops / seconds / 1e12, info


# one step of either arm: the same work, named the same way
STEP_LABEL = "quantize Q_train, K, V (per-head absmax) and Q_test (train-query scale), then ICL attention train->train + test->train"


def l2_label(w) -> str:
    """Timing hygiene: how the inputs of a step relate to the 126 MB L2 (no flush between steps
    where they exceed it; smaller workloads say so)."""
    mb = 2.0 * w.B * w.H * w.d * (3 * w.n_train + w.n_test) / 1e6
    return "bf16 inputs %.0f MB, %s the 126 MB L2; no flush between steps" % (mb, "larger than" if mb > 126 else "smaller than")


def workload_label(w) -> str:
    return f"{w.name}: B={w.B} H={w.H} d={w.d} n_train={w.n_train} n_test={w.n_test}"


def run_reference(args, w):
    """--impl reference: the CPU oracle, timed on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, info = [], None
    for i in range(args.warmup + args.steps):
        v, info = oracle_sample(w, args.ref_rows, seed=i)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    sec = info["seconds_attention"]
    print(json.dumps({
        "impl": "reference", "metric": "fp8_icl_attention_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sec, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_label(w), "step": STEP_LABEL, "l2": l2_label(w)},
        "impl_detail": "oracle quantize + exact attention over the dequantized operands, a bounded sample of "
                       "the step's query rows per timed step",
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": info["cores"], "kind": "oracle",
                         "sample": info["sample"]},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--rows", type=int, nargs=2, metavar=("N_TRAIN", "N_TEST"), default=None,
                    help="run the named workload's recipe at this many train / test rows (profiling on small cases)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-rows", type=int, default=96, help="oracle sample: query rows per head and call")
    ap.add_argument("--order-keys", default="auto", choices=["auto", "on", "off"],
                    help="quantize with fp8attn_quantize_qkv_ordered (the keys of largest norm first); auto: "
                         "from 32,768 train rows on, where its two extra launches cost under 1 %% of the step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-bf16", action="store_true")
    ap.add_argument("--no-fp8-gemm", action="store_true", help="skip the library FP8 GEMM rate (context figure)")
    ap.add_argument("--preroll", type=float, default=3.0,
                    help="seconds of untimed steps under the same load before each timed region, so that the "
                         "timed steps run at the clock the board's power limit settles on")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2609_13031_b200 import workloads as W
    w = W.CONFIGS[args.workload]
    if args.rows is not None:
        w = w.scaled(args.rows[0], args.rows[1])
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_13031_b200 import api, replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    api.load()                      # raises if the CUDA library is missing: no fallback
    peaks, peak_kind = load_peaks()

    # ---- inputs: seeded synthetic bf16 tensors, generated on the host into pinned memory ----
    host = {}
    for name, tid, rows in (("q_train", W.Q_TRAIN, w.n_train), ("k", W.K, w.n_train),
                            ("v", W.V, w.n_train), ("q_test", W.Q_TEST, w.n_test)):
        t = torch.empty((w.B, w.H, rows, w.d), dtype=torch.int16).pin_memory()
        W.fill(t.numpy().view(np.uint16), w, tid)
        host[name] = t.view(torch.bfloat16)
    dev = {k: torch.empty_like(v, device="cuda") for k, v in host.items()}
    for k in host:
        dev[k].copy_(host[k], non_blocking=True)
    # sized for FP8ATTN_SPLIT_TAIL, which both attention paths run with (it acts only on launches of
    # fewer than 8 CTAs per SM: C1 and C2 here; C3-C5 run exactly as without it)
    ws = api.new_workspace(w.B, w.H, n_train=w.n_train, n_test=w.n_test, d=w.d)
    fwd_flags = api.SPLIT_TAIL
    shape_tr, shape_te = (w.B, w.H, w.n_train, w.d), (w.B, w.H, w.n_test, w.d)
    buf = {
        "q8": torch.empty(shape_tr, dtype=torch.uint8, device="cuda"),
        "k8": torch.empty(shape_tr, dtype=torch.uint8, device="cuda"),
        "v8": torch.empty(shape_tr, dtype=torch.uint8, device="cuda"),
        "t8": torch.empty(shape_te, dtype=torch.uint8, device="cuda"),
        "sq": torch.empty((w.B, w.H), dtype=torch.float32, device="cuda"),
        "sk": torch.empty((w.B, w.H), dtype=torch.float32, device="cuda"),
        "sv": torch.empty((w.B, w.H), dtype=torch.float32, device="cuda"),
        "st": torch.empty((w.B, w.H), dtype=torch.float32, device="cuda"),
        "o_tr": torch.empty(shape_tr, dtype=torch.bfloat16, device="cuda"),
        "o_te": torch.empty(shape_te, dtype=torch.bfloat16, device="cuda"),
    }
    host_out = {"o_tr": torch.empty(shape_tr, dtype=torch.bfloat16).pin_memory(),
                "o_te": torch.empty(shape_te, dtype=torch.bfloat16).pin_memory()}

    order_keys = args.order_keys == "on" or (args.order_keys == "auto" and w.n_train >= 32768)
    if order_keys:
        buf["key_dest"] = torch.empty((w.B, w.H, w.n_train), dtype=torch.int32, device="cuda")

    def quantize_all():
        # all four quantizations (Q_train, K, V with their own scales; Q_test with Q_train's) in two
        # launches; with the key order, two more small launches and K8, V8 written in that order
        api.quantize_qkv(dev["q_train"], dev["k"], dev["v"], dev["q_test"], ws, out=buf, order_keys=order_keys)

    # the 16-bit comparison kernel runs on K, V in the same key order (reordered once, outside its timing)
    twin_kv = {"k": dev["k"], "v": dev["v"]}
    if order_keys and not args.no_bf16:
        quantize_all()
        twin_kv = {"k": api.reorder_rows(dev["k"], buf["key_dest"]), "v": api.reorder_rows(dev["v"], buf["key_dest"])}
        torch.cuda.synchronize()

    def attention_fp8():
        api.icl_forward_fp8(buf["q8"], buf["t8"], buf["k8"], buf["v8"], buf["sq"], buf["sk"], buf["sv"],
                            ws, 0.0, out_train=buf["o_tr"], out_test=buf["o_te"], flags=fwd_flags)

    def attention_bf16():
        api.icl_forward_bf16(dev["q_train"], dev["q_test"], twin_kv["k"], twin_kv["v"], ws, 0.0,
                             out_train=buf["o_tr"], out_test=buf["o_te"], flags=fwd_flags)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def max_over_ranks(ms: float) -> float:
        return replicas.max_over_ranks(ms, "cuda")

    # ---- device-resident timing: K steps, events per sub-kernel group ----
    for _ in range(args.warmup):
        quantize_all()
        attention_fp8()
    sync_all()
    status = api.last_device_status(ws)
    if status != (0, 0):
        raise RuntimeError(f"device status {status}")
    sampler = ClockSampler(local)
    sampler.start()

    def preroll(step_fn):
        """Untimed steps under the same load for at least --preroll seconds (at least one step):
        the timed steps then run at the clock that the power limit settles on, the state the
        sustained roofline denominator was measured in."""
        t0 = time.perf_counter()
        n = 0
        while True:
            step_fn()
            n += 1
            if n % 4 == 0 or n == 1:
                torch.cuda.synchronize()
                if time.perf_counter() - t0 >= args.preroll:
                    break
        torch.cuda.synchronize()
        return n, time.perf_counter() - t0

    def fp8_step():
        quantize_all()
        attention_fp8()

    pre_n, pre_s = preroll(fp8_step)
    sampler.restart()
    launches0 = api.launch_count()
    marks = []
    sync_all()
    e_start, e_end = ev(), ev()
    e_start.record()
    for _ in range(args.steps):
        a, b, c = ev(), ev(), ev()
        a.record()
        quantize_all()
        b.record()
        attention_fp8()
        c.record()
        marks.append((a, b, c))
    e_end.record()
    sync_all()
    launches = api.launch_count() - launches0
    clocks = sampler.snapshot()
    clocks["preroll_seconds"] = pre_s
    total_ms = max_over_ranks(e_start.elapsed_time(e_end))
    ms_step = total_ms / args.steps
    t_quant = np.array([a.elapsed_time(b) for a, b, _ in marks])
    t_attn = np.array([b.elapsed_time(c) for _, b, c in marks])
    ms_quant, ms_attn = float(np.mean(t_quant)), float(np.mean(t_attn))
    status = api.last_device_status(ws)
    if status != (0, 0):
        raise RuntimeError(f"device status {status}")

    # ---- the in-build BF16 path on the same inputs: same pre-roll, same number of launches ----
    ms_bf16, t_bf16, clocks_bf16 = None, None, None
    if not args.no_bf16:
        preroll(attention_bf16)
        sampler.restart()
        sync_all()
        bmarks = []
        for _ in range(args.steps):
            a, b = ev(), ev()
            a.record()
            attention_bf16()
            b.record()
            bmarks.append((a, b))
        sync_all()
        clocks_bf16 = sampler.snapshot()
        t_bf16 = np.array([a.elapsed_time(b) for a, b in bmarks])
        ms_bf16 = max_over_ranks(float(np.mean(t_bf16)))
    sampler.stop()

    # ---- end to end: the host-to-host call of the C-ABI (fp8attn_icl_step_host) ----
    # Every step hands pinned HOST tensors to the library and gets HOST results back; the call
    # copies in, quantizes, runs both attention calls and copies out, pipelined over chunks of
    # heads.  Throughput: steps alternate between two streams (own device scratch and own host
    # result buffers each), so that the copies of one step overlap the kernels of the other.
    shape = (w.B, w.H, w.n_train, w.n_test, w.d)
    host_flags = api.HOST_ORDER_KEYS if order_keys else 0
    n_slots = 2
    slots = []
    for _ in range(n_slots):
        slots.append({"stream": torch.cuda.Stream(),
                      "scratch": torch.empty(api.host_step_scratch_bytes(*shape, host_flags), dtype=torch.uint8, device="cuda"),
                      "o_tr": torch.empty_like(host_out["o_tr"]).pin_memory(),
                      "o_te": torch.empty_like(host_out["o_te"]).pin_memory()})

    def host_step(slot, flags=0, scratch=None):
        api.icl_step_host(host["q_train"], host["k"], host["v"], host["q_test"],
                          slot["scratch"] if scratch is None else scratch, flags=flags | host_flags,
                          out_train=slot["o_tr"], out_test=slot["o_te"])

    def e2e_run(n):
        for i in range(n):
            slot = slots[i % n_slots]
            with torch.cuda.stream(slot["stream"]):
                host_step(slot)

    def join_streams():
        cur = torch.cuda.current_stream()
        for slot in slots:
            cur.wait_stream(slot["stream"])

    sync_all()
    for slot in slots:
        slot["stream"].wait_stream(torch.cuda.current_stream())
    e2e_run(2)
    join_streams()
    sync_all()
    n_e2e = max(4, min(args.steps, 20))
    a, b = ev(), ev()
    a.record()
    for slot in slots:
        slot["stream"].wait_stream(torch.cuda.current_stream())
    e2e_run(n_e2e)
    join_streams()
    b.record()
    sync_all()
    ms_e2e = max_over_ranks(a.elapsed_time(b)) / n_e2e
    for slot in slots:
        st = api.host_step_status(slot["scratch"], *shape, host_flags)
        if st != (0, 0):
            raise RuntimeError(f"device status after the end-to-end steps: {st}")
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())
    # ---- one call, host to host, wall clock: the pipelined call, and the same call as one chunk ----
    def single_call(flags, scratch):
        ts = []
        for i in range(max(4, min(args.steps, 6))):
            sync_all()
            t0 = time.perf_counter()
            host_step(slots[0], flags=flags, scratch=scratch)
            torch.cuda.synchronize()
            if i > 0:                       # the first call of a kind pays its set-up
                ts.append(1e3 * (time.perf_counter() - t0))
        return max_over_ranks(float(np.median(ts)))

    ms_single = single_call(0, slots[0]["scratch"])
    slots[1]["scratch"] = None              # make room for the unpipelined call's larger scratch
    one_chunk = torch.empty(api.host_step_scratch_bytes(*shape, api.HOST_ONE_CHUNK | host_flags), dtype=torch.uint8,
                            device="cuda")
    ms_single_one_chunk = single_call(api.HOST_ONE_CHUNK, one_chunk)
    n_chunks = api.host_step_chunks(*shape, host_flags)
    del one_chunk

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N=1 only ----
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, info = oracle_sample(w, args.ref_rows)
        cpu_baseline = {"value": v, "unit": "TFLOP/s", "cores": info["cores"], "kind": "oracle",
                        "sample": info["sample"]}

    fp8_gemm = None
    if rank == 0 and world == 1 and not args.no_fp8_gemm:
        try:
            fp8_gemm = library_fp8_gemm_rate()
        except Exception as e:      # context figure only: report why it is missing
            fp8_gemm = str(e)[:120]

    if rank == 0:
        flops = w.flops
        tf = lambda ms: flops / (ms * 1e-3) / 1e12
        tf_step = world * tf(ms_step)
        tf_attn = tf(ms_attn)
        peak_fp8 = NOMINAL_FP8_OVER_BF16 * peaks["bf16_tflops_sustained"]
        peak_fp8_burst = NOMINAL_FP8_OVER_BF16 * peaks["bf16_tflops"]
        quant_bytes = w.B * w.H * w.d * (5 * 3 * w.n_train + 3 * w.n_test)
        if order_keys:
            # one more pass over K for the row norms, the norms written and read, the row map written and read twice
            quant_bytes += w.B * w.H * w.n_train * (2 * w.d + 4 * 5)
        # secondary roofline: the exponential path.  One exponential per score; the MUFU
        # evaluates 16 per clock per SM, and with the kernel's share of them on the FMA pipe
        # the limit is 16 / (1 - share).  Clock = the median SM clock sampled during the timed steps.
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        scores = float(w.B) * w.H * w.n_train * (w.n_train + w.n_test)
        softmax = None
        if clocks.get("sm_mhz"):
            per_clk_sm = scores / (ms_attn * 1e-3) / (sms * clocks["sm_mhz"] * 1e6)
            share = fma_share_of_exponentials(w, sms)
            softmax = {"scores_per_clk_per_sm": per_clk_sm,
                       "mufu_only_peak": SOFTMAX_MUFU_PER_CLK_SM,
                       "frac_of_mufu_only": per_clk_sm / SOFTMAX_MUFU_PER_CLK_SM,
                       "fma_share": share,
                       "with_fma_share_peak": SOFTMAX_MUFU_PER_CLK_SM / (1.0 - share),
                       "frac": per_clk_sm * (1.0 - share) / SOFTMAX_MUFU_PER_CLK_SM,
                       "clock_mhz": clocks["sm_mhz"], "sms": sms}
        traffic = ncu_dram_traffic(w.name)
        line = {
            "metric": "fp8_icl_attention_tflops", "value": tf_step, "unit": "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3",
            "data": "synthetic",
            "config": {"workload": workload_label(w), "step": STEP_LABEL, "l2": l2_label(w)},
            "impl_detail": {"calls": ("fp8attn_quantize_qkv_ordered" if order_keys else "fp8attn_quantize_qkv") +
                                     " (Q_train,K,V,Q_test) + fp8attn_icl_forward_ex (FP8ATTN_SPLIT_TAIL)",
                            "key_order": ("the keys of largest norm first (chosen and applied inside the timed quantization; "
                                          "the 16-bit comparison kernel runs on K, V in the same order)") if order_keys else "as given",
                            "preroll": "%d untimed steps (%.1f s) under the same load before the timed steps" % (pre_n, pre_s),
                            "replicas": world},
            "clocks": clocks,
            "e2e": {"value": world * tf(ms_e2e), "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
                    "kind": "fp8attn_icl_step_host on pinned host tensors, steps alternating between two streams "
                            "(copies of one step overlap the kernels of the other)",
                    "chunks_per_call": n_chunks,
                    "single_call_ms": ms_single, "single_call_value": world * tf(ms_single),
                    "single_call_kind": "median wall-clock latency of one fp8attn_icl_step_host call, host to host, "
                                        "synchronised before and after",
                    "single_call_one_chunk_ms": ms_single_one_chunk},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "kernel": "icl_attention_kernel<fp8>",
                         "achieved": tf_attn, "peak": peak_fp8, "unit": "TFLOP/s",
                         "frac": tf_attn / peak_fp8,
                         "achieved_median": tf(float(np.median(t_attn))),
                         "achieved_best": tf(float(np.min(t_attn))),
                         "traffic": None if traffic is None else traffic["bytes"],
                         "traffic_source": traffic,
                         "peak_source": f"2 x bf16_tflops_sustained ({peak_kind}), nominal fp8:bf16 ratio; the timed "
                                        "steps follow a pre-roll under load, i.e. the sustained clock state",
                         "frac_of_burst_peak": tf_attn / peak_fp8_burst,
                         "frac_of_nominal_4500": tf_attn / 4500.0,
                         "softmax": softmax,
                         "library_fp8_gemm_tflops": None if not isinstance(fp8_gemm, tuple) else
                         {"burst": fp8_gemm[0], "sustained": fp8_gemm[1],
                          "how": "torch._scaled_mm e4m3 8192^3, best of 10 / back to back for 3 s, same run"},
                         "frac_of_library_fp8_gemm_sustained": None if not isinstance(fp8_gemm, tuple)
                         else tf_attn / fp8_gemm[1],
                         "library_fp8_gemm_error": fp8_gemm if isinstance(fp8_gemm, str) else None},
            "cpu_baseline": cpu_baseline,
            "breakdown": {
                "ms_quantize": ms_quant, "ms_attention_fp8": ms_attn, "ms_attention_bf16": ms_bf16,
                "ms_attention_fp8_median": float(np.median(t_attn)), "ms_attention_fp8_best": float(np.min(t_attn)),
                "ms_attention_bf16_median": None if t_bf16 is None else float(np.median(t_bf16)),
                "ms_attention_bf16_best": None if t_bf16 is None else float(np.min(t_bf16)),
                "ms_quantize_median": float(np.median(t_quant)), "ms_quantize_best": float(np.min(t_quant)),
                "clocks_bf16": clocks_bf16,
                "attention_fp8_tflops": tf_attn,
                "attention_bf16_tflops": None if ms_bf16 is None else tf(ms_bf16),
                "speedup_vs_bf16_attention_only": None if ms_bf16 is None else ms_bf16 / ms_attn,
                "speedup_vs_bf16_with_quantize": None if ms_bf16 is None else ms_bf16 / (ms_attn + ms_quant),
                "quantize_gbs": quant_bytes / (ms_quant * 1e-3) / 1e9,
                "quantize_frac_of_hbm": quant_bytes / (ms_quant * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "paper_context": "up to 1.72x (d=64) / 1.82x (d=128) FP8 over 16-bit kernels on RTX PRO 6000",
            },
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
