#!/usr/bin/env python
"""Benchmark: compress + attend tokens/s on one B200 (or N independent replicas).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference]

A step is one pass of the whole hot path (elm_compress then elm_attend) over one batch of
seeded synthetic input already resident in HBM.  Rank 0 prints one JSON line.  The path has no
exchange step, so N > 1 runs N independent replicas ("replicas only") and adds their tokens.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of one attend launch at the workload's full size, from one
# single-pass ncu capture of that launch (bf16: read 1 083 738 880 + write 1 024 521 216 bytes; E4M3 storage:
# read 543 735 808 + write 1 019 808 000); workloads without a capture report null and say so
NCU_DRAM_BYTES_PER_ATTEND_LAUNCH = {"cfg5": 1083738880 + 1024521216, "cfg5[storage=e4m3]": 543735808 + 1019808000}

METRIC = "compress+attend tokens/sec per B200"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return {"hbm_gbs": pk["hbm_gbs"], "bf16_tflops": pk["bf16_tflops"],
                "bf16_tflops_sustained": pk.get("bf16_tflops_sustained", pk["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self._stop = threading.Event()
        self._thr = None

    def _nvml_loop(self):
        """Read-only NVML polling every 2 ms (an nvidia-smi call takes longer than the timed region)."""
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(self.gpu)
        mx = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
        bits = {"hw_slowdown": pynvml.nvmlClocksEventReasonHwSlowdown,
                "hw_thermal_slowdown": pynvml.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": pynvml.nvmlClocksEventReasonSwThermalSlowdown,
                "sw_power_cap": pynvml.nvmlClocksEventReasonSwPowerCap}
        while not self._stop.is_set():
            sm = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
            r = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
            pw = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
            self.rows.append([str(sm), str(mx), str(pw)] + ["Active" if r & b else "Not Active" for b in bits.values()])
            self._stop.wait(0.002)

    def _run(self):
        try:
            self._nvml_loop()
            return
        except Exception:
            pass
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                     timeout=5).stdout.strip()
                if out:
                    self.rows.append([c.strip() for c in out.splitlines()[0].split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thr.join(timeout=10)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        power = []
        for r in self.rows:
            try:
                power.append(float(r[2]))
            except (ValueError, IndexError):
                pass
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


def max_over_ranks(ms_local: float, dist, device) -> float:
    """The slowest rank's time (every rank gets it); `dist` is None for a single process."""
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank processes its own batch, the job's tokens add up."""
    return tokens_per_rank_step * world / (ms_per_step * 1e-3)


def algorithmic_counts(wl):
    """Flops and bytes the method itself needs per step (not what exact attention would need)."""
    es = {"bf16": 2, "e4m3": 1}.get(wl.dtype, 4)
    eo = 2 if wl.dtype == "e4m3" else es                      # O is bf16 for 8-bit inputs
    attend_flops = wl.batch * wl.q_heads * wl.n_q * wl.n_out * 4 * wl.d
    compress_flops = wl.batch * wl.kv_heads * wl.m * 8 * wl.d * wl.n_out ** 2
    hbm_bytes = wl.batch * wl.q_heads * wl.n_q * wl.d * (es + eo) + 2 * wl.batch * wl.kv_heads * wl.n * wl.d * es
    return attend_flops, compress_flops, hbm_bytes


def cpu_baseline(wl, Q, K, V, budget_heads=None):
    """The oracle as it stands, timed on this machine's cores on a bounded sample of the workload."""
    import numpy as np
    import oracle
    from paper_2606_10944_b200.workloads import as_f32_numpy
    cores = oracle.num_threads()
    problems = wl.batch * wl.kv_heads
    # compression cost per problem ~ 3 m n_out^2 kernel evaluations of 2d MACs; aim for <= ~20 s
    per_problem_s = 3.0 * wl.m * wl.n_out ** 2 * 2 * wl.d / 0.6e9
    waves = max(1, int(20.0 / max(per_problem_s, 1e-3)))
    heads = budget_heads or max(1, min(problems, cores * waves))
    Kf = as_f32_numpy(K).reshape(problems, wl.n, wl.d)[:heads]
    Vf = as_f32_numpy(V).reshape(problems, wl.n, wl.d)[:heads]
    t0 = time.perf_counter()
    idx, w, _ = oracle.compress2_batched(Kf, Vf, wl.log2_nout, wl.m, seed=1)
    t_c = time.perf_counter() - t0
    # attention: a fixed number of query rows of every query head (~0.5 us per coreset point)
    per_query_s = wl.n_out * 2 * wl.d / 0.6e9
    nq_s = int(max(8, min(wl.n_q, 8.0 * cores / (per_query_s * wl.batch * wl.q_heads))))
    Qf = as_f32_numpy(Q[:, :, :nq_s])
    Kall = as_f32_numpy(K)
    Vall = as_f32_numpy(V)
    # every query head needs a coreset for its KV head: reuse the sampled ones cyclically
    full_idx = np.stack([idx[i % heads] for i in range(problems)]).reshape(wl.batch, wl.kv_heads, -1)
    full_w = np.stack([w[i % heads] for i in range(problems)]).reshape(wl.batch, wl.kv_heads, -1)
    t0 = time.perf_counter()
    oracle.wtd_attention_batched(Qf, Kall, Vall, full_idx, full_w)
    t_a = time.perf_counter() - t0
    est = t_c * problems / heads + t_a * wl.n_q / nq_s
    return {"value": wl.batch * wl.n / est, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"compress of {heads}/{problems} KV problems at full n={wl.n} ({t_c:.2f} s) + attend of "
                      f"{nq_s}/{wl.n_q} query rows of all {wl.batch * wl.q_heads} query heads ({t_a:.2f} s), "
                      f"scaled linearly to the full step ({est:.1f} s)"}, est


def oracle_cfg1_one_thread_ms():
    """The oracle on the smallest workload (one attention problem, so one thread): full compress + attend."""
    import oracle
    from paper_2606_10944_b200.workloads import WORKLOADS, as_f32_numpy, generate
    w1 = WORKLOADS["cfg1"]
    Q, K, V = generate(w1, seed=1234)
    Qf, Kf, Vf = as_f32_numpy(Q), as_f32_numpy(K), as_f32_numpy(V)
    best = None
    for _ in range(3):
        t0 = time.perf_counter()
        idx, w, _ = oracle.compress2_batched(Kf.reshape(1, w1.n, w1.d), Vf.reshape(1, w1.n, w1.d), w1.log2_nout, w1.m, seed=1)
        oracle.wtd_attention_batched(Qf, Kf, Vf, idx.reshape(1, 1, -1), w.reshape(1, 1, -1))
        dt = (time.perf_counter() - t0) * 1e3
        best = dt if best is None else min(best, dt)
    return best


def run_reference(args, wl):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2606_10944_b200.workloads import generate
    Q, K, V = generate(wl, seed=args.data_seed)
    times = []
    base = None
    for i in range(args.warmup + args.steps):
        base, est = cpu_baseline(wl, Q, K, V, budget_heads=args.ref_heads)
        if i >= args.warmup:
            times.append(est)
        if sum(times) > 0 and (time.perf_counter() - T_START) > 240:
            break
    est = sum(times) / len(times)
    value = wl.batch * wl.n / est
    base["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(times), "warmup": args.warmup, "ms_per_step": est * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args), "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(wl, args):
    return {"workload": wl.name, "batch": wl.batch, "q_heads": wl.q_heads, "kv_heads": wl.kv_heads,
            "seq_len": wl.n, "head_dim": wl.d, "n_out": wl.n_out, "compress2_depth": wl.m, "g": wl.g,
            "storage": wl.dtype, "precision": args.precision, "recipe": wl.recipe,
            "parallelism": "replicas only", "l2": "inputs (>= 2.6 GB per step) exceed the 126 MB L2"
            if wl.name.startswith(("cfg5", "cfg4")) else "L2 flushed by a 256 MB write between steps"}


T_START = time.perf_counter()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--precision", default="fp32", choices=["fp32", "fp64"])
    ap.add_argument("--storage", default=None, choices=["f32", "bf16", "e4m3"],
                    help="storage type of Q, K, V instead of the workload's own (e4m3: 8-bit inputs, d = 128, O in bf16; "
                         "S = Q K^T then runs on 8-bit tensor-core operands)")
    ap.add_argument("--data-seed", type=int, default=1234)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-heads", type=int, default=None)
    ap.add_argument("--override", default="", help="comma list of Workload fields for small profiling "
                    "captures, e.g. q_heads=8,kv_heads=2,n=32768,n_q=32768 (the line then names the scaled case)")
    ap.add_argument("--only", default="both", choices=["both", "compress", "attend", "express", "prefill", "decode", "stream", "ragged"],
                    help="run one half of the step; or, instead of the step, the Offline-Express compression "
                         "(express) or the Thinformer Express prefill (prefill) of the same inputs with "
                         "mbar = log2(n_out) - 2; or (decode) one query per head over a cache of n_out and of "
                         "6 n_out entries, printed as its own JSON line (profiling captures only); or (ragged) "
                         "compress + attend on a sequence 7 %% shorter than the workload's, 32 sink and 32 "
                         "window rows kept (elm_compress_ragged)")
    ap.add_argument("--sustain-s", type=float, default=3.0,
                    help="seconds of back-to-back attend launches for the sustained-clock figure (0: skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()

    from paper_2606_10944_b200.workloads import WORKLOADS, generate
    wl = WORKLOADS[args.workload]
    if args.override:
        kv = dict(item.split("=") for item in args.override.split(","))
        wl = wl.scaled(name=f"{wl.name}[{args.override}]", **{k: int(v) for k, v in kv.items()})
    if args.storage and args.storage != wl.dtype:
        wl = wl.scaled(name=f"{wl.name}[storage={args.storage}]", dtype=args.storage)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import paper_2606_10944_b200 as elm

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    elm.load_library()
    warmup = max(args.warmup, 3)

    Q, K, V = generate(wl, seed=args.data_seed + rank)      # each replica has its own batch
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    dev = Qd.device
    dcode = {"f32": 0, "bf16": 1, "e4m3": 2}[wl.dtype]
    p, _ = elm.make_params(wl.batch, wl.q_heads, wl.kv_heads, wl.n, wl.n_q, wl.d, wl.log2_nout, wl.m, dcode, args.precision)
    cb, ab = elm.workspace_bytes(p)
    ws_c = torch.empty(cb, dtype=torch.uint8, device=dev)
    ws_a = torch.empty(ab, dtype=torch.uint8, device=dev)
    O = torch.empty(Qd.shape, dtype=torch.bfloat16 if wl.dtype == "e4m3" else Qd.dtype, device=dev)
    if wl.dtype == "e4m3":
        args.no_e2e = True          # the host-buffer entry point takes f32 and bf16 only
    small_inputs = not wl.name.startswith(("cfg4", "cfg5"))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small_inputs else None

    if args.only == "stream":
        # streaming Thinformer Express, one token per call, over the first tokens of the workload
        T = min(wl.n, 10 * wl.n_out)
        st = elm.Stream(Kd, Vd, wl.q_heads, wl.log2_nout, wl.log2_nout - 2, seed=args.seed, precision=args.precision)
        # [T, B, Hq, 1, d]: the tokens' queries one after the other; two library calls (elm_stream_steps), the
        # exact regime (4 n_out tokens) and the rest
        q_T = Qd[:, :, :T, :].permute(2, 0, 1, 3).unsqueeze(3).contiguous()
        o_T = torch.empty_like(q_T)
        torch.cuda.synchronize()
        marks = {}
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.perf_counter()
        e0.record()
        for lo, hi in ((0, 4 * wl.n_out), (4 * wl.n_out, T)):
            st.steps(q_T[lo:hi], out=o_T[lo:hi])
            torch.cuda.synchronize()
            marks[hi] = time.perf_counter() - w0
        e1.record()
        torch.cuda.synchronize()
        if rank == 0:
            print(json.dumps({"stream": {"tokens": T, "ms_total": e0.elapsed_time(e1),
                                         "us_per_token_first_4nout": marks[4 * wl.n_out] / (4 * wl.n_out) * 1e6,
                                         "us_per_token_after": (marks[T] - marks[4 * wl.n_out]) / (T - 4 * wl.n_out) * 1e6,
                                         "cache_entries_at_end": int(st.cache()[0].shape[-1])},
                              "config": workload_config(wl, args)}))
        return

    if args.only == "ragged":
        # a length that is not n_out 2^m: Algorithm 2 leaves points in every level; 32 + 32 rows kept exactly
        n_r = wl.n - wl.n // 14 - 37
        Kr, Vr = Kd[:, :, :n_r, :].contiguous(), Vd[:, :, :n_r, :].contiguous()
        Qr = Qd[:, :, :min(n_r, wl.n_q), :].contiguous()
        Or = torch.empty_like(Qr)
        pr, _ = elm.make_params(wl.batch, wl.q_heads, wl.kv_heads, n_r, Qr.shape[2], wl.d, wl.log2_nout, wl.m,
                                1 if wl.dtype == "bf16" else 0, args.precision)
        count, need = elm.compress_ragged_count(pr, 32, 32)
        ws_r = torch.empty(need, dtype=torch.uint8, device=dev)
        ws_ar = torch.empty(elm.attend_workspace_bytes(pr, count), dtype=torch.uint8, device=dev)

        def ragged_step(seed):
            idx, w = elm.compress_ragged(Kr, Vr, wl.log2_nout, wl.m, 32, 32, seed=seed, precision=args.precision,
                                         workspace=ws_r)
            elm.attend(Qr, Kr, Vr, idx, w, precision=args.precision, workspace=ws_ar, out=Or)

        for i in range(warmup):
            ragged_step(args.seed + i)
        torch.cuda.synchronize()
        elm.profile_enable(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.steps):
            ragged_step(args.seed + warmup + i)
        e1.record()
        torch.cuda.synchronize()
        prof = elm.profile_read()
        elm.profile_enable(False)
        ms = e0.elapsed_time(e1) / args.steps
        if rank == 0:
            print(json.dumps({"ragged": {"n": n_r, "n_sink": 32, "n_window": 32, "cache_entries": count,
                                         "ms_per_step": ms, "tokens_per_s": wl.batch * n_r / (ms * 1e-3),
                                         "stage_ms": {k: v[0] / args.steps for k, v in prof.items()}},
                              "config": workload_config(wl, args)}))
        return

    if args.only == "decode":
        # one new token per head over a weighted cache: HBM-bound; bytes = the cache rows of K and V once
        peaks = load_peaks()
        es = 2 if wl.dtype == "bf16" else 4
        q1 = Qd[:, :, :1, :].contiguous()
        out = []
        for n_core in (wl.n_out, 6 * wl.n_out):
            g = torch.Generator().manual_seed(7)
            idx = torch.stack([torch.randperm(wl.n, generator=g)[:n_core] for _ in range(wl.batch * wl.kv_heads)])
            idx = idx.reshape(wl.batch, wl.kv_heads, n_core).to(torch.int32).cuda()
            w = (torch.rand(wl.batch, wl.kv_heads, n_core, generator=g) + 0.05).cuda()
            p1, _ = elm.make_params(wl.batch, wl.q_heads, wl.kv_heads, wl.n, 1, wl.d, wl.log2_nout, wl.m,
                                    1 if wl.dtype == "bf16" else 0, args.precision)
            ws1 = torch.empty(elm.attend_workspace_bytes(p1, n_core), dtype=torch.uint8, device=dev)
            o1 = torch.empty_like(q1)
            for _ in range(warmup):
                elm.attend(q1, Kd, Vd, idx, w, precision=args.precision, workspace=ws1, out=o1)
            reps = max(args.steps, 20)
            big = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

            # device time from the library's own stage events (recorded around the two launches of a
            # call on its stream): the Python call itself takes longer than the kernels
            elm.profile_enable(True)
            for _ in range(reps):
                big.zero_()                                      # the cache rows leave L2 between tokens
                elm.attend(q1, Kd, Vd, idx, w, precision=args.precision, workspace=ws1, out=o1)
            torch.cuda.synchronize()
            total = elm.profile_read()["attend"][0]
            elm.profile_enable(False)
            us = total / reps * 1e3
            nbytes = wl.batch * wl.kv_heads * n_core * (2 * wl.d * es + 8)
            gbs = nbytes / (us * 1e-6) / 1e9
            out.append({"n_core": n_core, "us_per_token": us, "algorithmic_bytes": nbytes, "achieved_GBps": gbs,
                        "frac_of_measured_hbm": gbs / peaks["hbm_gbs"]})
        if rank == 0:
            print(json.dumps({"decode": out, "config": workload_config(wl, args), "l2": "256 MiB written between tokens"}))
        return

    state = {}

    def step(seed):
        if flush is not None:
            flush.zero_()
        if args.only == "prefill":
            elm.express_prefill(Qd, Kd, Vd, wl.log2_nout, wl.log2_nout - 2, seed=seed, precision=args.precision,
                                workspace=state.setdefault("ws_p", None), out=O)
            return
        if args.only == "express":
            state["idx"], state["w"] = elm.express_compress(Kd, Vd, wl.log2_nout, wl.log2_nout - 2, seed=seed,
                                                            precision=args.precision, workspace=state.get("ws_x"))
            return
        if args.only != "attend" or "idx" not in state:
            state["idx"], state["w"] = elm.compress(Kd, Vd, wl.log2_nout, wl.m, seed=seed, precision=args.precision,
                                                    workspace=ws_c)
        if args.only != "compress":
            elm.attend(Qd, Kd, Vd, state["idx"], state["w"], precision=args.precision, workspace=ws_a, out=O)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        step(args.seed + i)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush_ms = 0.0
    if flush is not None:           # cost of the flush itself, subtracted below
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.steps):
            flush.zero_()
        f1.record()
        torch.cuda.synchronize()
        flush_ms = f0.elapsed_time(f1)
    launches0 = elm.launch_count()
    # Inside the timed region only the dominant kernel's stage (attend) is bracketed by the library's events - the
    # roofline's numerator.  Events around every stage would sit between the compression's short dependent
    # launches and cost a tenth of its time, so the other stages are timed in a pass of their own afterwards.
    elm.profile_enable(2)
    with ClockSampler(local) as clocks:
        barrier()
        ev0.record()
        for i in range(args.steps):
            step(args.seed + i)
        ev1.record()
        barrier()
    stage = elm.profile_read()
    elm.profile_enable(False)
    launches = elm.launch_count() - launches0
    elm.profile_enable(1)
    barrier()
    for i in range(args.steps):
        step(args.seed + i)
    barrier()
    stage_all = elm.profile_read()
    elm.profile_enable(False)
    for k in stage_all:
        if k != "attend":
            stage[k] = stage_all[k]
    ms_total = max_over_ranks(ev0.elapsed_time(ev1) - flush_ms, dist, dev)
    ms_step = ms_total / args.steps
    tokens_per_step = wl.batch * wl.n * world
    value = whole_job_tokens_per_s(wl.batch * wl.n, world, ms_step)

    # end to end through the host-buffer entry point (pinned inputs, copies inside the timed region)
    e2e = None
    if not args.no_e2e and args.only not in ("prefill", "express"):
        Qp, Kp, Vp = Q.pin_memory(), K.pin_memory(), V.pin_memory()
        Oh = torch.empty_like(Q).pin_memory()
        scratch = torch.empty(elm.host_call_scratch_bytes(wl.batch, wl.q_heads, wl.kv_heads, wl.n, wl.n_q, wl.d,
                                                          wl.log2_nout, wl.m, Q.dtype, args.precision),
                              dtype=torch.uint8, device=dev)
        elm.compress_attend_host(Qp, Kp, Vp, wl.log2_nout, wl.m, seed=args.seed, precision=args.precision,
                                 scratch=scratch, out=Oh)
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for i in range(args.e2e_steps):
            elm.compress_attend_host(Qp, Kp, Vp, wl.log2_nout, wl.m, seed=args.seed + i,
                                     precision=args.precision, scratch=scratch, out=Oh)
        g1.record()
        barrier()
        e2e_ms = max_over_ranks(g0.elapsed_time(g1), dist, dev) / args.e2e_steps
        e2e = {"value": tokens_per_step / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": Q.numel() * Q.element_size() + 2 * K.numel() * K.element_size(),
               "d2h_bytes_per_step": Q.numel() * Q.element_size(), "steps": args.e2e_steps}
        del scratch

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    if args.only in ("prefill", "express"):
        # not the step of the headline metric: its own line (profiling captures only)
        what = "Thinformer Express prefill" if args.only == "prefill" else "Offline-Express compression"
        print(json.dumps({args.only: {"what": what, "mbar": wl.log2_nout - 2, "ms_per_call": ms_step,
                                      "tokens_per_s": value, "launches_per_call": launches // args.steps,
                                      "stage_ms": {k: v[0] / args.steps for k, v in stage.items()}},
                          "n_gpus": world, "steps": args.steps, "warmup": warmup,
                          "config": workload_config(wl, args)}))
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    attend_flops, compress_flops, hbm_bytes = algorithmic_counts(wl)
    stage_ms = {k: v[0] / args.steps for k, v in stage.items()}
    att_ms = stage_ms["attend"] or float("nan")     # zero only under --only compress
    clk = clocks.summary()
    # Which measured GEMM peak the tensor fractions are read against: the burst figure was taken on a kernel
    # timed alone at full clocks, the sustained one inside a seconds-long loop under the power cap.  A timed
    # region of well under a second at (nearly) the maximum SM clock never enters that regime, so the burst
    # peak is the denominator then; both fractions are printed either way.
    region_s = ms_total * 1e-3
    at_full_clock = clk["sm_mhz"] is not None and clk["sm_mhz"] >= 0.95 * clk["sm_max_mhz"]
    use_burst = region_s < 1.0 and at_full_clock
    tensor_peak = peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"]
    peak_name = "burst" if use_burst else "sustained"
    # 8-bit inputs: half of attend's flops (S = Q K^T) run at the 8-bit rate, nominally twice the bf16 rate, the
    # other half (P V) at the bf16 rate: the blended peak for the whole contraction is 4/3 of the bf16 figure
    fp8 = wl.dtype == "e4m3"
    blend = 4.0 / 3.0 if fp8 else 1.0
    tensor_peak *= blend
    # the dominant kernel: weighted attention (dense contraction -> tensor roofline) unless the
    # workload's coreset is so small that its Q/O traffic dominates
    t_tensor = attend_flops / (tensor_peak * 1e12)
    att_bytes = wl.batch * wl.q_heads * wl.n_q * wl.d * ({"bf16": 4, "e4m3": 3}.get(wl.dtype, 8))
    t_hbm = att_bytes / (peaks["hbm_gbs"] * 1e9)
    if wl.dtype in ("bf16", "e4m3") and t_tensor >= t_hbm:
        achieved = attend_flops / (att_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "attend", "achieved": achieved, "peak": tensor_peak,
                    "unit": "TFLOP/s", "frac": achieved / tensor_peak, "traffic": None,
                    "peak_source": f"{peaks['source']} bf16 {peak_name} ({region_s:.2f} s timed region at "
                                   f"{clk['sm_mhz']} of {clk['sm_max_mhz']} MHz)",
                    "frac_burst": achieved / (peaks["bf16_tflops"] * blend),
                    "frac_sustained": achieved / (peaks["bf16_tflops_sustained"] * blend), "ms_per_launch": att_ms}
        if fp8:
            roofline["peak_source"] += "; x 4/3: S = Q K^T at the nominal 2x rate of 8-bit operands, P V at the bf16 rate"
    else:
        achieved = att_bytes / (att_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "attend", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                    "peak_source": f"{peaks['source']} copy", "ms_per_launch": att_ms}
    roofline["traffic"] = NCU_DRAM_BYTES_PER_ATTEND_LAUNCH.get(wl.name)
    if roofline["traffic"] is None:
        roofline["traffic_note"] = "no ncu capture of this workload's attend launch"
    whole_burst_s = max((attend_flops / blend + compress_flops) / (peaks["bf16_tflops"] * 1e12), hbm_bytes / (peaks["hbm_gbs"] * 1e9))
    whole_sust_s = max((attend_flops / blend + compress_flops) / (peaks["bf16_tflops_sustained"] * 1e12),
                       hbm_bytes / (peaks["hbm_gbs"] * 1e9))
    whole_roof_s = whole_burst_s if use_burst else whole_sust_s

    # The same attend launch back to back for a few seconds, clocks sampled throughout: the like-for-like
    # numerator for the sustained peak (and time x clock, which does not depend on where the clock settles).
    sustained = None
    if args.sustain_s > 0 and args.only in ("both", "attend") and roofline["bound"] == "tensor":
        reps = max(8, int(args.sustain_s * 1e3 / att_ms))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(local) as sclk:
            torch.cuda.synchronize()
            s0.record()
            for _ in range(reps):
                elm.attend(Qd, Kd, Vd, state["idx"], state["w"], precision=args.precision, workspace=ws_a, out=O)
            s1.record()
            torch.cuda.synchronize()
        sms = s0.elapsed_time(s1) / reps
        sc = sclk.summary()
        ach = attend_flops / (sms * 1e-3) / 1e12
        sustained = {"launches": reps, "seconds": s0.elapsed_time(s1) * 1e-3, "ms_per_launch": sms, "achieved": ach,
                     "unit": "TFLOP/s", "frac_sustained": ach / (peaks["bf16_tflops_sustained"] * blend),
                     "frac_burst": ach / (peaks["bf16_tflops"] * blend), "clocks": sc,
                     "ms_x_mhz": sms * sc["sm_mhz"] if sc["sm_mhz"] else None}
        roofline["ms_x_mhz"] = att_ms * clk["sm_mhz"] if clk["sm_mhz"] else None

    base = None
    if not args.no_cpu_baseline:
        base, _ = cpu_baseline(wl, Q, K, V)
        base["cfg1_one_thread_ms"] = oracle_cfg1_one_thread_ms()

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"bf16": "bf16", "e4m3": "e4m3 (Q K^T) / bf16 (P V)"}.get(wl.dtype, "f32"), "data": "synthetic",
        "config": workload_config(wl, args),
        "roofline": roofline,
        "whole_path_roofline": {"roofline_ms": whole_roof_s * 1e3, "frac": whole_roof_s * 1e3 / ms_step,
                                "frac_burst": whole_burst_s * 1e3 / ms_step, "frac_sustained": whole_sust_s * 1e3 / ms_step,
                                "attend_flops": attend_flops, "compress_flops": compress_flops,
                                "hbm_bytes": hbm_bytes},
        "attend_sustained": sustained,
        "stage_ms": stage_ms,
        "stage_ms_note": "attend: the library's events inside the timed region; the other stages: a second pass of the same steps with events around every stage (which slows the compression's short launches, so they sum to more than the step leaves for them)",
        "cpu_baseline": base,
        "e2e": e2e,
        "gpu_launches": launches,
        "clocks": clk,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
