#!/usr/bin/env python
"""Benchmark of the V step (select -> re-encode -> dequantise) on synthetic layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one whole V step over one layer: pvt_vstep_select, pvt_vstep_encode
and pvt_dequant through the C ABI.  Default workload: a 4096 x 4096 fp32 layer,
one fp16 codebook of 65536 codewords (group size 8), tau = 0.01.  With N > 1
(launched by torch.distributed.run) every rank steps its own layer of the same
shape (layers are independent problems: no collective on the data path); the
reported value is the work of all ranks over the slowest rank's time.

Prints ONE JSON line on rank 0.
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

METRIC = "vstep_reencoded_groups_per_s"
UNIT = "groups/s"
FP32_LANES_PER_SM = 128  # FP32 FMA lanes of one sm_100 multiprocessor
FLOP_PER_PAIR = 16       # one codeword-pair evaluation = a dot product of 8 elements


def workloads():
    from paper_2405_14852_b200 import synth
    out = {}
    for cfg, entries in synth.CONFIGS.items():
        for which, e in enumerate(entries):
            for tau in e[7]:
                out[f"{e[0]}_tau{tau}"] = (cfg, which, tau)
    return out


DEFAULT_WORKLOAD = "llama2_7b_attn_4096x4096_1x16_tau0.01"


# --------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax = float(f[1])
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        # the busy samples are the upper half: idle gaps between steps pull the clock down
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax, "samples": len(sm),
                "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- our arm


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2405_14852_b200 import binding as B
    from paper_2405_14852_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the V step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg, which, tau = workloads()[args.workload]
    name, rows, cols, M, K, f16, rowmax, _ = synth.CONFIGS[cfg][which]
    B.pvt_set_m1_search({"auto": B.PVT_M1_AUTO, "fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR}[args.search])
    tensor_engine = M == 1 and f16 and (args.search == "tensor" or (args.search == "auto" and K >= 1024))

    def gpu_nearest(X, C):  # only the recipe of a second codebook needs it: the library's own search
        return _nearest_on_gpu(X, C)

    # every rank draws its own layer (seed offset): independent problems, no exchange
    L = synth.make_layer(rows, cols, cfg=rank_layer_seed(cfg, rank), num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         row_max_scale=rowmax, nearest=gpu_nearest, name=name)
    G = L.num_groups
    k = synth.subspace_size(tau, G)
    pairs_per_group = L.pairs_per_group()

    # host side (pinned) and device side of every array
    def pin(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        return t.pin_memory()

    h = {n: pin(getattr(L, n)) for n in ("W", "g", "scale", "codebooks", "codes")}
    d = {n: t.to(dev) for n, t in h.items()}
    codes0 = d["codes"].clone()
    out_dtype = torch.float16 if args.dequant_fp16 else torch.float32
    W_hat = torch.empty(rows, cols, dtype=out_dtype, device=dev)
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    h_idx = torch.empty(k, dtype=torch.int32).pin_memory()
    h_codes_out = torch.empty_like(h["codes"]).pin_memory()
    desc = B.make_layer(rows, cols, d["W"], d["g"], d["scale"], d["codebooks"], d["codes"], eta=L.eta, beam=L.beam)
    ws = B.new_workspace(desc, k, device=dev)
    flush = torch.empty(64 << 20, dtype=torch.int32, device=dev)  # 256 MiB, twice the L2

    def flush_l2():
        # write, then read: the write evicts every line of the step's arrays, the read leaves the L2 full of
        # clean lines, so that no write-back of the flush buffer is charged to the step that follows
        flush.fill_(1)
        flush.sum()

    def step():
        B.pvt_vstep_select(desc, k, idx, ws)
        B.pvt_vstep_encode(desc, idx, k, None, ws)
        B.pvt_dequant(desc, W_hat)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up
    for _ in range(max(args.warmup, 3)):
        d["codes"].copy_(codes0)
        step()
    torch.cuda.synchronize()
    st = B.pvt_status(ws)
    if st != 0:
        raise SystemExit(f"bench.py: device status word {st} after warm-up")

    # ---- device-resident timing: K steps, L2 flushed before each, per-kernel events inside the library
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    B.pvt_timing_enable(True)
    for kid in range(7):
        B.pvt_timing_read(kid)
    launches0 = B.pvt_launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in ev:
        d["codes"].copy_(codes0)  # same previous codes every step (untimed)
        flush_l2()                # evict W, g and the codebook from L2 (untimed)
        a.record()
        step()
        b.record()
    barrier()
    launches = B.pvt_launch_count() - launches0
    eager_ms = sum(a.elapsed_time(b) for a, b in ev)
    kern = {kid: B.pvt_timing_read(kid) for kid in range(5)}
    B.pvt_timing_enable(False)

    # ---- the same step as a CUDA graph (the three C-ABI calls captured once, replayed K times): the launch
    # gaps between the step's nine short kernels and four memsets disappear; this is the headline timing
    graphed = False
    total_ms = eager_ms
    if not args.no_graph:
        try:
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                step()
            for _ in range(3):
                d["codes"].copy_(codes0)
                gph.replay()
            barrier()
            for a, b in ev:
                d["codes"].copy_(codes0)
                flush_l2()
                a.record()
                gph.replay()
                b.record()
            barrier()
            total_ms = sum(a.elapsed_time(b) for a, b in ev)
            graphed = True
        except RuntimeError as exc:  # capture not possible: report the eager timing and say so
            print(f"bench.py: CUDA graph capture failed ({exc}); eager launches are timed", file=sys.stderr)
    B.pvt_timing_enable(True)
    # the P-step kernels that share the V step's inputs (not part of the timed step): same flush, own events
    gb = torch.empty((M, K, 8), dtype=torch.float64, device=dev)
    gs = torch.empty(rows, dtype=torch.float64, device=dev)
    master = d["codebooks"].float().reshape(-1).clone()
    adam_m, adam_v = torch.zeros_like(master), torch.zeros_like(master)
    scratch16 = torch.empty(master.numel(), dtype=torch.float16, device=dev)
    for i in range(min(args.steps, 10)):
        flush_l2()
        B.pvt_pstep_grad(desc, gb, gs)
        B.pvt_adam_update(master, gb.reshape(-1), adam_m, adam_v, i + 1, 3e-4, param_f16=scratch16)
    torch.cuda.synchronize()
    kern[B.PVT_KERNEL_PSTEP_GRAD] = B.pvt_timing_read(B.PVT_KERNEL_PSTEP_GRAD)
    kern[B.PVT_KERNEL_ADAM] = B.pvt_timing_read(B.PVT_KERNEL_ADAM)
    B.pvt_timing_enable(False)
    st = B.pvt_status(ws)
    if st != 0:
        raise SystemExit(f"bench.py: device status word {st} after the timed region")

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    e2e_steps = max(3, min(args.steps, 10))
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(e2e_steps)]
    h2d = sum(t.numel() * t.element_size() for t in h.values())
    d2h = h_idx.numel() * 4 + h_codes_out.numel() * h_codes_out.element_size()
    barrier()
    for a, b in ev2:
        a.record()
        for n in ("W", "g", "scale", "codebooks", "codes"):
            d[n].copy_(h[n], non_blocking=True)
        step()
        h_idx.copy_(idx, non_blocking=True)
        h_codes_out.copy_(d["codes"], non_blocking=True)
        b.record()
        b.synchronize()
    barrier()
    e2e_ms = sum(a.elapsed_time(b) for a, b in ev2) / e2e_steps
    clocks = sampler.stop() if rank == 0 else None

    # reference point for the streaming kernels at this size: a library fill of the dequantised matrix (the bytes
    # pvt_dequant writes), cold L2, timed the same way.  Outside the timed region; rank 0 only.
    fill_ms = None
    if rank == 0:
        spans = []
        for _ in range(5):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            W_hat.fill_(0)
            b.record()
            b.synchronize()
            spans.append(a.elapsed_time(b))
        fill_ms = sorted(spans)[len(spans) // 2]

    total_ms, e2e_ms = slowest_rank([total_ms, e2e_ms], dev, world)
    ms_per_step = total_ms / args.steps

    if rank == 0:
        peaks = _measured_peaks()
        props = torch.cuda.get_device_properties(local)
        sm_max_mhz = (clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz") or 1965.0
        alu_peak = props.multi_processor_count * FP32_LANES_PER_SM * 2 * sm_max_mhz * 1e6 / 1e12  # TFLOP/s
        ffma_measured = B.pvt_probe_fp32_tflops()  # the same pipe, measured in this job
        enc_ms, enc_n = kern[B.PVT_KERNEL_ENCODE_MAIN]
        enc_avg_ms = enc_ms / max(enc_n, 1)
        pairs = k * pairs_per_group
        achieved = FLOP_PER_PAIR * pairs / (enc_avg_ms * 1e-3) / 1e12
        hbm = peaks.get("hbm_gbs")
        stages = {}
        sel_ms, sel_n = kern[B.PVT_KERNEL_SELECT]
        aux_ms, aux_n = kern[B.PVT_KERNEL_ENCODE_AUX]
        dq_ms, dq_n = kern[B.PVT_KERNEL_DEQUANT]
        code_bytes = L.codes.dtype.itemsize * M
        dq_bytes = G * (code_bytes + 8 * W_hat.element_size())
        sel_bytes = G * 32 + 4 * k
        stages["select"] = {"ms": sel_ms / max(sel_n, 1), "algorithmic_bytes": sel_bytes,
                            "gbs": sel_bytes / (sel_ms / max(sel_n, 1) * 1e-3) / 1e9 if sel_n else None}
        stages["encode_search"] = {"ms": enc_avg_ms, "pairs": pairs,
                                   "pairs_per_s": pairs / (enc_avg_ms * 1e-3)}
        stages["encode_codebook_prep"] = {"ms": aux_ms / max(aux_n, 1)}
        rs_ms, rs_n = kern[B.PVT_KERNEL_ENCODE_RESCORE]
        stages["encode_rescore"] = {"ms": rs_ms / max(rs_n, 1)}
        stages["dequant"] = {"ms": dq_ms / max(dq_n, 1), "algorithmic_bytes": dq_bytes,
                             "gbs": dq_bytes / (dq_ms / max(dq_n, 1) * 1e-3) / 1e9 if dq_n else None}
        stages["dequant"]["library_fill_of_the_same_output_ms"] = fill_ms
        # per-stage rates: the whole encode call (codebook preparation + search + rescoring), alone and with
        # the selection in front of it
        t_enc_call = (aux_ms / max(aux_n, 1) + enc_avg_ms + rs_ms / max(rs_n, 1)) * 1e-3
        t_sel_call = sel_ms / max(sel_n, 1) * 1e-3
        stages["rates"] = {"groups_per_s_encode": k / t_enc_call if t_enc_call > 0 else None,
                           "groups_per_s_select_plus_encode": k / (t_enc_call + t_sel_call) if t_enc_call > 0 else None,
                           "pairs_per_s_encode": pairs / t_enc_call if t_enc_call > 0 else None}
        pg_ms, pg_n = kern[B.PVT_KERNEL_PSTEP_GRAD]
        ad_ms, ad_n = kern[B.PVT_KERNEL_ADAM]
        pg_bytes = G * (32 + code_bytes) + M * K * 8 * 8 + rows * 12
        ad_bytes = M * K * 8 * (8 + 4 * 6 + 2)
        stages["pstep_grad"] = {"ms": pg_ms / max(pg_n, 1), "algorithmic_bytes": pg_bytes,
                                "gbs": pg_bytes / (pg_ms / max(pg_n, 1) * 1e-3) / 1e9 if pg_n else None,
                                "note": "not part of the timed V step"}
        stages["adam"] = {"ms": ad_ms / max(ad_n, 1), "algorithmic_bytes": ad_bytes,
                          "gbs": ad_bytes / (ad_ms / max(ad_n, 1) * 1e-3) / 1e9 if ad_n else None,
                          "note": "not part of the timed V step"}
        if hbm:
            for s in ("select", "dequant", "pstep_grad", "adam"):
                if stages[s]["gbs"]:
                    stages[s]["frac_of_measured_hbm"] = stages[s]["gbs"] / hbm
        if tensor_engine:
            # dense contraction on the tensor cores: algorithmic flops against the measured fp16/bf16 peak
            tpeak = peaks.get("bf16_tflops")
            roofline = {"kernel": "encode search (M=1, tcgen05)", "bound": "tensor", "achieved": achieved,
                        "peak": tpeak, "unit": "TFLOP/s", "frac": achieved / tpeak,
                        "peak_is": ("measured bf16 matmul (fp16 operands run at the same rate)"
                                    if not peaks.get("fallback") else "fallback of the profiling recipe"),
                        "flop_per_pair": FLOP_PER_PAIR, "avg_launch_ms": enc_avg_ms, "launches": enc_n,
                        "executed_tflops": achieved * 4.0,  # operands are padded from depth 8 to depth 32
                        "frac_of_fp32_alu_roofline": achieved / alu_peak,
                        "fp32_fma_microbenchmark_tflops": ffma_measured,
                        "frac_of_epilogue_bound": (pairs / (enc_avg_ms * 1e-3)) /
                                                  (props.multi_processor_count * 128 * sm_max_mhz * 1e6),
                        "epilogue_bound_is": "one accumulator read per pair: 128 lanes per SM per clock",
                        # dram__bytes_read + dram__bytes_write of one launch (ncu, this kernel, default workload)
                        "traffic": 7.64e6 if args.workload == DEFAULT_WORKLOAD else None}
        else:
            roofline = {"kernel": "encode search (M=1, fp32 pipe)" if M == 1 else "encode beam search (M=2)",
                        "bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "TFLOP/s",
                        "frac": achieved / alu_peak,
                        "peak_is": f"{props.multi_processor_count} SMs x 128 FP32 lanes x 2 flop x "
                                   f"{sm_max_mhz:.0f} MHz (derived; no measured FP32 peak)",
                        "flop_per_pair": FLOP_PER_PAIR, "avg_launch_ms": enc_avg_ms, "launches": enc_n,
                        "fp32_fma_microbenchmark_tflops": ffma_measured,
                        # dram__bytes_read + dram__bytes_write of one launch (ncu, FP32 engine, default workload)
                        "traffic": 7.87e6 if (M == 1 and args.workload == DEFAULT_WORKLOAD) else None}
            if M == 2:
                # the kernel is bound by instruction issue; the pair evaluations of stage 2 themselves run on the
                # tensor pipe when the codebooks are fp16, so the FP32-pipe roofline is a yardstick, not a ceiling
                roofline["note"] = ("issue-bound; stage 2 (2048 of 2304 pairs per group) on the tensor pipe for fp16 "
                                    "codebooks, the FP32-pipe roofline is the yardstick the 16 flop per pair refer to")
        line = {
            "metric": METRIC, "value": job_value(k, world, ms_per_step), "unit": UNIT,
            "pairs_per_s": world * pairs / (ms_per_step * 1e-3),
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "ms_per_step_eager_launches": eager_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "rows": rows, "cols": cols, "group_dim": 8, "groups": G,
                       "num_codebooks": M, "codebook_size": K, "codebook_dtype": "f16" if f16 else "f32",
                       "tau": tau, "k": k, "pairs_per_group": pairs_per_group,
                       "search_engine": ("tensor" if tensor_engine else "fp32") if M == 1 else "beam",
                       "dequant_dtype": "f16" if args.dequant_fp16 else "f32",
                       "l2": "flushed before every timed step (256 MiB written, then read)",
                       "launch": ("CUDA graph replay of pvt_vstep_select + pvt_vstep_encode + pvt_dequant" if graphed
                                  else "eager launches"),
                       "parallelism": f"independent layers x{world}"},
            "e2e": {"value": world * k / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "what": "pinned host W, g, scale, codebook, codes -> device; select+encode+dequant; "
                            "idx and codes -> pinned host"},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "stages": stages,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(L, k, tau, budget_s=args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def rank_layer_seed(cfg: int, rank: int) -> int:
    """Every rank steps its own layer: the seed family of rank r is cfg + 100 r (layers are independent
    problems, so no rank ever needs another rank's data)."""
    return cfg + 100 * rank


def slowest_rank(times_ms, device, world: int):
    """Device times of this rank -> the maximum over all ranks (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_value(k_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: the groups all ranks re-encode per step over the slowest rank's step time."""
    return world * k_per_rank / (ms_per_step * 1e-3)


def _nearest_on_gpu(X, C):
    """Nearest codeword of C for every row of X with the library's own M = 1 search
    (input recipe of a second codebook; runs before anything is timed)."""
    import numpy as np
    import torch

    from paper_2405_14852_b200 import binding as B
    n = X.shape[0]
    rows = n
    W = torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).cuda()
    g = torch.zeros_like(W)
    scale = torch.ones(rows, dtype=torch.float32, device="cuda")
    books = torch.from_numpy(np.ascontiguousarray(C, dtype=np.float32)[None]).cuda()
    code_dtype = torch.uint8 if C.shape[0] <= 256 else torch.uint16
    codes = torch.zeros(n, 1, dtype=code_dtype, device="cuda")
    desc = B.make_layer(rows, 8, W, g, scale, books, codes, eta=0.0)
    ws = B.new_workspace(desc, n)
    idx = torch.arange(n, dtype=torch.int32, device="cuda")
    B.pvt_vstep_encode(desc, idx, n, None, ws)
    torch.cuda.synchronize()
    return codes.cpu().numpy()[:, 0].astype(np.int64)


def _measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except OSError:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "fallback": True}


# --------------------------------------------------------------------------- CPU arm


def cpu_baseline(L, k, tau, budget_s=15.0):
    """The CPU checker, as it stands, on a bounded sample of the same layer: norms and
    selection over all groups, the search on the first n selected groups (n sized for
    about `budget_s` seconds), dequantisation of the whole layer.  The search time is
    scaled to all k groups; the value is k over that estimated whole-step time."""
    import numpy as np

    from oracle import pvt_oracle as oracle
    threads = oracle.num_threads()
    t0 = time.perf_counter()
    norms = oracle.group_norms(L.g, L.eta)
    idx = oracle.select(norms, k)
    t_sel = time.perf_counter() - t0
    codes2 = L.codes.reshape(-1, L.num_codebooks)
    # calibrate on a small probe, then size the sample
    n0 = min(k, 256)
    t_probe = _time_oracle_encode(oracle, L, idx[:n0], codes2)
    n = int(min(k, max(n0, n0 * budget_s / max(t_probe, 1e-6))))
    t_enc = _time_oracle_encode(oracle, L, idx[:n], codes2)
    t0 = time.perf_counter()
    oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols)
    t_deq = time.perf_counter() - t0
    t_step = t_sel + t_enc * (k / n) + t_deq
    # the same search on one thread, on a sample smaller by the thread count (a few seconds)
    one_thread = None
    if threads > 1:
        n1 = max(1, min(n, n // threads))
        oracle.set_num_threads(1)
        try:
            t1 = _time_oracle_encode(oracle, L, idx[:n1], codes2)
        finally:
            oracle.set_num_threads(threads)
        one_thread = {"pairs_per_s": n1 * L.pairs_per_group() / t1, "sample_groups": n1, "seconds": t1}
    return {"value": k / t_step, "unit": UNIT, "cores": threads, "kind": "oracle", "search_on_one_thread": one_thread,
            "sample": f"norms+selection over all {L.num_groups} groups ({t_sel:.2f} s), search of the first {n} of "
                      f"{k} selected groups ({t_enc:.2f} s, scaled by k/n), dequantisation of the whole layer "
                      f"({t_deq:.2f} s)",
            "pairs_per_s": n * L.pairs_per_group() / t_enc, "estimated_step_s": t_step}


def _time_oracle_encode(oracle, L, idx, codes2):
    import numpy as np
    t0 = time.perf_counter()
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    oracle.encode(t, L.codebooks, codes2[idx.astype(np.int64)], L.beam)
    return time.perf_counter() - t0


def run_reference(args):
    """The CPU checker timed as the reference arm: every step is one bounded sample of
    the workload (selection over all groups, search of n selected groups, whole-layer
    dequantisation); value = groups re-encoded per second of that step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np

    from oracle import pvt_oracle as oracle
    from paper_2405_14852_b200 import synth
    cfg, which, tau = workloads()[args.workload]
    name, rows, cols, M, K, f16, rowmax, _ = synth.CONFIGS[cfg][which]

    def nearest(X, C):
        return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]

    L = synth.make_layer(rows, cols, cfg=cfg, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         row_max_scale=rowmax, nearest=nearest, name=name)
    k = synth.subspace_size(tau, L.num_groups)
    codes2 = L.codes.reshape(-1, M)
    threads = oracle.num_threads()
    # sample size: about 2 s of search per step
    idx_full = oracle.select(oracle.group_norms(L.g, L.eta), k)
    n0 = min(k, 128)
    t_probe = _time_oracle_encode(oracle, L, idx_full[:n0], codes2)
    n = int(min(k, max(n0, n0 * 2.0 / max(t_probe, 1e-6))))
    warm = max(args.warmup, 1)
    times = []
    for i in range(warm + args.steps):
        t0 = time.perf_counter()
        idx = oracle.select(oracle.group_norms(L.g, L.eta), k)
        t_sel = time.perf_counter() - t0
        t_enc = _time_oracle_encode(oracle, L, idx[:n], codes2)
        t0 = time.perf_counter()
        oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols)
        t_deq = time.perf_counter() - t0
        if i >= warm:
            times.append(t_sel + t_enc * (k / n) + t_deq)
    t_step = sum(times) / len(times)
    value = k / t_step
    sample = (f"per step: norms+selection over all {L.num_groups} groups, search of the first {n} of {k} selected "
              f"groups (time scaled by k/n), dequantisation of the whole layer")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": warm, "ms_per_step": t_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "rows": rows, "cols": cols, "groups": L.num_groups,
                       "num_codebooks": M, "codebook_size": K, "tau": tau, "k": k},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- the calls beyond the V step proper


def run_next_rows(args):
    """Times the calls that widen the path (trust-ratio step, local search, three and four codebooks, groups of
    16 weights) on synthetic layers of the benchmark shapes and prints one JSON line.  Not the headline metric."""
    import numpy as np
    import torch

    from paper_2405_14852_b200 import binding as B
    from paper_2405_14852_b200 import synth
    from paper_2405_14852_b200.vstep import VStepLayer

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the V step has no CPU path")
    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")

    def timed(fn, reps=5):
        spans = []
        for i in range(reps + 2):
            flush.fill_(1)
            flush.sum()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            b.synchronize()
            if i >= 2:
                spans.append(a.elapsed_time(b))
        return sorted(spans)[len(spans) // 2]

    out = {"what": "median of 5 cold-L2 calls each, CUDA events; synthetic layers of the benchmark shapes"}

    # trust-ratio step on the default workload's layer (its random previous codes make every change large, so
    # the cut falls early; the cost is that of ranking and re-encoding k_max groups either way)
    L = synth.make_layer(4096, 4096, cfg=2, codebook_size=65536, codebook_fp16=True)
    dev = VStepLayer.from_host(L)
    k = synth.subspace_size("0.01", L.num_groups)
    dev.step_trust(k, 0.01)
    out["trust_step_4096x4096_1x16_kmax20971"] = {"ms": timed(lambda: dev.step_trust(k, 0.01))}
    out["plain_select_plus_encode_same_layer"] = {"ms": timed(lambda: dev.encode(dev.select(k)))}
    del dev

    # local search after the two-codebook beam search
    L = synth.make_layer(11008, 4096, cfg=3, num_codebooks=2, codebook_size=256, codebook_fp16=True,
                         nearest=_nearest_on_gpu)
    dev = VStepLayer.from_host(L)
    k = synth.subspace_size("0.01", L.num_groups)
    idx = dev.select(k)
    dev.encode(idx)
    out["local_search_11008x4096_2x8_k56360"] = {"ms": timed(lambda: B.pvt_vstep_refine(dev.desc, idx, k, 64))}
    out["beam_search_same_layer"] = {"ms": timed(lambda: dev.encode(idx))}
    del dev

    # three and four codebooks
    for M in (3, 4):
        L = synth.make_layer(11008, 4096, cfg=3, num_codebooks=M, codebook_size=256, codebook_fp16=True,
                             nearest=_nearest_on_gpu)
        dev = VStepLayer.from_host(L)
        idx = dev.select(k)
        ms = timed(lambda: dev.encode(idx))
        pairs = k * L.pairs_per_group()
        out[f"beam_search_11008x4096_{M}x8_k56360"] = {"ms": ms, "pairs_per_s": pairs / (ms * 1e-3)}
        out[f"dequant_11008x4096_{M}x8"] = {"ms": timed(lambda: dev.dequant())}
        del dev

    # groups of 16 weights, one codebook of 65 536
    L = synth.make_layer(4096, 4096, cfg=2, codebook_size=65536, codebook_fp16=True, group_dim=16)
    dev = VStepLayer.from_host(L)
    k = synth.subspace_size("0.01", L.num_groups)
    idx = dev.select(k)
    ms = timed(lambda: dev.encode(idx), reps=3)
    out["g16_4096x4096_1x16_k10485"] = {"select_ms": timed(lambda: dev.select(k)), "search_ms": ms,
                                        "pairs_per_s": k * 65536 / (ms * 1e-3),
                                        "dequant_ms": timed(lambda: dev.dequant())}
    torch.cuda.synchronize()
    if dev.status() != 0:
        raise SystemExit("bench.py: device status word set")
    print(json.dumps({"next_rows": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--search", default="auto", choices=["auto", "fp32", "tensor"],
                    help="engine of the single-codebook search")
    ap.add_argument("--dequant-fp16", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA graph replay")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--list", action="store_true")
    ap.add_argument("--next-rows", action="store_true",
                    help="time the calls beyond the V step proper (trust-ratio step, local search, 3-4 codebooks, "
                         "groups of 16) instead of the headline metric")
    args = ap.parse_args()
    if args.list:
        print("\n".join(workloads()))
        return
    if args.next_rows:
        run_next_rows(args)
        return
    if args.workload not in workloads():
        raise SystemExit(f"unknown workload {args.workload}; --list shows the names")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
