#!/usr/bin/env python
"""Benchmark of the V step (select -> re-encode -> dequantise) on synthetic layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one whole V step over the workload: for every layer of it, pvt_vstep_select,
pvt_vstep_encode and pvt_dequant through the C ABI, all on one stream.  The default workload is
the largest one of the benchmark table that one GPU holds: the seven linear layers of one
Llama-2-70B decoder block (2 x 8192x8192, 2 x 8192x1024, 2 x 28672x8192, 8192x28672; fp32 weights
and update, one fp16 codebook of 65536 codewords per layer, groups of 8) with every group
re-encoded (tau = 1.0): 106 954 752 groups, 7.0e12 codeword pairs per step.  The single-layer
workloads of the table are available by name (--list).  With N > 1 (launched by
torch.distributed.run) every rank steps its own copy of the workload (layers are independent
problems: no collective on the data path); the reported value is the work of all ranks over the
slowest rank's time.

Besides the headline, the line carries `sub` (the 4096x4096, tau = 0.01 layer with the search on
the tensor cores and on the FP32 pipe) and `sweep` (every single-layer workload of the table,
briefly).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import hashlib
import json
import os
import re
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
BLOCK_PREFIX = "llama2_70b_block_1x16"
DEFAULT_WORKLOAD = BLOCK_PREFIX + "_tau1.0"
SUB_WORKLOAD = "llama2_7b_attn_4096x4096_1x16_tau0.01"
GRAPH_BELOW_MS = 5.0     # steps shorter than this are timed as CUDA graph replays (launch gaps matter there)


def workloads():
    """name -> ("layer", cfg, entry, tau) or ("block", tau)."""
    from paper_2405_14852_b200 import synth
    out = {}
    for cfg, entries in synth.CONFIGS.items():
        for which, e in enumerate(entries):
            for tau in e[7]:
                out[f"{e[0]}_tau{tau}"] = ("layer", cfg, which, tau)
    for tau in ("0.01", "1.0"):
        out[f"{BLOCK_PREFIX}_tau{tau}"] = ("block", tau)
    return out


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
        sm, smax, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax = float(f[1])
                power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax, "sm_mhz_min": sm[0] if sm else None,
                "samples": len(sm), "power_w_max": max(power) if power else None, "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- layers on the device


class DeviceLayer:
    """One synthetic layer: pinned host arrays, device arrays, descriptor, index buffer, outputs."""

    def __init__(self, L, tau, dev, out_dtype, keep_host=True):
        import numpy as np
        import torch

        from paper_2405_14852_b200 import binding as B
        from paper_2405_14852_b200 import synth
        self.L = L
        self.name = L.name
        self.rows, self.cols, self.M, self.K = L.rows, L.cols, L.num_codebooks, L.codebook_size
        self.G = L.num_groups
        self.tau = tau
        self.k = synth.subspace_size(tau, self.G)
        self.pairs = self.k * L.pairs_per_group()
        self.h = {}
        self.d = {}
        for n in ("W", "g", "scale", "codebooks", "codes"):
            a = np.ascontiguousarray(getattr(L, n))
            t = torch.from_numpy(a)
            if keep_host:
                pinned = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
                pinned.copy_(t)
                self.h[n] = pinned
                self.d[n] = pinned.to(dev, non_blocking=True)
            else:
                self.d[n] = t.to(dev)
        torch.cuda.synchronize()
        self.codes0 = self.d["codes"].clone()
        self.W_hat = torch.empty(self.rows, self.cols, dtype=out_dtype, device=dev)
        self.idx = torch.empty(self.k, dtype=torch.int32, device=dev)
        self.desc = B.make_layer(self.rows, self.cols, self.d["W"], self.d["g"], self.d["scale"], self.d["codebooks"],
                                 self.d["codes"], eta=L.eta, beam=L.beam)
        self.ws_bytes = B.pvt_workspace_bytes(self.desc, self.k)
        self.code_bytes = L.codes.dtype.itemsize * self.M
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.d.values())

    def set_tau(self, tau, dev):
        import torch

        from paper_2405_14852_b200 import binding as B
        from paper_2405_14852_b200 import synth
        self.tau = tau
        self.k = synth.subspace_size(tau, self.G)
        self.pairs = self.k * self.L.pairs_per_group()
        self.idx = torch.empty(self.k, dtype=torch.int32, device=dev)
        self.ws_bytes = B.pvt_workspace_bytes(self.desc, self.k)


class Runner:
    """Steps a list of DeviceLayers through the three C-ABI calls and times them."""

    def __init__(self, layers, dev, world=1):
        import torch

        from paper_2405_14852_b200 import binding as B
        self.B = B
        self.torch = torch
        self.layers = layers
        self.dev = dev
        self.world = world
        # one workspace serves every layer: the calls of a step run one after the other on one stream
        self.ws = torch.empty(max(l.ws_bytes for l in layers), dtype=torch.uint8, device=dev)
        B.pvt_workspace_init(self.ws)
        self.k = sum(l.k for l in layers)
        self.pairs = sum(l.pairs for l in layers)
        self.G = sum(l.G for l in layers)
        # the whole workload as one pvt_vstep_block call (select -> encode -> dequantise per layer, one stream)
        self.block = B.Block([l.desc for l in layers], [l.k for l in layers], [l.idx for l in layers],
                             [l.W_hat for l in layers])

    def step(self):
        self.B.pvt_vstep_block(self.block, self.ws)

    def restore_codes(self):
        for l in self.layers:
            l.d["codes"].copy_(l.codes0)

    def barrier(self):
        import torch.distributed as dist
        self.torch.cuda.synchronize()
        if self.world > 1:
            dist.barrier()
        self.torch.cuda.synchronize()

    def check_status(self, where):
        st = self.B.pvt_status(self.ws)
        if st != 0:
            raise SystemExit(f"bench.py: device status word {st} {where}")

    def timed(self, steps, warmup, flush_l2, allow_graph=True):
        """W warm-up steps, then K timed steps (L2 flushed and the previous codes restored before each, both
        untimed): eager launches with the library's per-kernel events, and -- when a step is short enough for
        launch gaps to matter -- the same step replayed from a CUDA graph.  Returns a dict of timings."""
        torch, B = self.torch, self.B
        for _ in range(max(warmup, 3)):
            self.restore_codes()
            self.step()
        torch.cuda.synchronize()
        self.check_status("after warm-up")
        B.pvt_timing_enable(True)
        for kid in range(9):
            B.pvt_timing_read(kid)
        launches0 = B.pvt_launch_count()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        self.barrier()
        for a, b in ev:
            self.restore_codes()
            flush_l2()
            a.record()
            self.step()
            b.record()
        self.barrier()
        launches = B.pvt_launch_count() - launches0
        eager_ms = sum(a.elapsed_time(b) for a, b in ev)
        kern = {kid: B.pvt_timing_read(kid) for kid in range(5)}
        B.pvt_timing_enable(False)
        out = {"eager_ms_per_step": eager_ms / steps, "ms_per_step": eager_ms / steps, "graphed": False,
               "launches": int(launches), "kern": kern}
        if allow_graph and eager_ms / steps < GRAPH_BELOW_MS:
            try:
                side = torch.cuda.Stream(device=self.dev)
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    self.step()
                torch.cuda.current_stream().wait_stream(side)
                torch.cuda.synchronize()
                gph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gph):
                    self.step()
                for _ in range(3):
                    self.restore_codes()
                    gph.replay()
                self.barrier()
                launches0 = B.pvt_launch_count()
                for a, b in ev:
                    self.restore_codes()
                    flush_l2()
                    a.record()
                    gph.replay()
                    b.record()
                self.barrier()
                out["ms_per_step"] = sum(a.elapsed_time(b) for a, b in ev) / steps
                out["graphed"] = True
            except RuntimeError as exc:  # capture not possible: report the eager timing and say so
                print(f"bench.py: CUDA graph capture failed ({exc}); eager launches are timed", file=sys.stderr)
        self.check_status("after the timed region")
        return out

    def e2e(self, steps):
        """The same step with host buffers: every layer's W, g, scale, codebook and codes copied from pinned
        host memory inside the timed region, the selected indices and the new codes copied back.  The copies run on
        a stream of their own, so that a layer's inputs arrive while the layer before it is searched and its results
        leave while the next one is searched (every layer has device arrays of its own); the timed region runs from
        before the first copy to after the last result has reached the host."""
        torch = self.torch
        h_idx = [torch.empty(l.k, dtype=torch.int32, pin_memory=True) for l in self.layers]
        h_codes = [torch.empty(l.h["codes"].shape, dtype=l.h["codes"].dtype, pin_memory=True) for l in self.layers]
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        h2d = sum(l.h2d_bytes for l in self.layers)
        d2h = sum(t.numel() * t.element_size() for t in h_idx + h_codes)
        B = self.B
        main = torch.cuda.current_stream()
        up, down = torch.cuda.Stream(device=self.dev), torch.cuda.Stream(device=self.dev)
        self.barrier()
        for a, b in ev:
            a.record(main)
            up.wait_stream(main)
            down.wait_stream(main)
            arrived, done = [], []
            for l in self.layers:  # host -> device, in layer order, on the upload stream
                with torch.cuda.stream(up):
                    for n in ("W", "g", "scale", "codebooks", "codes"):
                        l.d[n].copy_(l.h[n], non_blocking=True)
                    e = torch.cuda.Event()
                    e.record(up)
                    arrived.append(e)
            for l, e_in, hi, hc in zip(self.layers, arrived, h_idx, h_codes):
                main.wait_event(e_in)
                B.pvt_vstep_select(l.desc, l.k, l.idx, self.ws)
                B.pvt_vstep_encode(l.desc, l.idx, l.k, None, self.ws)
                B.pvt_dequant(l.desc, l.W_hat)
                e = torch.cuda.Event()
                e.record(main)
                with torch.cuda.stream(down):  # device -> host once the layer is finished
                    down.wait_event(e)
                    hi.copy_(l.idx, non_blocking=True)
                    hc.copy_(l.d["codes"], non_blocking=True)
            main.wait_stream(down)
            main.wait_stream(up)
            b.record(main)
            b.synchronize()
        self.barrier()
        return sum(a.elapsed_time(b) for a, b in ev) / steps, h2d, d2h


def make_flush(dev):
    import torch
    flush = torch.empty(64 << 20, dtype=torch.int32, device=dev)  # 256 MiB, twice the L2

    def flush_l2():
        # write, then read: the write evicts every line of the step's arrays, the read leaves the L2 full of
        # clean lines, so that no write-back of the flush buffer is charged to the step that follows
        flush.fill_(1)
        flush.sum()
    return flush_l2


def build_layers(kind, rank, dev, out_dtype, keep_host=True):
    """Host generation (in parallel threads: the generators release the interpreter lock) + upload."""
    from paper_2405_14852_b200 import synth
    if kind[0] == "block":
        tau = kind[1]
        n = len(synth.BLOCK_70B)
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(n, os.cpu_count() or 1)) as pool:
            host = list(pool.map(lambda i: synth.make_block_layer(i, seed_offset=100 * rank), range(n)))
        out = []
        for L in host:
            out.append(DeviceLayer(L, tau, dev, out_dtype, keep_host))
        return out
    _, cfg, which, tau = kind
    name, rows, cols, M, K, f16, rowmax, _ = synth.CONFIGS[cfg][which]
    L = synth.make_layer(rows, cols, cfg=rank_layer_seed(cfg, rank), num_codebooks=M, codebook_size=K,
                         codebook_fp16=f16, row_max_scale=rowmax, nearest=_nearest_on_gpu, name=name)
    return [DeviceLayer(L, tau, dev, out_dtype, keep_host)]


# --------------------------------------------------------------------------- rooflines


def device_peaks(local, clocks=None):
    import torch
    peaks = _measured_peaks()
    props = torch.cuda.get_device_properties(local)
    sm_max_mhz = (clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz") or 1965.0
    peaks["sm_count"] = props.multi_processor_count
    peaks["sm_max_mhz_used"] = sm_max_mhz
    peaks["alu_tflops"] = props.multi_processor_count * FP32_LANES_PER_SM * 2 * sm_max_mhz * 1e6 / 1e12
    peaks["epilogue_pairs_per_s"] = props.multi_processor_count * 128 * sm_max_mhz * 1e6
    return peaks


def search_roofline(engine, pairs_per_step, enc_ms, enc_n, steps, peaks, traffic):
    """Roofline record of the search kernel: algorithmic flops of the launches of one step over their summed
    duration (CUDA events inside the library, around every launch, on the launching stream)."""
    per_step_ms = enc_ms / max(steps, 1)
    achieved = FLOP_PER_PAIR * pairs_per_step / (per_step_ms * 1e-3) / 1e12
    common = {"achieved": achieved, "unit": "TFLOP/s", "flop_per_pair": FLOP_PER_PAIR,
              "launches": enc_n, "avg_launch_ms": enc_ms / max(enc_n, 1), "kernel_ms_per_step": per_step_ms,
              "pairs_per_s": pairs_per_step / (per_step_ms * 1e-3), "traffic": traffic}
    if engine == "tensor":
        tpeak = peaks.get("bf16_tflops_sustained" if per_step_ms > 50.0 else "bf16_tflops") or peaks.get("bf16_tflops")
        which = "sustained" if per_step_ms > 50.0 and peaks.get("bf16_tflops_sustained") else "burst"
        r = {"kernel": "encode_m1_tc_kernel (exhaustive search, tcgen05)", "bound": "tensor", "peak": tpeak,
             "frac": achieved / tpeak,
             "peak_is": (f"measured bf16 matmul, {which} figure (fp16 operands run at the same rate)"
                         if not peaks.get("fallback") else "fallback of the profiling recipe"),
             "frac_of_fp32_alu_roofline": achieved / peaks["alu_tflops"],
             "frac_of_epilogue_bound": common["pairs_per_s"] / peaks["epilogue_pairs_per_s"],
             "epilogue_bound_is": "one accumulator read per pair: 128 lanes per SM per clock at the maximum SM clock"}
    else:
        r = {"kernel": "encode_m1_kernel (exhaustive search, FP32 pipe)" if engine == "fp32"
             else "encode_m2_kernel (beam search)", "bound": "alu", "peak": peaks["alu_tflops"],
             "frac": achieved / peaks["alu_tflops"],
             "peak_is": f"{peaks['sm_count']} SMs x 128 FP32 lanes x 2 flop x {peaks['sm_max_mhz_used']:.0f} MHz "
                        f"(derived; no measured FP32 peak)"}
        if engine == "beam":
            r["note"] = ("issue-bound; stage 2 (2048 of 2304 pairs per group) on the tensor pipe for fp16 codebooks; "
                         "the search as written needs 16 (K1 + K2) + 2 B K2 flop per group (B.K2 cross terms reuse "
                         "<t, c2>), the 16 flop per pair of the metric count every pair as a full dot product")
    r.update(common)
    return r


def engine_of(layer, search):
    if layer.M != 1:
        return "beam"
    f16 = layer.L.codebooks.dtype.itemsize == 2
    if f16 and (search == "tensor" or (search == "auto" and layer.K >= 1024)):
        return "tensor"
    return "fp32"


_PROFILE_OF = {"tensor": ("encode_m1_tc_kernel_8192x1024_1x16_tau1.0.md", ["pvt_encode_m1_tc.cu", "pvt_encode_m1.cuh"]),
               "fp32": ("encode_m1_fp32_kernel_4096x4096_1x16_tau0.01.md", ["pvt_encode_m1.cu", "pvt_encode_m1.cuh"])}


def kernel_source_hash(files):
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2405_14852_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(engine, targets_per_step):
    """DRAM bytes of the search kernel per step from the committed ncu summary, scaled by the number of targets
    (the traffic is the gathered W, g rows and the per-target records: proportional to the targets).  None when
    there is no summary or the kernel's source has changed since the counters were taken."""
    if engine not in _PROFILE_OF:
        return None
    name, files = _PROFILE_OF[engine]
    try:
        text = open(os.path.join(ROOT, "profiles", name)).read()
    except OSError:
        return None
    m_hash = re.search(r"kernel_source_sha256_16:\s*([0-9a-f]{16})", text)
    m_bytes = re.search(r"dram_bytes_per_target:\s*([0-9.eE+]+)", text)
    if not m_hash or not m_bytes or m_hash.group(1) != kernel_source_hash(files):
        return None
    return float(m_bytes.group(1)) * targets_per_step


def stage_record(runner, t, steps, peaks, out_itemsize):
    kern = t["kern"]
    B = runner.B
    hbm = peaks.get("hbm_gbs")

    def per_step(kid):
        ms, n = kern[kid]
        return ms / max(steps, 1), n

    sel_ms, _ = per_step(B.PVT_KERNEL_SELECT)
    enc_ms, _ = per_step(B.PVT_KERNEL_ENCODE_MAIN)
    aux_ms, _ = per_step(B.PVT_KERNEL_ENCODE_AUX)
    dq_ms, _ = per_step(B.PVT_KERNEL_DEQUANT)
    rs_ms, _ = per_step(B.PVT_KERNEL_ENCODE_RESCORE)
    # the selection reads g once (32 B per group) and writes the indices; with k = G it is the index list itself
    sel_bytes = sum((l.G * 32 if l.k < l.G else 0) + 4 * l.k for l in runner.layers)
    dq_bytes = sum(l.G * (l.code_bytes + 8 * out_itemsize) for l in runner.layers)
    st = {"select": {"ms": sel_ms, "algorithmic_bytes": sel_bytes, "gbs": sel_bytes / (sel_ms * 1e-3) / 1e9 if sel_ms else None},
          "encode_search": {"ms": enc_ms, "pairs": runner.pairs, "pairs_per_s": runner.pairs / (enc_ms * 1e-3) if enc_ms else None},
          "encode_codebook_prep": {"ms": aux_ms},
          "encode_rescore": {"ms": rs_ms},
          "dequant": {"ms": dq_ms, "algorithmic_bytes": dq_bytes, "gbs": dq_bytes / (dq_ms * 1e-3) / 1e9 if dq_ms else None}}
    if hbm:
        for s in ("select", "dequant"):
            if st[s]["gbs"]:
                st[s]["frac_of_measured_hbm"] = st[s]["gbs"] / hbm
    t_enc_call = (aux_ms + enc_ms + rs_ms) * 1e-3
    if t_enc_call > 0:
        st["rates"] = {"groups_per_s_encode": runner.k / t_enc_call,
                       "groups_per_s_select_plus_encode": runner.k / (t_enc_call + sel_ms * 1e-3),
                       "pairs_per_s_encode": runner.pairs / t_enc_call}
    return st


# --------------------------------------------------------------------------- our arm


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2405_14852_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the V step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    kind = workloads()[args.workload]
    search_mode = {"auto": B.PVT_M1_AUTO, "fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR}
    B.pvt_set_m1_search(search_mode[args.search])
    out_dtype = torch.float16 if args.dequant_fp16 else torch.float32
    t0 = time.perf_counter()
    layers = build_layers(kind, rank, dev, out_dtype)
    setup_s = time.perf_counter() - t0
    runner = Runner(layers, dev, world)
    flush_l2 = make_flush(dev)
    engine = engine_of(layers[0], args.search)
    steps = args.steps

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    t = runner.timed(steps, args.warmup, flush_l2, allow_graph=not args.no_graph)
    e2e_steps = max(3, min(steps, 5))
    e2e_ms, h2d, d2h = runner.e2e(e2e_steps)
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_ms = slowest_rank([t["ms_per_step"], e2e_ms], dev, world)
    ms_per_step = total_ms

    if rank == 0:
        peaks = device_peaks(local, clocks)
        ffma_measured = B.pvt_probe_fp32_tflops()  # the FP32 pipe, measured in this job
        enc_ms, enc_n = t["kern"][B.PVT_KERNEL_ENCODE_MAIN]
        roofline = search_roofline(engine, runner.pairs, enc_ms, enc_n, steps, peaks,
                                   recorded_traffic(engine, runner.k))
        roofline["fp32_fma_microbenchmark_tflops"] = ffma_measured
        stages = stage_record(runner, t, steps, peaks, runner.layers[0].W_hat.element_size())
        # reference point for the streaming kernels: a library fill of the dequantised matrices (the bytes
        # pvt_dequant writes), cold L2, timed the same way, outside the timed region
        spans = []
        for _ in range(3):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for l in runner.layers:
                l.W_hat.fill_(0)
            b.record()
            b.synchronize()
            spans.append(a.elapsed_time(b))
        stages["dequant"]["library_fill_of_the_same_output_ms"] = sorted(spans)[1]

        L0 = runner.layers[0]
        config = {"workload": args.workload,
                  "layers": [{"name": l.name, "rows": l.rows, "cols": l.cols, "groups": l.G, "k": l.k} for l in runner.layers],
                  "group_dim": 8, "groups": runner.G, "num_codebooks": L0.M, "codebook_size": L0.K,
                  "codebook_dtype": "f16" if L0.L.codebooks.dtype.itemsize == 2 else "f32",
                  "tau": L0.tau, "k": runner.k, "pairs_per_step": runner.pairs,
                  "search_engine": engine, "dequant_dtype": "f16" if args.dequant_fp16 else "f32",
                  "l2": "flushed before every timed step (256 MiB written, then read)",
                  "launch": ("CUDA graph replay of one pvt_vstep_block call" if t["graphed"]
                             else "one pvt_vstep_block call per step (select + encode + dequantise per layer, one stream)"),
                  "parallelism": f"independent workloads x{world}"}
        line = {
            "metric": METRIC, "value": job_value(runner.k, world, ms_per_step), "unit": UNIT,
            "pairs_per_s": world * runner.pairs / (ms_per_step * 1e-3),
            "n_gpus": world, "steps": steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "ms_per_step_eager_launches": t["eager_ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config,
            "e2e": {"value": world * runner.k / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "what": "per layer: pinned host W, g, scale, codebook, codes -> device; select+encode+dequant; "
                            "idx and codes -> pinned host; copies on their own streams, overlapping other layers' search"},
            "gpu_launches": t["launches"],
            "roofline": roofline, "stages": stages, "clocks": clocks, "setup_s": setup_s,
        }
        del runner
        if not args.no_sub:
            line["sub"] = sub_record(args, dev, local, peaks, flush_l2, layers)
        if not args.no_sweep:
            line["sweep"] = sweep_record(args, dev, peaks, flush_l2, layers if kind[0] == "block" else None)
        if not args.no_next:
            line["stages"].update(pstep_record(dev, peaks, flush_l2))
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(layers, budget_s=args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def sub_record(args, dev, local, peaks, flush_l2, resident_layers):
    """The 4096 x 4096, one codebook of 65 536, tau = 0.01 layer with the exhaustive search on either engine."""
    import torch

    from paper_2405_14852_b200 import binding as B
    kind = workloads()[SUB_WORKLOAD]
    layers = build_layers(kind, 0, dev, torch.float32, keep_host=False)
    out = {"workload": SUB_WORKLOAD, "k": layers[0].k, "pairs": layers[0].pairs}
    for engine, mode in (("tensor", B.PVT_M1_TENSOR), ("fp32", B.PVT_M1_FP32)):
        B.pvt_set_m1_search(mode)
        for l in layers:
            l.set_tau(l.tau, dev)
        runner = Runner(layers, dev)
        steps = 20
        t = runner.timed(steps, 3, flush_l2)
        enc_ms, enc_n = t["kern"][B.PVT_KERNEL_ENCODE_MAIN]
        r = search_roofline(engine, runner.pairs, enc_ms, enc_n, steps, peaks, recorded_traffic(engine, runner.k)
                            if engine == "fp32" else recorded_traffic(engine, runner.k))
        st = stage_record(runner, t, steps, peaks, 4)
        out[engine] = {"ms_per_step": t["ms_per_step"], "groups_per_s": runner.k / (t["ms_per_step"] * 1e-3),
                       "pairs_per_s": runner.pairs / (t["ms_per_step"] * 1e-3), "graph_replay": t["graphed"],
                       "roofline": r,
                       "stages_ms": {k: v["ms"] for k, v in st.items() if isinstance(v, dict) and "ms" in v},
                       "select_frac_of_measured_hbm": st["select"].get("frac_of_measured_hbm"),
                       "dequant_frac_of_measured_hbm": st["dequant"].get("frac_of_measured_hbm")}
        del runner
    B.pvt_set_m1_search({"auto": B.PVT_M1_AUTO, "fp32": B.PVT_M1_FP32, "tensor": B.PVT_M1_TENSOR}[args.search])
    return out


def sweep_record(args, dev, peaks, flush_l2, block_layers):
    """Every single-layer workload of the table, briefly (3 timed steps each after 3 warm-up steps): step time,
    rates and the search kernel's fraction of its bound.  The 70B shapes reuse the block's resident layers."""
    import torch

    from paper_2405_14852_b200 import binding as B
    from paper_2405_14852_b200 import synth
    rows_out = []
    by_shape = {}
    if block_layers:
        for l in block_layers:
            by_shape.setdefault((l.rows, l.cols), l)
    for cfg, entries in synth.CONFIGS.items():
        for which, e in enumerate(entries):
            name, rows, cols, M, K, f16, rowmax, taus = e
            layer = by_shape.get((rows, cols)) if cfg == 5 else None
            own = layer is None
            if own:
                layer = build_layers(("layer", cfg, which, taus[0]), 0, dev,
                                     torch.float16 if cfg == 4 else torch.float32, keep_host=False)[0]
            saved_tau = layer.tau
            for tau in taus:
                layer.set_tau(tau, dev)
                runner = Runner([layer], dev)
                t = runner.timed(3, 3, flush_l2)
                engine = engine_of(layer, args.search)
                enc_ms, enc_n = t["kern"][B.PVT_KERNEL_ENCODE_MAIN]
                r = search_roofline(engine, runner.pairs, enc_ms, enc_n, 3, peaks, None)
                st = stage_record(runner, t, 3, peaks, layer.W_hat.element_size())
                rec = {"workload": f"{name}_tau{tau}", "k": layer.k, "ms_per_step": t["ms_per_step"],
                       "graph_replay": t["graphed"],
                       "groups_per_s": layer.k / (t["ms_per_step"] * 1e-3),
                       "pairs_per_s": layer.pairs / (t["ms_per_step"] * 1e-3),
                       "select_ms": st["select"]["ms"], "search_ms": st["encode_search"]["ms"],
                       "rescore_ms": st["encode_rescore"]["ms"], "dequant_ms": st["dequant"]["ms"],
                       "select_frac_hbm": st["select"].get("frac_of_measured_hbm"),
                       "dequant_frac_hbm": st["dequant"].get("frac_of_measured_hbm"),
                       "search_bound": r["bound"], "search_frac": r["frac"]}
                if engine == "tensor":
                    rec["search_frac_of_epilogue_bound"] = r["frac_of_epilogue_bound"]
                    rec["search_frac_of_fp32_alu_roofline"] = r["frac_of_fp32_alu_roofline"]
                rows_out.append(rec)
                del runner
            if own:
                del layer
                torch.cuda.empty_cache()
            else:
                layer.set_tau(saved_tau, dev)
    return rows_out


def pstep_record(dev, peaks, flush_l2):
    """The P-step kernels that share the V step's inputs (not part of the timed step), on the 4096 x 4096 layer."""
    import torch

    from paper_2405_14852_b200 import binding as B
    layer = build_layers(workloads()[SUB_WORKLOAD], 0, dev, torch.float32, keep_host=False)[0]
    M, K, rows, G = layer.M, layer.K, layer.rows, layer.G
    B.pvt_timing_enable(True)
    for kid in (B.PVT_KERNEL_PSTEP_GRAD, B.PVT_KERNEL_ADAM):
        B.pvt_timing_read(kid)
    gb = torch.empty((M, K, 8), dtype=torch.float64, device=dev)
    gs = torch.empty(rows, dtype=torch.float64, device=dev)
    master = layer.d["codebooks"].float().reshape(-1).clone()
    adam_m, adam_v = torch.zeros_like(master), torch.zeros_like(master)
    scratch16 = torch.empty(master.numel(), dtype=torch.float16, device=dev)
    n = 10
    for i in range(n):
        flush_l2()
        B.pvt_pstep_grad(layer.desc, gb, gs)
        B.pvt_adam_update(master, gb.reshape(-1), adam_m, adam_v, i + 1, 3e-4, param_f16=scratch16)
    torch.cuda.synchronize()
    pg_ms, pg_n = B.pvt_timing_read(B.PVT_KERNEL_PSTEP_GRAD)
    ad_ms, ad_n = B.pvt_timing_read(B.PVT_KERNEL_ADAM)
    B.pvt_timing_enable(False)
    hbm = peaks.get("hbm_gbs")
    pg_bytes = G * (32 + layer.code_bytes) + M * K * 8 * 8 + rows * 12
    ad_bytes = M * K * 8 * (8 + 4 * 6 + 2)
    out = {}
    for key, ms, cnt, nbytes in (("pstep_grad", pg_ms, pg_n, pg_bytes), ("adam", ad_ms, ad_n, ad_bytes)):
        rec = {"ms": ms / max(cnt, 1), "algorithmic_bytes": nbytes, "gbs": nbytes / (ms / max(cnt, 1) * 1e-3) / 1e9 if cnt else None,
               "note": f"not part of the timed V step; {SUB_WORKLOAD}'s layer"}
        if hbm and rec["gbs"]:
            rec["frac_of_measured_hbm"] = rec["gbs"] / hbm
        out[key] = rec
    return out


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
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "fallback": True}


# --------------------------------------------------------------------------- CPU arm


def _time_oracle_encode(oracle, L, idx, codes2):
    import numpy as np
    t0 = time.perf_counter()
    t = oracle.targets(L.W, L.g, L.scale, L.eta, idx)
    oracle.encode(t, L.codebooks, codes2[idx.astype(np.int64)], L.beam)
    return time.perf_counter() - t0


def _oracle_sample(oracle, L, k, search_budget_s, probe=256):
    """The CPU checker, as it stands, on one layer: norms and selection over all its groups, the search on the
    first n selected groups (n sized for about `search_budget_s` seconds), dequantisation of the whole layer."""
    t0 = time.perf_counter()
    idx = oracle.select(oracle.group_norms(L.g, L.eta), k)
    t_sel = time.perf_counter() - t0
    codes2 = L.codes.reshape(-1, L.num_codebooks)
    n0 = min(k, probe)
    t_probe = _time_oracle_encode(oracle, L, idx[:n0], codes2)
    n = int(min(k, max(n0, n0 * search_budget_s / max(t_probe, 1e-6))))
    t_enc = _time_oracle_encode(oracle, L, idx[:n], codes2)
    t0 = time.perf_counter()
    oracle.dequant(L.codes, L.codebooks, L.scale, L.rows, L.cols)
    t_deq = time.perf_counter() - t0
    return idx, codes2, n, t_sel, t_enc, t_deq


def _extrapolate(sample_layer, k_sample, n, t_sel, t_enc, t_deq, G_total, k_total, pairs_total):
    """Whole-workload step time of the checker from its timings on one layer: selection and dequantisation
    scale with the groups, the search with the codeword pairs."""
    pairs_n = n * sample_layer.pairs_per_group()
    return (t_sel + t_deq) * (G_total / sample_layer.num_groups) + t_enc * (pairs_total / pairs_n)


def _pick_sample_layer(layers):
    """The smallest layer of the workload stands for it on the CPU."""
    return min(layers, key=lambda l: l.G)


def cpu_baseline(layers, budget_s=12.0):
    from oracle import pvt_oracle as oracle
    threads = oracle.num_threads()
    dl = _pick_sample_layer(layers)
    L = dl.L
    G_total, k_total, pairs_total = sum(l.G for l in layers), sum(l.k for l in layers), sum(l.pairs for l in layers)
    idx, codes2, n, t_sel, t_enc, t_deq = _oracle_sample(oracle, L, dl.k, budget_s)
    t_step = _extrapolate(L, dl.k, n, t_sel, t_enc, t_deq, G_total, k_total, pairs_total)
    one_thread = None
    if threads > 1:
        n1 = max(1, min(n, n // threads))
        oracle.set_num_threads(1)
        try:
            t1 = _time_oracle_encode(oracle, L, idx[:n1], codes2)
        finally:
            oracle.set_num_threads(threads)
        one_thread = {"pairs_per_s": n1 * L.pairs_per_group() / t1, "sample_groups": n1, "seconds": t1}
    whole = len(layers) == 1 and n == dl.k
    return {"value": k_total / t_step, "unit": UNIT, "cores": threads, "kind": "oracle",
            "search_on_one_thread": one_thread,
            "sample": (f"layer {L.name}: norms+selection over its {L.num_groups} groups ({t_sel:.2f} s), search of the "
                       f"first {n} of its {dl.k} selected groups ({t_enc:.2f} s), dequantisation of the layer "
                       f"({t_deq:.2f} s); " + ("measured on the whole workload" if whole else
                       f"extrapolated to the workload's {G_total} groups (selection, dequantisation) and "
                       f"{pairs_total:.3e} codeword pairs (search), linearly")),
            "extrapolated": not whole,
            "pairs_per_s": n * L.pairs_per_group() / t_enc, "estimated_step_s": t_step}


def host_layers(kind):
    """Host arrays for the CPU arm: only the layer that is sampled is generated."""
    import numpy as np

    from oracle import pvt_oracle as oracle
    from paper_2405_14852_b200 import synth

    def nearest(X, C):
        return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]

    class HL:  # the fields of DeviceLayer that the CPU arm reads
        def __init__(self, L, tau):
            self.L, self.G, self.tau = L, L.num_groups, tau
            self.k = synth.subspace_size(tau, self.G)
            self.pairs = self.k * L.pairs_per_group()
            self.name, self.rows, self.cols, self.M, self.K = L.name, L.rows, L.cols, L.num_codebooks, L.codebook_size

    class Shape(HL):  # a layer that is only counted, never generated
        def __init__(self, name, rows, cols, M, K, tau):
            self.L = None
            self.G = rows * (cols // 8)
            self.tau = tau
            self.k = synth.subspace_size(tau, self.G)
            self.pairs = self.k * K
            self.name, self.rows, self.cols, self.M, self.K = name, rows, cols, M, K

    if kind[0] == "block":
        tau = kind[1]
        shapes = synth.block_layer_shapes()
        smallest = min(range(len(shapes)), key=lambda i: shapes[i][1] * shapes[i][2])
        out = []
        for i, (name, rows, cols, M, K, f16, rowmax) in enumerate(shapes):
            out.append(HL(synth.make_block_layer(i), tau) if i == smallest else
                       Shape(f"llama2_70b_{name}_{rows}x{cols}_1x16", rows, cols, M, K, tau))
        return out
    _, cfg, which, tau = kind
    name, rows, cols, M, K, f16, rowmax, _ = synth.CONFIGS[cfg][which]
    L = synth.make_layer(rows, cols, cfg=cfg, num_codebooks=M, codebook_size=K, codebook_fp16=f16,
                         row_max_scale=rowmax, nearest=nearest, name=name)
    return [HL(L, tau)]


def run_reference(args):
    """The CPU checker timed as the reference arm: every step is one bounded sample of the workload (selection
    over all groups of its smallest layer, search of n of that layer's selected groups for about two seconds,
    dequantisation of that layer), extrapolated linearly to the whole workload; value = groups re-encoded per
    second of that step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import pvt_oracle as oracle
    kind = workloads()[args.workload]
    layers = host_layers(kind)
    dl = min((l for l in layers if l.L is not None), key=lambda l: l.G)
    L = dl.L
    G_total, k_total, pairs_total = sum(l.G for l in layers), sum(l.k for l in layers), sum(l.pairs for l in layers)
    threads = oracle.num_threads()
    warm = max(args.warmup, 1)
    times = []
    n = None
    for i in range(warm + args.steps):
        idx, codes2, n, t_sel, t_enc, t_deq = _oracle_sample(oracle, L, dl.k, 2.0, probe=128)
        if i >= warm:
            times.append(_extrapolate(L, dl.k, n, t_sel, t_enc, t_deq, G_total, k_total, pairs_total))
    t_step = sum(times) / len(times)
    value = k_total / t_step
    whole = len(layers) == 1 and n == dl.k
    sample = (f"per step, layer {L.name}: norms+selection over its {L.num_groups} groups, search of the first {n} of "
              f"its {dl.k} selected groups, dequantisation of the layer; " +
              ("the whole workload" if whole else f"extrapolated linearly to {G_total} groups and {pairs_total:.3e} pairs"))
    first = layers[0]
    config = {"workload": args.workload,
              "layers": [{"name": l.name, "rows": l.rows, "cols": l.cols, "groups": l.G, "k": l.k} for l in layers],
              "group_dim": 8, "groups": G_total, "num_codebooks": first.M, "codebook_size": first.K,
              "codebook_dtype": "f16" if first.K > 256 or first.M > 1 else "f32",
              "tau": first.tau, "k": k_total, "pairs_per_step": pairs_total,
              "search_engine": "cpu checker (binary64)", "dequant_dtype": "f32",
              "l2": "not applicable", "launch": "host threads", "parallelism": "host cores"}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": warm, "ms_per_step": t_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "extrapolated": not whole},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- the calls beyond the V step proper


def run_next_rows(args):
    """Times the calls that widen the path (trust-ratio step, local search, three and four codebooks, groups of
    16 weights) on synthetic layers of the benchmark shapes and prints one JSON line.  Not the headline metric."""
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

    # trust-ratio step on the 4096 x 4096 layer (its random previous codes make every change large, so
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
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--search", default="auto", choices=["auto", "fp32", "tensor"],
                    help="engine of the single-codebook search")
    ap.add_argument("--dequant-fp16", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="never time a CUDA graph replay")
    ap.add_argument("--no-sub", action="store_true", help="leave out the 4096x4096 record with both search engines")
    ap.add_argument("--no-sweep", action="store_true", help="leave out the sweep over the single-layer workloads")
    ap.add_argument("--no-next", action="store_true", help="leave out the P-step kernels' timings")
    ap.add_argument("--only", action="store_true", help="the headline workload only (no sub, sweep, P step, CPU leg)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--list", action="store_true")
    ap.add_argument("--next-rows", action="store_true",
                    help="time the calls beyond the V step proper (trust-ratio step, local search, 3-4 codebooks, "
                         "groups of 16) instead of the headline metric")
    args = ap.parse_args()
    if args.only:
        args.no_sub = args.no_sweep = args.no_next = args.no_cpu_baseline = True
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
