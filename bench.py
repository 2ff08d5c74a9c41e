#!/usr/bin/env python
"""Benchmark of the paged GQA decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5a|c5b] [--impl ours|reference]

A step is one decode_attn call (plan + partition + merge kernels) over one synthetic batch whose
KV cache is resident in HBM.  Rank 0 prints ONE JSON line.  The metric is KV-cache GB/s: the
algorithmic bytes of the call (attended K+V rows, block-table entries touched, seq_lens, q, out,
lse) divided by the CUDA-event time.  With N > 1 (torchrun, one rank per GPU) every rank runs an
independent replica of the workload -- the path has no exchange step -- and the value is the sum
of the replicas' bytes over the slowest rank's time.

--impl reference times the fp64 CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "decode-attn KV-cache GB/s (fraction of 8 TB/s HBM); sequences/s per layer"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel come from the ncu captures
# summarised under profiles/; profiles/dram_traffic.txt lists them by kernel, workload and library version.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
WORKLOAD_TEXT = {
    "c1": "c1: 1 seq x 512 tok, page 16, contiguous, seed 0, 3 keys x20",
    "c2": "c2: 64 seqs, len U[1024,16384], 48q/8kv heads, d128, page 16, permuted pool, seed 1",
    "c3": "c3: 256 seqs, len log-uniform [512,32768], page 16, pages scattered in a ~20 GB pool, seed 2",
    "c4": "c4: 8 seqs x 131072 tok, page 64, seed 3",
    "c5a": "c5a: 128 seqs, 16384-token shared prefix + U[0,8192] suffix, page 16, full attention, seed 4",
    "c5b": "c5b: same as c5a with a sliding window of 8192",
}


# ----------------------------------------------------------------------------- helpers

def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def reduce_over_ranks(value: float, op: str, device) -> float:
    """max / sum of a scalar over all ranks (identity when not distributed)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_replicas(bytes_per_step: float, seqs_per_step: float, ms_per_step: float, device):
    """Whole-job numbers for independent replicas: units add up, time is the slowest rank's."""
    ms = reduce_over_ranks(ms_per_step, "max", device)
    total_bytes = reduce_over_ranks(bytes_per_step, "sum", device)
    total_seqs = reduce_over_ranks(seqs_per_step, "sum", device)
    return total_bytes / (ms * 1e-3) / 1e9, total_seqs / (ms * 1e-3), ms


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def ncu_traffic(kernel: str, workload: str, version: int):
    """(bytes per launch, library version of the capture) for the newest capture of `kernel` on `workload`
    listed in profiles/dram_traffic.txt; the bytes are None unless that capture is of the running version
    (the kernel may have changed since)."""
    best = None
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                fld = line.split()
                if len(fld) < 5 or fld[0].startswith("#") or fld[0] != kernel or fld[1] != workload:
                    continue
                ver, rd, wr = int(fld[2]), int(fld[3]), int(fld[4])
                if best is None or ver > best[1]:
                    best = (rd + wr, ver)
    except OSError:
        return None, None
    if best is None:
        return None, None
    return (best[0] if best[1] == version else None), best[1]


class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            text = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(case, every: int):
    """Time the CPU oracle, as it stands, on every `every`-th sequence of the workload."""
    import oracle
    ids = list(range(0, case.B, every))
    sub = workloads.host_subcase(case, ids)
    threads = oracle.max_threads()
    t0 = time.perf_counter()
    if sub.k_scale is not None:   # 8-bit cache
        ref, ref_lse = oracle.decode_attn_fp8kv_oracle(sub.q, sub.k_pages, sub.v_pages, sub.k_scale, sub.v_scale, sub.block_table,
                                        sub.seq_lens, sub.window, sub.scale, 0)
    else:
        ref, ref_lse = oracle.decode_attn_oracle(sub.q, sub.k_pages, sub.v_pages, sub.block_table, sub.seq_lens,
                                                 sub.window, sub.scale, 0)
    dt = time.perf_counter() - t0
    nbytes = sub.algorithmic_bytes(4)
    return {"ids": ids, "ref": ref, "ref_lse": ref_lse,
            "value": nbytes / dt / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"every {every}th sequence of {case.name} ({len(ids)} of {case.B} sequences, "
                      f"{int(sub.attended_tokens().sum())} attended tokens, {dt:.2f} s wall)",
            "seconds": dt, "seq_per_s": len(ids) / dt}


def parity_against(sample, out, lse):
    """The timed oracle run's result against the device result of the same sequences, element by element,
    at the fp32 bar |d| <= 1e-3 + 1e-3 |ref| (out and lse)."""
    ids = sample["ids"]
    worst, outside, n = 0.0, 0, 0
    for got, ref in ((out[ids].float().cpu().numpy().astype(np.float64), np.asarray(sample["ref"], dtype=np.float64)),
                     (lse[ids].float().cpu().numpy().astype(np.float64), np.asarray(sample["ref_lse"], dtype=np.float64))):
        both_ninf = np.isneginf(got) & np.isneginf(ref)
        ref0 = np.where(both_ninf, 0.0, ref)
        with np.errstate(invalid="ignore"):
            err = np.where(both_ninf, 0.0, np.abs(got - ref0))
        outside += int((~(err <= 1e-3 + 1e-3 * np.abs(ref0))).sum())
        worst = max(worst, float(np.nanmax(err)) if err.size else 0.0)
        n += err.size
    return {"max_abs_err": worst, "outside_tolerance": outside, "elements": n, "sequences": len(ids),
            "tolerance": "|d| <= 1e-3 + 1e-3 |oracle|, out and lse"}


def kv_text(args) -> str:
    return "; KV cache as FP8 E4M3 codes with per-KV-head fp32 factors" if args.kv == "fp8" else ""


def make_case(args, device, workload=None):
    workload = workload or args.workload
    if args.kv == "fp8":
        if workload == "c1":
            raise SystemExit("--kv fp8: c1 is a bf16 parity configuration")
        return workloads.RECIPES[workload](device, kv_dtype="fp8")
    return workloads.RECIPES[workload](device)


# ----------------------------------------------------------------------------- reference arm

def run_reference(args):
    rank, world, local = dist_env()
    if rank != 0:
        return 0
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    case = make_case(args, dev)
    every = max(args.ref_every, 1)
    # a step = the oracle over every `every`-th sequence of the workload (all 64 of c2: about half a second
    # on 16 cores), so K steps after W warm-up runs stay within a few minutes
    for _ in range(args.warmup):
        oracle_sample(case, every)
    res = [oracle_sample(case, every) for _ in range(max(1, args.steps))]
    best = dict(res[0])
    sec = statistics.mean(r["seconds"] for r in res)      # the line's value is bytes over the MEAN step time
    best["value"] = best["value"] * best["seconds"] / sec
    best["seq_per_s"] = best["seq_per_s"] * best["seconds"] / sec
    ms = sec * 1e3
    nbytes_ref = case.algorithmic_bytes(4)
    line = {
        "impl": "reference", "metric": METRIC, "value": best["value"], "unit": "GB/s", "n_gpus": args.gpus,
        "steps": len(res), "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        # the same keys and values as the other arm's line for this workload (what was sampled is in cpu_baseline)
        "config": {"workload": WORKLOAD_TEXT[args.workload] + kv_text(args), "sequences": case.B,
                   "attended_tokens": int(case.attended_tokens().sum()), "algorithmic_bytes": nbytes_ref,
                   "l2": "inputs exceed L2 (no flush)" if nbytes_ref > 4 * 126e6 else "inputs fit L2; not flushed",
                   "parallelism": "replicas only" if world > 1 else "1 GPU", "grid_blocks": 0,
                   "path": "decode_attn_fp8kv" if args.kv == "fp8" else "decode_attn"},
        "seq_per_s": best["seq_per_s"], "frac_of_8TBs": best["value"] / NOMINAL_HBM_GBS,
        "cpu_baseline": {k: best[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": best["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------- our arm

def run_ours(args):
    import paper_2512_10977_b200 as da   # raises if the CUDA library is missing

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    line = measure(args, da, args.workload, device, rank, world, local, with_cpu=world == 1 and not args.no_cpu_baseline)
    plain = not (args.extend or args.cascade or args.flush_l2 or args.kv == "fp8")
    if plain and args.workload == "c2" and not args.no_also:
        # the metric's target names two workloads; the second one rides along in the same line
        c3 = measure(args, da, "c3", device, rank, world, local, with_cpu=False)
        if rank == 0:
            keys = ("value", "unit", "ms_per_step", "frac_of_8TBs", "seq_per_s", "roofline", "e2e", "clocks",
                    "gpu_launches", "steps")
            line["also"] = {"c3": dict({k: c3[k] for k in keys}, workload=c3["config"]["workload"],
                                       algorithmic_bytes=c3["config"]["algorithmic_bytes"])}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def measure(args, da, workload, device, rank, world, local, with_cpu):
    """Times one workload on this rank (device-resident, dominant kernel alone, end to end) and returns
    rank 0's JSON line for it (None on the other ranks)."""
    case = make_case(args, device, workload)
    kv8 = args.kv == "fp8"
    out = torch.empty(case.q.shape, dtype=torch.float32, device=device)
    lse = torch.empty(case.q.shape[:2], dtype=torch.float32, device=device)
    nbytes = case.algorithmic_bytes(4)
    stream = torch.cuda.current_stream()
    lib = da.lib()

    prefix = 0
    if args.cascade:
        if workload != "c5a":
            raise SystemExit("--cascade applies to the shared-prefix workload c5a (full attention)")
        prefix = 16384
        da.set_option("cascade_overlap", args.cascade_overlap)

    Lq = int(args.extend)
    if Lq:
        if prefix or case.window:
            raise SystemExit("--extend takes a workload without window, and not --cascade")
        if int(case.lens.min()) < Lq:
            raise SystemExit("--extend: every sequence must hold at least that many tokens")
        q_ext = torch.randn((case.B, Lq) + tuple(case.q.shape[1:]), device=device,
                            generator=torch.Generator(device=device).manual_seed(7)).to(torch.bfloat16)
        out = torch.empty(q_ext.shape, dtype=torch.float32, device=device)
        lse = torch.empty(q_ext.shape[:3], dtype=torch.float32, device=device)
        Hq_, Dh_ = case.q.shape[1], case.q.shape[2]
        nbytes += case.B * (Lq - 1) * (Hq_ * Dh_ * 2 + Hq_ * Dh_ * 4 + Hq_ * 4)   # the extra queries' q, out, lse

    def step():
        if Lq and kv8:
            da.decode_attn_fp8kv_extend_wide(q_ext, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                        case.block_table, case.seq_lens, case.scale, out=out, lse=lse, stream=stream)
        elif Lq:
            da.decode_attn_extend(q_ext, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                  case.scale, out=out, lse=lse, stream=stream)
        elif prefix and kv8:
            da.decode_attn_fp8kv_cascade(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                         case.seq_lens, prefix, case.scale, out=out, lse=lse, stream=stream)
        elif prefix:
            da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                   prefix, case.scale, out=out, lse=lse, stream=stream)
        elif kv8:
            da.decode_attn_fp8kv(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                 case.seq_lens, case.window, case.scale, out=out, lse=lse, stream=stream)
        else:
            da.decode_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                           case.window, case.scale, out=out, lse=lse, stream=stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    assert da.read_device_status() == (0, 0, 0, 0)

    # ---- device-resident timing: K steps, events on the launching stream
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    K = args.steps
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    kev0 = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    kev1 = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    for e in kev0 + kev1:     # materialise the handles
        e.record(stream)
    barrier()
    launches0 = da.launch_count()
    t_all0 = torch.cuda.Event(enable_timing=True)
    t_all1 = torch.cuda.Event(enable_timing=True)
    # --flush-l2: a 512 MB write between steps evicts the 126 MB L2 (for workloads whose inputs fit it or
    # are partly re-read from it); the flush itself is outside every step's events
    flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device=device) if args.flush_l2 else None

    def flush():
        if flush_buf is not None:
            flush_buf.zero_()

    # The timed region: exactly K steps between two events, nothing else on the stream (an event
    # recorded between two calls would keep the next call's first kernel from being placed while the
    # previous call's last kernel drains).  With --flush-l2 every step needs its own pair of events,
    # so that the flush stays outside them.
    t_all0.record(stream)
    for i in range(K):
        if flush_buf is not None:
            flush()
            starts[i].record(stream)
        step()
        if flush_buf is not None:
            stops[i].record(stream)
    t_all1.record(stream)
    barrier()
    launches = da.launch_count() - launches0
    ms_total = t_all0.elapsed_time(t_all1)
    if flush_buf is None:
        # per-step figures (median, minimum) from a second pass with an event pair around every step
        for i in range(K):
            starts[i].record(stream)
            step()
            stops[i].record(stream)
        torch.cuda.synchronize()
    per_step = [a.elapsed_time(b) for a, b in zip(starts, stops)]
    ms_per_step = sum(per_step) / K if args.flush_l2 else ms_total / K

    # ---- the partition kernel alone (the dominant kernel), bracketed inside the library
    kernel_ms = None
    if hasattr(lib, "decode_attn_set_profile_events"):
        import ctypes
        lib.decode_attn_set_profile_events.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        durs = []
        for i in range(K):
            flush()
            lib.decode_attn_set_profile_events(kev0[i].cuda_event, kev1[i].cuda_event)
            step()
        lib.decode_attn_set_profile_events(None, None)
        torch.cuda.synchronize()
        durs = [a.elapsed_time(b) for a, b in zip(kev0, kev1)]
        kernel_ms = statistics.mean(durs)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: per-step inputs from pinned host memory, result read back to the host
    q_src = q_ext if Lq else case.q
    q_h, bt_h, sl_h = (t.cpu().pin_memory() for t in (q_src, case.block_table, case.seq_lens))
    out_h = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    h2d = q_h.numel() * 2 + bt_h.numel() * 4 + sl_h.numel() * 4
    d2h = out_h.numel() * 4 + lse_h.numel() * 4

    q_d, bt_d, sl_d = (torch.empty_like(t, device=device) for t in (q_h, bt_h, sl_h))

    def e2e_step():
        if Lq:
            q_d.copy_(q_h, non_blocking=True); bt_d.copy_(bt_h, non_blocking=True); sl_d.copy_(sl_h, non_blocking=True)
            if kv8:
                da.decode_attn_fp8kv_extend_wide(q_d, case.k_pages, case.v_pages, case.k_scale, case.v_scale, bt_d, sl_d,
                                            case.scale, out=out, lse=lse, stream=stream)
            else:
                da.decode_attn_extend(q_d, case.k_pages, case.v_pages, bt_d, sl_d, case.scale, out=out, lse=lse,
                                      stream=stream)
            out_h.copy_(out, non_blocking=True); lse_h.copy_(lse, non_blocking=True)
        elif prefix:   # the cascade has no host-io entry point: same copies, made here on the same stream
            q_d.copy_(q_h, non_blocking=True); bt_d.copy_(bt_h, non_blocking=True); sl_d.copy_(sl_h, non_blocking=True)
            if kv8:
                da.decode_attn_fp8kv_cascade(q_d, case.k_pages, case.v_pages, case.k_scale, case.v_scale, bt_d, sl_d,
                                             prefix, case.scale, out=out, lse=lse, stream=stream)
            else:
                da.decode_attn_cascade(q_d, case.k_pages, case.v_pages, bt_d, sl_d, prefix, case.scale,
                                       out=out, lse=lse, stream=stream)
            out_h.copy_(out, non_blocking=True); lse_h.copy_(lse, non_blocking=True)
        elif kv8:
            da.decode_attn_fp8kv_host_io(q_h, case.k_pages, case.v_pages, case.k_scale, case.v_scale, bt_h, sl_h,
                                         case.window, case.scale, out_h, lse_h, stream=stream)
        else:
            da.decode_attn_host_io(q_h, case.k_pages, case.v_pages, bt_h, sl_h, case.window, case.scale,
                                   out_h, lse_h, stream=stream)

    for _ in range(3):
        e2e_step()
    barrier()
    if args.flush_l2:
        ee0 = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        ee1 = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        for i in range(K):
            flush()
            ee0[i].record(stream)
            e2e_step()
            ee1[i].record(stream)
        barrier()
        e2e_ms = sum(a.elapsed_time(b) for a, b in zip(ee0, ee1)) / K
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / K
    # (not bit for bit: the host-buffer call folds two-piece pairs inside the partition kernel, the
    #  device-resident one in the merge kernel -- the same sums in another order)
    assert torch.allclose(out_h, out.cpu(), atol=2e-5, rtol=1e-4), "host-io result differs from the device-resident call"

    gbs, seqs, ms = aggregate_replicas(nbytes, case.B, ms_per_step, device)
    e2e_gbs, _, e2e_ms_max = aggregate_replicas(nbytes, case.B, e2e_ms, device)

    if rank != 0:
        return None
    peak, peak_src = measured_peak()
    kms = kernel_ms if kernel_ms is not None else ms_per_step
    achieved = nbytes / (kms * 1e-3) / 1e9
    kname = "partition_kernel_fp8" if kv8 else "partition_kernel"
    traffic, traffic_ver = ncu_traffic(kname, workload, da.version())
    roofline = {"bound": "hbm", "kernel": "partition_kernel (8-bit cache)" if kv8 else "partition_kernel",
                "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                "kernel_ms": kms, "traffic": traffic, "traffic_capture_library_version": traffic_ver,
                "library_version": da.version()}
    G_ = case.q.shape[1] // case.k_pages.shape[1]
    ext_stream = bool(Lq) and ((kv8 and Lq * G_ <= 48) or Lq * G_ <= da.get_option("extend_stream_rows"))
    if ext_stream:
        # a few new tokens ride through the streaming kernels as a wider group: still bound by HBM
        roofline["kernel"] = f"partition_kernel ({Lq} query tokens x {G_} heads per KV head)"
        roofline["traffic"] = None   # the ncu capture is of the single-token call
    elif Lq:
        # one kernel, a dense causal contraction: algorithmic flops = QK^T and PV over each query's keys
        Hq, Dh = case.q.shape[1], case.q.shape[2]
        keys = sum(float(L - Lq) * Lq + Lq * (Lq + 1) / 2.0 for L in case.lens)
        flops = 4.0 * Hq * Dh * keys
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                tpeak, tsrc = float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
        except Exception:
            tpeak, tsrc = 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"
        tf = flops / (kms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "prefix_kernel (extend mode)", "achieved": tf, "peak": tpeak,
                    "unit": "TFLOP/s", "frac": tf / tpeak, "peak_source": tsrc, "kernel_ms": kms, "traffic": None}
    if prefix:
        # the profile events bracket the prefix kernel: a dense contraction, measured against the
        # bf16 tensor peak.  Algorithmic flops: QK^T and PV once each over the shared prefix.
        Hq, Dh = case.q.shape[1], case.q.shape[2]
        flops = 4.0 * case.B * Hq * prefix * Dh
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                tpeak, tsrc = float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
        except Exception:
            tpeak, tsrc = 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"
        tf = flops / (kms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "prefix_kernel", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s",
                    "frac": tf / tpeak, "peak_source": tsrc, "kernel_ms": kms, "traffic": None,
                    "note": "the suffix pass (partition_kernel, HBM-bound) takes the larger share of the call"}
    line = {
        "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8 e4m3 (f32 accumulate)" if kv8 else "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[workload] + kv_text(args), "sequences": case.B,
                   "attended_tokens": int(case.attended_tokens().sum()), "algorithmic_bytes": nbytes,
                   "l2": ("flushed between steps (512 MB write, outside the timed events)" if args.flush_l2 else
                          ("inputs exceed L2 (no flush)" if nbytes > 4 * 126e6 else "inputs fit L2; not flushed")),
                   "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "grid_blocks": da.get_option("grid_blocks"),
                   "path": (f"decode_attn{'_fp8kv' if kv8 else ''}_extend, {Lq} new tokens per sequence (causal, " +
                            ("streaming kernels)" if ext_stream else
                             ("pages widened to bf16, then tcgen05)" if kv8 else "tcgen05)"))) if Lq else
                           (("cascade over the 8-bit cache (shared prefix widened to bf16, then tcgen05)" if kv8 else
                             "cascade (shared prefix on tcgen05)") if prefix else
                            ("decode_attn_fp8kv" if kv8 else "decode_attn"))},
    }
    if prefix:
        line["config"]["cascade_overlap"] = args.cascade_overlap
    if workload in ("c5a", "c5b") and not Lq:
        # sequences share prefix pages: `value` counts every sequence's reads (logical bytes); these count
        # each physical K/V row once
        uniq = case.unique_kv_bytes()
        line["config"]["unique_kv_bytes"] = uniq
        line["unique_kv_gbs"] = uniq * world / (ms * 1e-3) / 1e9
    line.update({
        "frac_of_8TBs": gbs / world / NOMINAL_HBM_GBS, "seq_per_s": seqs,
        "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
        "roofline": roofline,
        "e2e": {"value": e2e_gbs, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms_max,
                "note": "q, block_table, seq_lens from pinned host memory and out, lse back to it every step; "
                        "the KV cache is resident state"},
        "gpu_launches": launches, "clocks": clocks,
    })
    if with_cpu:
        sample = oracle_sample(case, args.ref_every)
        line["cpu_baseline"] = {k: v for k, v in sample.items() if k in ("value", "unit", "cores", "kind", "sample")}
        if not Lq:
            # the oracle's result for those sequences is at hand: compare it with what the timed calls wrote
            # (the cascade computes plain decode attention, so the same oracle serves it)
            line["parity"] = parity_against(sample, out, lse)
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOAD_TEXT))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-every", type=int, default=1, help="oracle sample: every n-th sequence")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="default run: do not time c3 beside c2")
    ap.add_argument("--extend", type=int, default=0, metavar="LQ",
                    help="time decode_attn_extend with LQ new (causal) query tokens per sequence instead of decode_attn")
    ap.add_argument("--flush-l2", action="store_true",
                    help="write 512 MB between steps so that every step starts with a cold L2 (c1, c5a, c5b)")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"],
                    help="cache element type: bf16 (decode_attn, the headline) or fp8 (decode_attn_fp8kv)")
    ap.add_argument("--cascade", action="store_true",
                    help="c5a only: attend the shared 16384-token prefix once for the batch (decode_attn_cascade)")
    ap.add_argument("--cascade-overlap", type=int, default=1, choices=[0, 1, 2],
                    help="--cascade: the library's option of that name (0: the two passes one after the other, "
                         "1: side by side where the library's estimate favours it, 2: wherever the shapes allow)")
    args = ap.parse_args()
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
