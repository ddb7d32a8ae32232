#!/usr/bin/env python
"""Benchmark of the aggregation primitive (AP) hot path on B200.

One step = one forward AP (mean) + one backward AP (mean) over a synthetic graph shaped like the
paper's Reddit workload (232,965 vertices, 114,615,892 directed edges, 602 features), through
the C ABI of libdgagg.  The graph ingest and the CSR->CSC build run once per graph (as in
training, where the graph is static over epochs); they are timed separately and reported under
"ingest".  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload NAME] [--scale S] [--feat F] [--op sum|mean] [--dtype f32|bf16]
                  [--set knob=value ...] [--sorted-ids] [--epochs E] [--e2e-steps S]
                  [--no-cpu-baseline] [--no-probe] [--workloads all|none]
  python bench.py --probe        # only the gather ceilings of this GPU

Beside the device-resident step the line carries: the roofline object of the slower of the two
calls (compulsory bytes, DRAM traffic from the ncu captures, gather ceilings measured in the
same run), the same step end to end from pinned host memory ("e2e"), the CPU oracle on a row
sample ("cpu_baseline"), the time of one full-batch GraphSAGE epoch ("epoch"), and, in the
default run on one GPU, "workloads": one record per workload shape of the paper's Table 2 at
full size (the tiny graph, Reddit-like at both layer widths, Products-like, Proteins-like at
three widths, Papers-like), each with forward and backward times, compulsory bytes, roofline
fractions, its own clock record and a sampled CPU-oracle time.

N > 1 (under torchrun): the path has no exchange step and is not sharded, so every rank runs
an independent replica of the same workload; the value is the units all ranks processed over
the slowest rank's time.
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

METRIC = "ap_fwd_bwd_edge_feat_per_s"
UNIT = "edge*feat/s"
NOMINAL_HBM_GBS = 8000.0
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
KERNEL_SOURCES = ["dg_aggregate_kernels.cuh", "dg_aggregate.cu", "dg_aggregate_fold.cu"]


def kernel_source_hash():
    """sha256 over the files that hold the aggregation kernels and their launch shapes: a
    capture is only quoted for the kernels it was taken with."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2104_06700_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload, F, op, scale, direction):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one dg_aggregate_fwd / _bwd
    call, summed over its launches, from the ncu captures whose figures are kept in
    profiles/dram_traffic.txt (the same file the tables under profiles/ quote).  None when no
    capture exists for the workload or the kernel sources have changed since it was taken."""
    if not os.path.exists(TRAFFIC_FILE):
        return None
    want_hash = kernel_source_hash()
    with open(TRAFFIC_FILE) as f:
        for line in f:
            t = line.split("#")[0].split()
            if len(t) != 8:
                continue
            wl, f_, op_, sc, src_hash, fwd, bwd, factor = t
            if (wl, int(f_), op_, float(sc)) == (workload, F, op, float(scale)) and src_hash == want_hash:
                return float({"fwd": fwd, "bwd": bwd}[direction]) * float(factor)
    return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="reddit_like")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--feat", type=int, default=0, help="feature width (0 = the workload's)")
    ap.add_argument("--op", default=None, choices=[None, "sum", "mean"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--epochs", type=int, default=5,
                    help="GraphSAGE epochs to time after 3 warm-up epochs (0 = skip)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0,
                    help="target CPU time of the oracle sample")
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"],
                    help="storage of the gathered matrices (sums and outputs are fp32 either "
                         "way); bf16 is reported separately, the headline is f32")
    ap.add_argument("--no-probe", action="store_true",
                    help="skip the two gather-ceiling measurements added to the roofline object")
    ap.add_argument("--probe", action="store_true",
                    help="measure the gather ceilings of this GPU (dg_probe_gather) and exit")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sorted-ids", action="store_true",
                    help="keep the generator's construction order of vertex ids (communities "
                         "contiguous) instead of a random permutation; reported separately")
    ap.add_argument("--reorder", default="none", choices=["none", "out_degree", "in_degree"],
                    help="rename the vertices hub-first with dg_graph_reorder before the run "
                         "(reported separately)")
    ap.add_argument("--other-calls", action="store_true",
                    help="also time dg_aggregate_edge_grad and two dg_ap_fwd operator pairs on "
                         "the chosen workload (the default run does so on the headline workload "
                         "and on two others)")
    ap.add_argument("--workloads", default="all", choices=["all", "none"],
                    help="all: after the headline step, one record per workload shape at full "
                         "size (default run on one GPU only); none: the headline alone")
    ap.add_argument("--set", action="append", default=[],
                    help="library knob name=value (heavy_threshold, slice_features, rows_per_block)")
    return ap.parse_args()


def default_op(workload):
    return {"reddit_like": "mean", "products_like": "mean"}.get(workload, "sum")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def compulsory_bytes(n, nnz, F, weighted, n_ref, inv_deg_gather, in_bytes=4):
    """Bytes one AP call must move once: pointers, indices, weights, the referenced rows of the
    input matrix read once, the output written once (+ the 1/deg vector for the mean backward)."""
    b = (n + 1) * 8 + nnz * 4 + (nnz * 4 if weighted else 0) + n_ref * F * in_bytes + n * F * 4
    if inv_deg_gather:
        b += n * 4
    return b


def device_memory_bytes(torch):
    if torch.cuda.is_available():
        return torch.cuda.get_device_properties(torch.cuda.current_device()).total_memory
    return 183e9


def workload_config(args, sg, F, op, weighted, world, two_buffers):
    """The `config` object of the JSON line: the same for both arms on the same workload."""
    return {"workload": args.workload, "scale": args.scale, "n": sg.n, "nnz": sg.nnz, "F": F,
            "op": op, "weighted": weighted, "step": "fwd AP + bwd AP", "replicas": world,
            "sorted_ids": bool(args.sorted_ids), "reorder": args.reorder,
            "buffers": "H=dOut, out=dH (two n x F buffers)" if two_buffers
                       else "H, out, dOut, dH separate",
            "l2": "inputs larger than L2 (no flush needed)" if sg.n * F * 4 > 252e6
                  else "inputs fit L2: warm-L2 numbers",
            "knobs": args.set}


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """Slowest rank's time: all-reduce(MAX) over the default process group (NCCL on GPUs, gloo in
    the CPU tests); the identity for one rank."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_step: float, ms_per_step: float, world: int) -> float:
    """Units all replicas processed per second: every rank runs the same workload (weak scaling)
    and the step time is the slowest rank's."""
    return world * units_per_step / (ms_per_step * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def oracle_sample(sg_host, H, G, op_code, n_rows, seed=0):
    """Runs the oracle (forward over sampled rows, backward over sampled columns) and returns
    (edge*feat processed, seconds)."""
    import numpy as np
    import oracle
    rowptr, colidx, w, colptr, rowidx_T, w_T = sg_host
    n = rowptr.shape[0] - 1
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(n, size=min(n_rows, n), replace=False))
    F = H.shape[1]
    work = int((rowptr[rows + 1] - rowptr[rows]).sum() + (colptr[rows + 1] - colptr[rows]).sum()) * F
    t0 = time.perf_counter()
    oracle.ap_forward(rowptr, colidx, w, H, op_code, rows=rows)
    oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op_code, cols=rows)
    return work, time.perf_counter() - t0


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2104_06700_b200 import synth
    op = args.op or default_op(args.workload)
    op_code = oracle.OP_MEAN if op == "mean" else oracle.OP_SUM
    import torch
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    sg = synth.make(args.workload, device=dev, scale=args.scale)
    F = args.feat or sg.F
    rowptr, colidx = sg.rowptr.cpu().numpy(), sg.colidx.cpu().numpy()
    w = None if sg.edge_w is None else sg.edge_w.cpu().numpy()
    colptr, rowidx_T, w_T, _ = oracle.transpose(rowptr, colidx, w)
    H = synth.features(sg.n, F, 100, "cpu").numpy()
    G = synth.features(sg.n, F, 101, "cpu").numpy()
    host = (rowptr, colidx, w, colptr, rowidx_T, w_T)
    # size the sample so that all steps together take about two minutes at most
    work, sec = oracle_sample(host, H, G, op_code, 64)
    per_row = sec / 64
    budget = min(args.cpu_seconds, 120.0 / max(1, args.steps + args.warmup))
    n_rows = int(max(64, min(sg.n, budget / max(per_row, 1e-9))))
    for i in range(args.warmup):
        oracle_sample(host, H, G, op_code, n_rows, seed=i)
    tot_work, tot_sec = 0, 0.0
    for i in range(args.steps):
        wk, sc = oracle_sample(host, H, G, op_code, n_rows, seed=1000 + i)
        tot_work += wk
        tot_sec += sc
    value = tot_work / tot_sec
    sample = f"{n_rows} sampled destination rows (fwd) and source columns (bwd) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_sec / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": workload_config(args, sg, F, op, w is not None, 1,
                                  4 * sg.n * F * 4 > 0.6 * device_memory_bytes(torch)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def probe_rate(binding, torch, dev, table_bytes, row_floats, count=1 << 25, reps=3):
    """GB/s of gathered bytes dg_probe_gather reaches on a table of the given size."""
    rows = int(table_bytes // (row_floats * 4))
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    table = torch.zeros((rows, row_floats), dtype=torch.float32, device=dev)
    idx = torch.randint(0, rows, (count,), generator=gen, device=dev, dtype=torch.int32)
    sink = torch.empty(((count + 511) // 512) * 128, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(2):
        binding.dg_probe_gather(table, idx, sink)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(reps):
        binding.dg_probe_gather(table, idx, sink)
    b.record(stream)
    torch.cuda.synchronize()
    return count * row_floats * 4 / (a.elapsed_time(b) / reps * 1e-3) / 1e9


def run_probe():
    """Random-row gather rates of this GPU (one JSON line): from an L2-resident and an HBM-sized
    table and from a mix of the two (dg_probe_gather), and from a block's own and a cluster partner's shared memory
    (dg_probe_gather_smem), each also as bytes per clock per SM at the SM clock sampled meanwhile."""
    import torch
    from paper_2104_06700_b200 import binding
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    count = 1 << 26
    sink = torch.empty(((count + 511) // 512) * 128 + 16 * 128, dtype=torch.float32, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    out = {"probe": "dg_probe_gather / dg_probe_gather_smem", "gathers": count,
           "unit": "GB/s of gathered bytes; B/clk/SM at the sampled SM clock", "sms": sms}

    def timed(call, label, row_bytes):
        for _ in range(3):
            call()
        sampler = ClockSampler(dev.index or 0)
        sampler.start()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        reps = 0
        t0 = time.perf_counter()
        while reps < 5 or time.perf_counter() - t0 < 0.5:
            call()
            reps += 1
        b.record(stream)
        torch.cuda.synchronize()
        clk = sampler.stop()
        gbs = count * row_bytes / (a.elapsed_time(b) / reps * 1e-3) / 1e9
        mhz = clk.get("sm_mhz") or 0
        out[label] = {"GBs": gbs, "sm_mhz": mhz,
                      "B_per_clk_per_SM": gbs * 1e9 / (mhz * 1e6 * sms) if mhz else None}

    for label, table_bytes in (("l2_30MB", 30e6), ("hbm_16GB", 16e9)):
        for row_floats in (128, 64, 32, 16, 8):
            rows = int(table_bytes // (row_floats * 4))
            table = torch.zeros((rows, row_floats), dtype=torch.float32, device=dev)
            idx = torch.randint(0, rows, (count,), generator=gen, device=dev, dtype=torch.int32)
            timed(lambda: binding.dg_probe_gather(table, idx, sink), f"{label}_row{row_floats * 4}B",
                  row_floats * 4)
            del table, idx
            torch.cuda.empty_cache()
    # mixed traffic: a share of the gathers goes to a hot set that stays in L2, the rest anywhere in
    # an HBM-sized table (what a power-law graph does to the forward pass)
    rows, hot_rows = int(16e9 // 512), int(30e6 // 512)
    table = torch.zeros((rows, 128), dtype=torch.float32, device=dev)
    for share in (0.25, 0.5, 0.75):
        idx = torch.randint(0, rows, (count,), generator=gen, device=dev, dtype=torch.int32)
        hot = torch.randint(0, hot_rows, (count,), generator=gen, device=dev, dtype=torch.int32)
        pick = torch.rand(count, generator=gen, device=dev) < share
        idx = torch.where(pick, hot * (rows // hot_rows), idx)
        del hot, pick
        timed(lambda: binding.dg_probe_gather(table, idx, sink),
              f"mixed_hbm_16GB_hot_30MB_share{int(share * 100)}_row512B", 512)
        del idx
    del table
    torch.cuda.empty_cache()
    for remote in (False, True):
        for row_floats in (128, 32, 16, 8):
            stage_rows = (192 * 1024) // (row_floats * 4)
            idx = torch.randint(0, stage_rows, (count,), generator=gen, device=dev, dtype=torch.int32)
            timed(lambda: binding.dg_probe_gather_smem(row_floats, stage_rows, idx, sink, remote),
                  f"smem_{'remote' if remote else 'local'}_192KB_row{row_floats * 4}B", row_floats * 4)
            del idx
    print(json.dumps(out))


def distinct_counts(torch, sg):
    """(distinct sources referenced, non-empty rows): what the compulsory-bytes formula needs."""
    seen = torch.zeros(sg.n, dtype=torch.bool, device=sg.colidx.device)
    for s0 in range(0, sg.nnz, 1 << 28):
        seen[sg.colidx[s0:s0 + (1 << 28)].long()] = True
    n_ref = int(seen.sum())
    del seen
    return n_ref, int(((sg.rowptr[1:] - sg.rowptr[:-1]) > 0).sum())


def sub_problem(torch, ptr, idx, w, seg_ids):
    """The segments `seg_ids` of a CSR / CSC (device tensors) as a compact problem on the host:
    (sub_ptr, neighbour ids renumbered 0..k-1, weights, device tensor of the k distinct ids)."""
    seg = torch.as_tensor(seg_ids, device=ptr.device, dtype=torch.int64)
    lo, lens = ptr[seg], ptr[seg + 1] - ptr[seg]
    sub_ptr = torch.zeros(seg.numel() + 1, dtype=torch.int64, device=ptr.device)
    torch.cumsum(lens, 0, out=sub_ptr[1:])
    total = int(sub_ptr[-1])
    owner = torch.repeat_interleave(torch.arange(seg.numel(), device=ptr.device), lens)
    pos = lo[owner] + (torch.arange(total, device=ptr.device) - sub_ptr[owner])
    uniq, inv = torch.unique(idx[pos].long(), return_inverse=True)
    sub_w = None if w is None else w[pos].cpu().numpy()
    return sub_ptr.cpu().numpy(), inv.to(torch.int32).cpu().numpy(), sub_w, uniq


def oracle_sample_compact(torch, sg, csc, H, G, op_code, n_rows, seed=0):
    """The oracle on `n_rows` sampled destination rows (forward) and as many sampled source columns
    (backward), each given to it as a compact sub-problem, so that no full-size array has to
    fit the host (every output row depends only on its own segment).  Only the oracle calls are
    timed.  Returns (edge*feat processed, seconds)."""
    import numpy as np
    import oracle
    colptr, rowidx_T, w_T = csc
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(sg.n, size=min(n_rows, sg.n), replace=False))
    F = H.shape[1]
    work, sec = 0, 0.0
    for ptr, idx, w, X, fwd in ((sg.rowptr, sg.colidx, sg.edge_w, H, True),
                                (colptr, rowidx_T, w_T, G, False)):
        sp, si, sw, uniq = sub_problem(torch, ptr, idx, w, rows)
        k = max(len(rows), uniq.numel())
        ptr_k = np.full(k + 1, sp[-1], dtype=np.int64)
        ptr_k[:len(sp)] = sp
        Xk = np.zeros((k, F), dtype=np.float32)
        Xk[:uniq.numel()] = X[uniq].float().cpu().numpy()
        sel = np.arange(len(rows))
        work += int(sp[-1]) * F
        if fwd:
            t0 = time.perf_counter()
            oracle.ap_forward(ptr_k, si, sw, Xk, op_code, rows=sel)
            sec += time.perf_counter() - t0
        else:
            # the mean's divisor is the in-degree of the destination: a CSR row pointer that
            # gives every renumbered destination its true in-degree
            deg = (sg.rowptr[uniq + 1] - sg.rowptr[uniq]).cpu().numpy()
            rp = np.zeros(k + 1, dtype=np.int64)
            rp[1:len(deg) + 1] = np.cumsum(deg)
            rp[len(deg) + 1:] = rp[len(deg)]
            t0 = time.perf_counter()
            oracle.ap_backward(rp, ptr_k, si, sw, Xk, op_code, cols=sel)
            sec += time.perf_counter() - t0
    return work, sec


def cpu_baseline_sampled(torch, sg, csc, H, G, op, seconds):
    """cpu_baseline record of one workload: the oracle on a row sample of about `seconds`."""
    import oracle
    o_op = oracle.OP_MEAN if op == "mean" else oracle.OP_SUM
    wk, sc = oracle_sample_compact(torch, sg, csc, H, G, o_op, 256)
    n_rows = int(max(256, min(sg.n, seconds * 256 / max(sc, 1e-6))))
    wk, sc = oracle_sample_compact(torch, sg, csc, H, G, o_op, n_rows, seed=1)
    return {"value": wk / sc, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n_rows} of {sg.n} destination rows (fwd) and source columns (bwd) as "
                      f"compact sub-problems, {sc:.1f} s, fp64 accumulation"}


def median(xs):
    xs = sorted(xs)
    return xs[len(xs) // 2] if len(xs) % 2 else 0.5 * (xs[len(xs) // 2 - 1] + xs[len(xs) // 2])


def direction_record(ms_list, comp_bytes, gather_bytes, units, peak, ceilings):
    med, best = median(ms_list), min(ms_list)
    r = {"ms_median": med, "ms_best": best, "compulsory_bytes": comp_bytes,
         "GBs": comp_bytes / med / 1e6, "frac_of_measured": comp_bytes / med / 1e6 / peak,
         "frac_of_8TBs": comp_bytes / med / 1e6 / NOMINAL_HBM_GBS,
         "edge_feat_per_s": units / (med * 1e-3), "gather_GBs": gather_bytes / med / 1e6}
    if ceilings:
        r["gather_frac_of_l2_ceiling"] = r["gather_GBs"] / ceilings["l2_GBs"]
        r["gather_frac_of_hbm_ceiling"] = r["gather_GBs"] / ceilings["hbm_GBs"]
    return r


def time_calls(torch, fwd_call, bwd_call, reps, flush, device_index):
    """Times `reps` forward and backward calls, each between its own pair of CUDA events on the
    current stream, with an L2 flush (a write larger than L2) before every call when `flush` is
    a buffer.  SM clocks are sampled while the region runs."""
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        fwd_call(); bwd_call()
    marks = [[ev() for _ in range(4)] for _ in range(reps)]
    sampler = ClockSampler(device_index)
    sampler.start()
    torch.cuda.synchronize()
    for m in marks:
        if flush is not None:
            flush.zero_()
        m[0].record(stream); fwd_call(); m[1].record(stream)
        if flush is not None:
            flush.zero_()
        m[2].record(stream); bwd_call(); m[3].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    return ([m[0].elapsed_time(m[1]) for m in marks], [m[2].elapsed_time(m[3]) for m in marks],
            clocks)


WORKLOAD_PLAN = [
    # name, feature widths, ops, epoch dims (or None), training share of the vertices, reorder
    ("tiny", (64,), ("sum", "mean"), None, None, None),
    ("reddit_like", (602, 256), ("mean",), None, None, None),
    ("products_like", (100, 256), ("sum", "mean"), [100, 256, 256, 47], 196615 / 2449029, None),
    # the same graph renamed hub-first by dg_graph_reorder (pre-processing, timed under ingest)
    ("products_like", (100, 256), ("sum", "mean"), [100, 256, 256, 47], 196615 / 2449029,
     "out_degree"),
    ("proteins_like", (8, 64, 256), ("sum",), None, None, None),
    ("papers_like", (128,), ("sum",), None, None, None),
]


def time_one(torch, call, reps, flush):
    """ms of `call` per repetition (median, best), each between its own pair of CUDA events."""
    stream = torch.cuda.current_stream()
    for _ in range(3):
        call()
    marks = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(reps)]
    torch.cuda.synchronize()
    for a, b in marks:
        if flush is not None:
            flush.zero_()
        a.record(stream); call(); b.record(stream)
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in marks]
    return median(ms), min(ms)


def extra_records(torch, binding, synth, name, g, sg, F, n_ref, peak, flush):
    """The calls beyond sum / mean on one loaded graph: the edge-weight gradient (one sampled dot
    product per edge, Section 2.2 of the paper) and the general AP of Table 1 with a full
    |E| x F edge-feature matrix (mul / sum) and with the max reducer (copylhs / max).  Compulsory
    bytes: index arrays, every referenced row once, the edge stream once, the output once."""
    dev = sg.colidx.device
    out = []
    H = synth.features(sg.n, F, 100, dev)
    G = synth.features(sg.n, F, 101, dev)
    cold = sg.n * F * 4 <= 252e6
    fl = flush if cold else None
    idx_bytes = (sg.n + 1) * 8 + sg.nnz * 4

    def rec(call_name, ms, comp, note):
        med, best = ms
        return {"workload": name, "F": F, "call": call_name, "ms_median": med, "ms_best": best,
                "compulsory_bytes": comp, "GBs": comp / med / 1e6,
                "frac_of_measured": comp / med / 1e6 / peak,
                "edge_feat_per_s": sg.nnz * F / (med * 1e-3), "note": note,
                "l2": "flushed before every call" if cold else "inputs larger than L2"}

    dW = torch.empty(sg.nnz, dtype=torch.float32, device=dev)
    ms = time_one(torch, lambda: g.dg_aggregate_edge_grad(H, G, binding.DG_OP_SUM, dW=dW), 10, fl)
    out.append(rec("dg_aggregate_edge_grad (sum)", ms,
                   idx_bytes + n_ref * F * 4 + sg.n * F * 4 + sg.nnz * 4,
                   "dW[k] = <H[u_k], dOut[v_k]>: both rows per edge, H[u] gathered"))
    del dW
    fO = torch.empty_like(H)
    arg = torch.empty((sg.n, F), dtype=torch.int32, device=dev)
    ms = time_one(torch, lambda: g.dg_ap_fwd(H, None, binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX,
                                             fO=fO, arg=arg), 10, fl)
    out.append(rec("dg_ap_fwd (copylhs, max) + arg", ms,
                   idx_bytes + n_ref * F * 4 + 2 * sg.n * F * 4, "element-wise max with arg indices"))
    if g.dg_graph_get_param("self_loops") == 0:
        try:
            g.dg_graph_get_csc()
            have_csc = True
        except binding.DgError:
            have_csc = False
        if have_csc:
            dV = torch.empty_like(H)
            bwd = lambda: binding._check(binding.lib().dg_ap_bwd(
                g._h, G.data_ptr(), H.data_ptr(), None, 1, F, binding.DG_BIN_COPY_LHS,
                binding.DG_RED_MAX, arg.data_ptr(), dV.data_ptr(), None,
                torch.cuda.current_stream().cuda_stream))
            ms = time_one(torch, bwd, 10, fl)
            out.append(rec("dg_ap_bwd (copylhs, max): dV", ms,
                           idx_bytes + sg.nnz * 4 + 3 * sg.n * F * 4,
                           "gather over the CSC with an equality test on arg (dO and arg rows per "
                           "edge), no atomics"))
            del dV
    del arg
    if sg.nnz * F * 4 <= 24e9:
        fE = torch.rand((sg.nnz, F), device=dev, dtype=torch.float32)
        ms = time_one(torch, lambda: g.dg_ap_fwd(H, fE, binding.DG_BIN_MUL, binding.DG_RED_SUM,
                                                 fO=fO), 10, None)
        out.append(rec("dg_ap_fwd (mul, sum), |E| x F edge features", ms,
                       idx_bytes + n_ref * F * 4 + sg.n * F * 4 + sg.nnz * F * 4,
                       "the edge stream (nnz x F x 4 bytes, read once) dominates: HBM-streaming bound"))
        dE = torch.empty_like(fE)
        bwd_e = lambda: binding._check(binding.lib().dg_ap_bwd(
            g._h, G.data_ptr(), H.data_ptr(), fE.data_ptr(), F, F, binding.DG_BIN_MUL,
            binding.DG_RED_SUM, None, None, dE.data_ptr(), torch.cuda.current_stream().cuda_stream))
        ms = time_one(torch, bwd_e, 10, None)
        out.append(rec("dg_ap_bwd (mul, sum): dE, |E| x F", ms,
                       idx_bytes + n_ref * F * 4 + sg.n * F * 4 + sg.nnz * F * 4,
                       "dE[k] = dO[v] * fV[u]: one written row per edge (nnz x F x 4 bytes) dominates"))
        del fE, dE
    return out


def run_workloads(torch, binding, synth, dev, device_index, peak, ceilings, cpu_seconds, skip):
    """One record per (workload, width, op) of WORKLOAD_PLAN at full size; `skip` names
    (workload, F, op) triples that the caller has measured already."""
    records, ingest, epochs, extras = [], {}, {}, []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for name, widths, ops, dims, frac, reorder in WORKLOAD_PLAN:
        torch.cuda.empty_cache()
        t0 = time.perf_counter()
        sg = synth.make(name, device=dev)
        torch.cuda.synchronize()
        gen_s = time.perf_counter() - t0
        torch.cuda.empty_cache()
        reorder_ms = None
        if reorder:
            g0 = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            renamed = g0.dg_graph_reorder(binding.DG_ORDER_OUT_DEGREE if reorder == "out_degree"
                                          else binding.DG_ORDER_IN_DEGREE)
            torch.cuda.synchronize()
            reorder_ms = 1e3 * (time.perf_counter() - t0)
            del g0
            sg.rowptr, sg.colidx, sg.edge_w = renamed.rowptr, renamed.colidx, renamed.edge_w
            torch.cuda.empty_cache()
        else:
            renamed = None
        label = name + (f" (reorder {reorder})" if reorder else "")
        tkey = name + (f"+{reorder}" if reorder else "")     # key in profiles/dram_traffic.txt
        weighted = sg.edge_w is not None
        n_ref, n_nonempty = distinct_counts(torch, sg)
        t0 = time.perf_counter()
        # the handle dg_graph_reorder returned knows that its rows are hub-first
        g = renamed if renamed is not None else binding.dg_graph_create(
            sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
        torch.cuda.synchronize()
        create_ms = None if renamed is not None else 1e3 * (time.perf_counter() - t0)
        need_csc, need_scratch = g.dg_graph_transpose_workspace()
        csc_buf = torch.empty(need_csc, dtype=torch.uint8, device=dev)
        scratch = torch.empty(need_scratch, dtype=torch.uint8, device=dev)
        g.dg_graph_transpose(csc_buf, scratch)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(torch.cuda.current_stream())
        g.dg_graph_transpose(csc_buf, scratch)
        e1.record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        ingest[label] = {"generate_s": gen_s, "graph_create_ms": create_ms,
                         "transpose_ms": e0.elapsed_time(e1),
                         "transpose_edges_per_s": sg.nnz / (e0.elapsed_time(e1) * 1e-3),
                         "reorder_ms": reorder_ms}
        del scratch
        torch.cuda.empty_cache()
        colptr, rowidx_T, w_T, _ = g.dg_graph_get_csc()
        for F in widths:
            mat_bytes = sg.n * F * 4
            two_buffers = 4 * mat_bytes > 0.6 * torch.cuda.get_device_properties(dev).total_memory
            H = synth.features(sg.n, F, 100, dev)
            out = torch.empty_like(H)
            G, dH = (H, out) if two_buffers else (synth.features(sg.n, F, 101, dev),
                                                  torch.empty_like(H))
            cold = mat_bytes <= 252e6          # inputs that would stay L2-resident: flush
            for op in ops:
                if (name, F, op) in skip:
                    continue
                code = binding.DG_OP_MEAN if op == "mean" else binding.DG_OP_SUM
                fwd_call = lambda: g.dg_aggregate_fwd(H, code, out=out)
                bwd_call = lambda: g.dg_aggregate_bwd(G, code, dH=dH)
                fwd_call(); bwd_call()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(torch.cuda.current_stream()); fwd_call(); bwd_call()
                b.record(torch.cuda.current_stream())
                torch.cuda.synchronize()
                est = max(a.elapsed_time(b), 1e-3)
                reps = int(min(200, max(5 if est > 100 else 10, 400.0 / est)))
                f_ms, b_ms, clocks = time_calls(torch, fwd_call, bwd_call, reps,
                                                flush if cold else None, device_index)
                b_fwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_ref, False)
                b_bwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_nonempty, op == "mean")
                rec = {"workload": name, "scale": 1.0, "n": sg.n, "nnz": sg.nnz, "F": F, "op": op,
                       "weighted": weighted, "reorder": reorder or "none", "dtype": "f32",
                       "reps": reps,
                       "l2": "flushed before every call (inputs fit L2)" if cold
                             else "inputs larger than L2 (no flush needed)",
                       "buffers": "H=dOut, out=dH (two n x F buffers)" if two_buffers
                                  else "H, out, dOut, dH separate",
                       "fwd": direction_record(f_ms, b_fwd, sg.nnz * F * 4, sg.nnz * F, peak, ceilings),
                       "bwd": direction_record(b_ms, b_bwd, sg.nnz * F * 4, sg.nnz * F, peak, ceilings),
                       "traffic": {"fwd": ncu_traffic(tkey, F, op, 1.0, "fwd"),
                                   "bwd": ncu_traffic(tkey, F, op, 1.0, "bwd")},
                       "clocks": clocks}
                rec["cpu_baseline"] = None if cpu_seconds <= 0 else cpu_baseline_sampled(
                    torch, sg, (colptr, rowidx_T, w_T), H, G, op, cpu_seconds)
                records.append(rec)
            # the gathered matrices stored as bf16 (sums and outputs fp32): the two largest graphs
            if (name, F, reorder) in (("products_like", 100, None), ("papers_like", 128, None)):
                if two_buffers:
                    # no room for a third matrix: the bf16 copy is packed into H's own storage,
                    # chunk by chunk from the front (H is not needed as fp32 after this point)
                    flat16 = H.view(-1).view(torch.bfloat16)
                    rows = max(1, (1 << 28) // F)
                    for s0 in range(0, sg.n, rows):
                        e0 = min(sg.n, s0 + rows)
                        tmp = H[s0:e0].to(torch.bfloat16)
                        flat16[s0 * F:e0 * F] = tmp.view(-1)
                        del tmp
                    Hb = flat16[:sg.n * F].view(sg.n, F)
                else:
                    Hb = H.to(torch.bfloat16)
                Gb = Hb if two_buffers else G.to(torch.bfloat16)
                for op in ops:
                    code = binding.DG_OP_MEAN if op == "mean" else binding.DG_OP_SUM
                    fwd_call = lambda: g.dg_aggregate_fwd_bf16(Hb, code, out=out)
                    bwd_call = lambda: g.dg_aggregate_bwd_bf16(Gb, code, dH=dH)
                    f_ms, b_ms, clocks = time_calls(torch, fwd_call, bwd_call, 5 if mat_bytes > 1e10 else 10,
                                                    None, device_index)
                    b_fwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_ref, False, 2)
                    b_bwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_nonempty, op == "mean", 2)
                    records.append({
                        "workload": name, "scale": 1.0, "n": sg.n, "nnz": sg.nnz, "F": F, "op": op,
                        "weighted": weighted, "reorder": "none",
                        "dtype": "f32 sums over bf16-stored inputs (not the fp32 headline)",
                        "reps": len(f_ms), "l2": "inputs larger than L2 (no flush needed)",
                        "fwd": direction_record(f_ms, b_fwd, sg.nnz * F * 2, sg.nnz * F, peak, None),
                        "bwd": direction_record(b_ms, b_bwd, sg.nnz * F * 2, sg.nnz * F, peak, None),
                        "traffic": {"fwd": None, "bwd": None}, "clocks": clocks,
                        "cpu_baseline": None})
                del Hb, Gb
            if dims and F == dims[0]:
                epochs[label] = epoch_plain(torch, g, sg, H, dims, frac, dev)
            del H, out, G, dH
            torch.cuda.empty_cache()
            if (name, F, reorder) in (("products_like", 100, None), ("proteins_like", 64, None)):
                extras += extra_records(torch, binding, synth, name, g, sg, F, n_ref, peak, flush)
                torch.cuda.empty_cache()
        del g, renamed, csc_buf, colptr, rowidx_T, w_T, sg
        torch.cuda.empty_cache()
    return records, ingest, epochs, extras


def epoch_plain(torch, g, sg, H, dims, frac, dev, epochs=5):
    """ms per full-batch GraphSAGE epoch in the paper's order (aggregate, then Linear)."""
    from paper_2104_06700_b200 import graphsage
    torch.manual_seed(1234)
    model = graphsage.GraphSAGE(g, dims).to(dev)
    labels = torch.randint(0, dims[-1], (sg.n,), device=dev)
    train_idx = torch.nonzero(torch.rand(sg.n, device=dev) < frac).flatten()
    run_epoch = graphsage.make_epoch(model, H, labels, train_idx)
    for _ in range(3):
        run_epoch()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(torch.cuda.current_stream())
    for _ in range(epochs):
        loss = run_epoch()
    b.record(torch.cuda.current_stream())
    torch.cuda.synchronize()
    calls = graphsage.aggregation_calls(dims)
    return {"ms_per_epoch": a.elapsed_time(b) / epochs, "epochs": epochs, "dims": dims,
            "loss": float(loss), "train_vertices": int(train_idx.numel()),
            "aggregations": [f"{d}:{w}" for d, w in calls],
            "aggregator": "(sum + self) / (deg + 1), then Linear; ReLU; Adam"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.probe:
        run_probe()
        return

    import torch
    import torch.distributed as dist
    from paper_2104_06700_b200 import binding, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the aggregation kernels have no fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    op = args.op or default_op(args.workload)
    op_code = binding.DG_OP_MEAN if op == "mean" else binding.DG_OP_SUM

    # ---------------------------------------------------------------- inputs (seeded, synthetic)
    extra = {"sorted_ids": True} if args.sorted_ids else {}
    sg = synth.make(args.workload, device=dev, scale=args.scale, **extra)
    torch.cuda.empty_cache()
    F = args.feat or sg.F
    weighted = sg.edge_w is not None
    n_ref, n_rows_nonempty = distinct_counts(torch, sg)
    reorder_ms = None
    if args.reorder != "none":
        g0 = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        renamed = g0.dg_graph_reorder(binding.DG_ORDER_OUT_DEGREE if args.reorder == "out_degree"
                                      else binding.DG_ORDER_IN_DEGREE)
        torch.cuda.synchronize()
        reorder_ms = 1e3 * (time.perf_counter() - t0)
        del g0
        # the run continues on the renamed graph (the features are random either way)
        sg.rowptr, sg.colidx, sg.edge_w = renamed.rowptr, renamed.colidx, renamed.edge_w
        torch.cuda.empty_cache()
    else:
        renamed = None
    mat_bytes = sg.n * F * 4
    # Four n x F matrices (H, out, dOut, dH) when they fit next to the graph; otherwise two, with
    # the backward pass reading the forward pass's input buffer and overwriting its output.
    two_buffers = 4 * mat_bytes > 0.6 * torch.cuda.get_device_properties(dev).total_memory

    # ---------------------------------------------------------------- ingest (once per graph)
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    g = renamed if renamed is not None else binding.dg_graph_create(
        sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
    torch.cuda.synchronize()
    create_ms = 1e3 * (time.perf_counter() - t0)
    for name_value in args.set:
        k, v = name_value.split("=")
        g.dg_graph_set_param(k, int(v))
    need_csc, need_scratch = g.dg_graph_transpose_workspace()
    csc = torch.empty(need_csc, dtype=torch.uint8, device=dev)
    scratch = torch.empty(need_scratch, dtype=torch.uint8, device=dev)
    g.dg_graph_transpose(csc, scratch)          # warm-up
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record(stream)
    g.dg_graph_transpose(csc, scratch)
    e1.record(stream)
    torch.cuda.synchronize()
    transpose_ms = e0.elapsed_time(e1)
    del scratch
    torch.cuda.empty_cache()
    bf16 = args.dtype == "bf16"
    H = synth.features(sg.n, F, 100, dev)
    out = torch.empty_like(H)
    if two_buffers:
        G, dH = H, out
    else:
        G = synth.features(sg.n, F, 101, dev)
        dH = torch.empty_like(H)
    if bf16:      # gathered matrices in bf16; the fp32 outputs keep their buffers
        H = H.to(torch.bfloat16)
        G = H if two_buffers else G.to(torch.bfloat16)
        torch.cuda.empty_cache()
    agg_fwd = g.dg_aggregate_fwd_bf16 if bf16 else g.dg_aggregate_fwd
    agg_bwd = g.dg_aggregate_bwd_bf16 if bf16 else g.dg_aggregate_bwd

    # ---------------------------------------------------------------- device-resident timing
    def step():
        agg_fwd(H, op_code, out=out)
        agg_bwd(G, op_code, dH=dH)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    def timed_region():
        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
        launches0 = binding.dg_kernel_launch_count()
        marks = [ev() for _ in range(2 * args.steps + 1)]
        torch.cuda.synchronize()
        marks[0].record(stream)
        for i in range(args.steps):
            agg_fwd(H, op_code, out=out)
            marks[2 * i + 1].record(stream)
            agg_bwd(G, op_code, dH=dH)
            marks[2 * i + 2].record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        n_launch = binding.dg_kernel_launch_count() - launches0
        clk = sampler.stop() if rank == 0 else None
        tot = marks[0].elapsed_time(marks[-1])
        f_list = [marks[2 * i].elapsed_time(marks[2 * i + 1]) for i in range(args.steps)]
        b_list = [marks[2 * i + 1].elapsed_time(marks[2 * i + 2]) for i in range(args.steps)]
        return tot, f_list, b_list, n_launch, clk

    def clocks_bad(clk):
        """Thermal or hardware slowdown, or SM clocks far below maximum with no reason given."""
        if not clk or clk.get("sm_mhz") is None:
            return False
        bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clk["reasons"])
        stuck = clk["sm_mhz"] < 0.7 * clk["sm_max_mhz"] and not clk["reasons"]
        return bool(bad) or stuck

    total_ms, fwd_list, bwd_list, launches, clocks = timed_region()
    remeasured = False
    if rank == 0 and world == 1 and clocks_bad(clocks):      # rejected: measure once more
        remeasured = True
        total_ms, fwd_list, bwd_list, launches, clocks = timed_region()
    fwd_ms, bwd_ms = sum(fwd_list) / len(fwd_list), sum(bwd_list) / len(bwd_list)
    if clocks is not None:
        clocks["remeasured"] = remeasured
        clocks["rejected"] = clocks_bad(clocks)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    units_per_step = 2 * sg.nnz * F                 # forward + backward edge*feature products
    value = whole_job_value(units_per_step, ms_per_step, world)

    # ---------------------------------------------------------------- roofline of the dominant kernel
    peak, peak_kind = measured_peaks()
    b_fwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_ref, False, 2 if bf16 else 4)
    b_bwd = compulsory_bytes(sg.n, sg.nnz, F, weighted, n_rows_nonempty, op == "mean",
                             2 if bf16 else 4)
    dom = "fwd" if fwd_ms >= bwd_ms else "bwd"
    dom_ms, dom_bytes = (fwd_ms, b_fwd) if dom == "fwd" else (bwd_ms, b_bwd)
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    # one dg_aggregate_* call is one launch, or one launch per source block (each launch then
    # handles that share of the edges and of the gathered matrix)
    per_call = max(1, round(launches / (2 * args.steps)))
    traffic = None
    if not bf16 and not args.set and not args.sorted_ids and args.reorder == "none":
        t = ncu_traffic(args.workload, F, op, args.scale, dom)
        traffic = None if t is None else t / per_call
    roofline = {
        "bound": "hbm",
        "kernel": ("ap_kernel_r40" if ((weighted or (dom == "bwd" and op == "mean")) and F >= 64)
                   or F <= 16 else "ap_kernel")
                  + f" ({dom}: {per_call} launch(es) per dg_aggregate_{dom} call)",
        "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "launches_per_call": per_call,
        "algorithmic_bytes_per_launch": dom_bytes / per_call, "ms_per_launch": dom_ms / per_call,
        "traffic": traffic,
        "fabric_peak_GBs": 148 * 64 * (clocks["sm_mhz"] or 0) * 1e6 / 1e9 if clocks else None,
        "fwd": {"ms": fwd_ms, "bytes": b_fwd, "GBs": b_fwd / fwd_ms / 1e6,
                "edge_feat_per_s": sg.nnz * F / (fwd_ms * 1e-3)},
        "bwd": {"ms": bwd_ms, "bytes": b_bwd, "GBs": b_bwd / bwd_ms / 1e6,
                "edge_feat_per_s": sg.nnz * F / (bwd_ms * 1e-3)},
        "gather_bytes_per_launch": sg.nnz * F * (2 if bf16 else 4),
        "gather_GBs": sg.nnz * F * (2 if bf16 else 4) / (dom_ms * 1e-3) / 1e9,
    }

    # what this GPU can deliver to a gather at all: the aggregation's own ceilings
    ceilings = None
    if rank == 0 and world == 1 and not args.no_probe and not two_buffers:
        l2_c = probe_rate(binding, torch, dev, 30e6, 128)
        hbm_c = probe_rate(binding, torch, dev, 8e9, 128)
        ceilings = {"l2_GBs": l2_c, "hbm_GBs": hbm_c}
        roofline["gather_ceilings"] = {
            "how": "dg_probe_gather, random 512-byte rows, 30 MB table (L2) and 8 GB table (HBM)",
            "l2_GBs": l2_c, "hbm_GBs": hbm_c,
            "gathered_frac_of_l2_ceiling": roofline["gather_GBs"] / l2_c,
            "gathered_frac_of_hbm_ceiling": roofline["gather_GBs"] / hbm_c}

    # ---------------------------------------------------------------- GraphSAGE epoch (composite)
    epoch_info = None
    epoch_dims = {"reddit_like": [602, 256, 41], "products_like": [100, 256, 256, 47],
                  "papers_like": [128, 256, 256, 172]}     # reduced scales only (memory)
    if (args.epochs > 0 and args.workload in epoch_dims and not args.feat and not two_buffers
            and not bf16):
        from paper_2104_06700_b200 import graphsage
        dims = epoch_dims[args.workload]
        frac = {"reddit_like": 0.65, "products_like": 196615 / 2449029,
                "papers_like": 0.011}[args.workload]          # training share of the vertices
        torch.manual_seed(1234)
        model = graphsage.GraphSAGE(g, dims).to(dev)
        labels = torch.randint(0, dims[-1], (sg.n,), device=dev)
        train_idx = torch.nonzero(torch.rand(sg.n, device=dev) < frac).flatten()
        run_epoch = graphsage.make_epoch(model, H, labels, train_idx)
        for _ in range(3):
            run_epoch()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(args.epochs):
            last_loss = run_epoch()
        b.record(stream)
        torch.cuda.synchronize()
        ep_ms = a.elapsed_time(b) / args.epochs
        calls = graphsage.aggregation_calls(dims)
        # the algebraically equal order for layers that narrow: Linear first, then aggregate
        torch.manual_seed(1234)
        model_pf = graphsage.GraphSAGE(g, dims, project_first=True).to(dev)
        run_pf = graphsage.make_epoch(model_pf, H, labels, train_idx)
        for _ in range(3):
            run_pf()
        torch.cuda.synchronize()
        a2, b2 = ev(), ev()
        a2.record(stream)
        for _ in range(args.epochs):
            run_pf()
        b2.record(stream)
        torch.cuda.synchronize()
        pf_calls = graphsage.aggregation_calls(dims, True)
        del model_pf, run_pf
        # the same, aggregating bf16-rounded activations (mixed precision; not the headline)
        torch.manual_seed(1234)
        model_bf = graphsage.GraphSAGE(g, dims, project_first=True, bf16_aggregate=True).to(dev)
        run_bf = graphsage.make_epoch(model_bf, H, labels, train_idx)
        for _ in range(3):
            run_bf()
        torch.cuda.synchronize()
        a3, b3 = ev(), ev()
        a3.record(stream)
        for _ in range(args.epochs):
            run_bf()
        b3.record(stream)
        torch.cuda.synchronize()
        del model_bf, run_bf
        # the aggregator fused into the library's kernels: a second handle over the same CSR
        # with the "self_loops" attribute (its CSC tabulates 1/(deg+1) for the mean's backward)
        g_self = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
        g_self.dg_graph_set_param("self_loops", 1)
        for kv in args.set:
            k, v = kv.split("=")
            g_self.dg_graph_set_param(k, int(v))
        g_self.dg_graph_transpose()
        fused_ms = {}
        for key, pf in (("aggregate_first", False), ("project_first", True)):
            torch.manual_seed(1234)
            model_f = graphsage.GraphSAGE(g_self, dims, project_first=pf,
                                          fused_aggregator=True).to(dev)
            run_f = graphsage.make_epoch(model_f, H, labels, train_idx)
            for _ in range(3):
                run_f()
            torch.cuda.synchronize()
            a4, b4 = ev(), ev()
            a4.record(stream)
            for _ in range(args.epochs):
                loss_f = run_f()
            b4.record(stream)
            torch.cuda.synchronize()
            fused_ms[key] = a4.elapsed_time(b4) / args.epochs
            fused_ms[key + "_loss"] = float(loss_f)
            del model_f, run_f
        del g_self
        epoch_info = {"ms_per_epoch": ep_ms, "epochs": args.epochs, "dims": dims,
                      "project_first": {"ms_per_epoch": a2.elapsed_time(b2) / args.epochs,
                                        "aggregations": [f"{d}:{w}" for d, w in pf_calls],
                                        "note": "Linear before the aggregation where a layer "
                                                "narrows; same function up to fp32 rounding",
                                        "ms_per_epoch_bf16_aggregation":
                                            a3.elapsed_time(b3) / args.epochs},
                      "fused_aggregator": {"ms_per_epoch": fused_ms["aggregate_first"],
                                           "ms_per_epoch_project_first": fused_ms["project_first"],
                                           "loss": fused_ms["aggregate_first_loss"],
                                           "note": "own row and 1/(deg+1) inside the aggregation "
                                                   "kernels (graph attribute self_loops)"},
                      "train_vertices": int(train_idx.numel()), "loss": float(last_loss),
                      "aggregations": [f"{d}:{w}" for d, w in calls],
                      "ap_edge_feat_per_epoch": sg.nnz * sum(w for _, w in calls),
                      "aggregator": "(sum + self) / (deg + 1), then Linear; ReLU; Adam"}
        del model, run_epoch

    # ---------------------------------------------------------------- end to end from host memory
    e2e = None
    if two_buffers:
        e2e = {"value": None, "unit": UNIT, "skipped": "host copies of the feature matrices of "
               "this workload exceed what the run pins; measured on the default workload"}
    elif args.e2e_steps > 0 and not bf16:
        Hh = torch.empty((sg.n, F), dtype=torch.float32).pin_memory()
        Gh = torch.empty((sg.n, F), dtype=torch.float32).pin_memory()
        Hh.copy_(H); Gh.copy_(G)
        outh = torch.empty_like(Hh).pin_memory()
        dHh = torch.empty_like(Hh).pin_memory()
        ws = torch.empty(g.dg_aggregate_host_workspace(F), dtype=torch.uint8, device=dev)
        g.dg_aggregate_host(Hh, Gh, op_code, outh, dHh, ws)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(args.e2e_steps):
            g.dg_aggregate_host(Hh, Gh, op_code, outh, dHh, ws)
        b.record(stream)
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b)
        e2e_ms = max_over_ranks(e2e_ms, world, dev) / args.e2e_steps
        e2e = {"value": whole_job_value(units_per_step, e2e_ms, world), "unit": UNIT,
               "h2d_bytes_per_step": 2 * sg.n * F * 4, "d2h_bytes_per_step": 2 * sg.n * F * 4,
               "ms_per_step": e2e_ms, "steps": args.e2e_steps,
               "call": "dg_aggregate_host (pinned host H, dOut in; out, dH back)"}
        del Hh, Gh, outh, dHh, ws

    # ---------------------------------------------------------------- CPU baseline (rank 0, N=1)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and two_buffers and not bf16:
        # the host cannot hold this workload's matrices: row sample as compact sub-problems
        cpu = cpu_baseline_sampled(torch, sg, g.dg_graph_get_csc()[:3], H, G, op, args.cpu_seconds)
    elif rank == 0 and world == 1 and not args.no_cpu_baseline and not bf16:
        import oracle
        colptr, rowidx_T, w_T, _ = g.dg_graph_get_csc()
        host = (sg.rowptr.cpu().numpy(), sg.colidx.cpu().numpy(),
                None if sg.edge_w is None else sg.edge_w.cpu().numpy(),
                colptr.cpu().numpy(), rowidx_T.cpu().numpy(),
                None if w_T is None else w_T.cpu().numpy())
        Hn, Gn = H.cpu().numpy(), G.cpu().numpy()
        o_op = oracle.OP_MEAN if op == "mean" else oracle.OP_SUM
        # size the sample for about cpu_seconds of work: calibrate on 64 rows, then on a tenth
        wk, sc = oracle_sample(host, Hn, Gn, o_op, 64)
        n_rows = int(max(64, min(sg.n, 0.1 * args.cpu_seconds / max(sc / 64, 1e-9))))
        wk, sc = oracle_sample(host, Hn, Gn, o_op, n_rows, seed=2)
        n_rows = int(max(64, min(sg.n, args.cpu_seconds / max(sc / n_rows, 1e-9))))
        wk, sc = oracle_sample(host, Hn, Gn, o_op, n_rows, seed=1)
        cpu = {"value": wk / sc, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"{n_rows} of {sg.n} destination rows (fwd) and source columns (bwd), "
                         f"{sc:.1f} s, fp64 accumulation"}

    # ---------------------------------------------------------------- every workload shape (N = 1)
    workloads = workloads_ingest = workloads_epoch = workloads_extras = None
    default_run = (args.workload == "reddit_like" and args.scale == 1.0 and not args.feat
                   and not bf16 and not args.set and not args.sorted_ids and op == "mean"
                   and args.reorder == "none")
    want_extras = args.other_calls or (default_run and args.workloads == "all")
    if rank == 0 and world == 1 and want_extras and not two_buffers:
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        workloads_extras = extra_records(torch, binding, synth, args.workload, g, sg, F, n_ref, peak,
                                         flush_buf)
        del flush_buf
    if rank == 0 and world == 1 and args.workloads == "all" and default_run:
        head = {"workload": args.workload, "scale": 1.0, "n": sg.n, "nnz": sg.nnz, "F": F, "op": op,
                "weighted": weighted, "reorder": "none", "dtype": "f32", "reps": args.steps,
                "l2": "inputs larger than L2 (no flush needed)",
                "buffers": "H, out, dOut, dH separate",
                "fwd": direction_record(fwd_list, b_fwd, sg.nnz * F * 4, sg.nnz * F, peak, ceilings),
                "bwd": direction_record(bwd_list, b_bwd, sg.nnz * F * 4, sg.nnz * F, peak, ceilings),
                "traffic": {"fwd": ncu_traffic(args.workload, F, op, 1.0, "fwd"),
                            "bwd": ncu_traffic(args.workload, F, op, 1.0, "bwd")},
                "clocks": clocks, "cpu_baseline": cpu, "note": "the headline step of this line"}
        ingest_head = {"graph_create_ms": create_ms, "transpose_ms": transpose_ms,
                       "transpose_edges_per_s": sg.nnz / (transpose_ms * 1e-3)}
        del H, out, G, dH, g, csc, sg
        torch.cuda.empty_cache()
        head_extras = workloads_extras or []
        workloads, workloads_ingest, workloads_epoch, workloads_extras = run_workloads(
            torch, binding, synth, dev, local_rank, peak, ceilings,
            0.0 if args.no_cpu_baseline else min(3.0, args.cpu_seconds),
            skip={(args.workload, F, op)})
        workloads.insert(2, head)
        workloads_extras = head_extras + workloads_extras
        workloads_ingest[args.workload + " (headline run)"] = ingest_head
        sg = type("Shape", (), {"n": head["n"], "nnz": head["nnz"]})()

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if not bf16 else "f32 sums over bf16-stored inputs", "data": "synthetic",
            "config": workload_config(args, sg, F, op, weighted, world, two_buffers),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks, "epoch": epoch_info,
            "ingest": {"graph_create_ms": create_ms, "transpose_ms": transpose_ms,
                       "transpose_edges_per_s": sg.nnz / (transpose_ms * 1e-3) if transpose_ms else None,
                       "reorder_ms": reorder_ms},
            "workloads": workloads, "workloads_ingest": workloads_ingest,
            "workloads_epoch": workloads_epoch, "other_calls": workloads_extras,
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
