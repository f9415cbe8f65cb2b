#!/usr/bin/env python
"""Benchmark of the transposable N:M mask search.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the approximate 2:4 search (Algorithm 1 + completion, packed mask, masked
weights and objective in one fused pass) over the 12288 x 49152 bf16 matrix whose entries are N(0, 0.02)
quantised to 256 levels (ties in nearly every block).  Prints ONE JSON line.

`--impl reference` times the CPU oracle as it stands on a bounded sample of the same matrix.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads  # noqa: E402

FULL_ROWS, COLS = 12288, 49152
ROWS = FULL_ROWS
N_KEEP, M_BLOCK = 2, 4
BYTES_PER_WEIGHT = 2 + 2 + 1.0 / 8          # read W, write masked W, write one mask bit (bf16)
# dram__bytes_read.sum + dram__bytes_write.sum of one full-size launch of the search kernel in steady state (mean of three
# consecutive launches after the first, caches not flushed between them); None when the kernel has changed since the counters were taken
TRAFFIC_BYTES_PER_LAUNCH = 1207.99e6 + 1282.66e6
TRAFFIC_SOURCE = ("ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --cache-control none on the full-size launch "
                  "(profiles/tma24_kernel_approx_2_4_bf16_12288x49152_launches.md)")
METRIC = "transposable-mask weights/s (2:4 approx, bf16, 1 GPU: achieved HBM GB/s vs peak in `roofline`)"
WORKLOAD = "%dx49152 bf16, N(0,0.02) quantised to 256 levels (frequent ties), 2:4 approximate, per-step recompute"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,timestamp")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, since=None):
        """Summary of the samples; `since` (a time.perf_counter() value) keeps only those taken after that moment."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        cut = None
        if since is not None:
            import datetime
            cut = datetime.datetime.now() - datetime.timedelta(seconds=time.perf_counter() - since)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                if cut is not None and len(f) >= 10:
                    try:
                        import datetime
                        if datetime.datetime.strptime(f[9], "%Y/%m/%d %H:%M:%S.%f") < cut:
                            continue
                    except ValueError:
                        pass
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                try:
                    pw.append(float(f[3]))
                except ValueError:
                    pass
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w=statistics.median(pw) if pw else None)
        return out


def time_oracle(W: np.ndarray, rows: int, threads: int):
    from oracle import tm_oracle as orc
    sample = np.ascontiguousarray(W[:rows])
    t0 = time.perf_counter()
    orc.find_mask(sample, N_KEEP, M_BLOCK, orc.APPROX, threads=threads)
    dt = time.perf_counter() - t0
    return sample.size / dt, dt


def run_reference(args):
    """The CPU oracle on a bounded row-strip sample per step (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import tm_oracle as orc
    orc.build()
    rows = 192
    W = workloads.quantised_bf16(rows, COLS, 0.02, 5)
    for _ in range(args.warmup):
        orc.find_mask(W, N_KEEP, M_BLOCK, orc.APPROX, threads=1)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.find_mask(W, N_KEEP, M_BLOCK, orc.APPROX, threads=1)
    dt = (time.perf_counter() - t0) / args.steps
    value = W.size / dt
    sample = "first %d rows of the %dx%d matrix per step (%d weights), single thread" % (rows, FULL_ROWS, COLS, W.size)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": {"workload": WORKLOAD % FULL_ROWS, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "weights/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "weights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_gpu(args):
    import torch
    import torch.distributed as dist

    import paper_2102_08124_b200 as tm
    from paper_2102_08124_b200 import build as tm_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        tm_build.build()
    if world > 1:
        dist.barrier()
    tm.load_library()

    # every rank searches its own matrix (blocks are independent: no exchange on the data path)
    ROWS = args.rows
    Wh = workloads.quantised_bf16(ROWS, COLS, 0.02, 5 + rank)
    W = torch.from_numpy(Wh.view(np.int16)).cuda().view(torch.bfloat16)
    mask = torch.empty((ROWS, tm.tm_mask_words_per_row(COLS)), dtype=torch.int32, device="cuda")
    masked = torch.empty_like(W)
    obj = torch.zeros((1,), dtype=torch.float64, device="cuda")

    def step():
        tm.tm_find_mask_bf16(W, N_KEEP, M_BLOCK, tm.TM_APPROX, mask_out=mask, masked_w_out=masked, objective_out=obj)

    def sync():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # a first look before the part heats up: W warm-up steps, K timed steps (reported beside the main number)
    for _ in range(max(args.warmup, 3)):
        step()
    sync()
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record()
    for _ in range(args.steps):
        step()
    b1.record()
    sync()
    ms_cold = b0.elapsed_time(b1) / args.steps

    # Sustained measurement.  The clock sampler starts first; an extended warm-up (at least W steps, at least 0.6 s) lets
    # the part settle at the clock it holds under load; then R blocks of exactly K steps are timed back to back with CUDA
    # events on the launching stream (R chosen so that the timed region lasts about half a second and the sampler sees
    # it), bracketed by a barrier and a synchronize.  The reported step time is the median block.
    sampler = ClockSampler(local_rank)
    if rank == 0 and not args.skip_clocks:
        sampler.start()
    warm, t_warm = 0, time.perf_counter()
    while warm < max(args.warmup, 3) or (not args.skip_clocks and time.perf_counter() - t_warm < 0.6):
        step()
        warm += 1
        if warm % 8 == 0:
            torch.cuda.synchronize()
    sync()
    repeats = args.repeats or max(10, min(200, int(0.5 / max(ms_cold * 1e-3 * args.steps, 1e-6))))
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    sync()
    t_region = time.perf_counter()
    marks[0].record()
    for r in range(repeats):
        for _ in range(args.steps):
            step()
        marks[r + 1].record()
    sync()
    region_s = time.perf_counter() - t_region
    blocks_ms = sorted(marks[r].elapsed_time(marks[r + 1]) / args.steps for r in range(repeats))
    ms = statistics.median(blocks_ms)
    clocks = sampler.stop(since=t_region) if (rank == 0 and not args.skip_clocks) else None
    status = tm.tm_device_status()
    t = torch.tensor([ms, blocks_ms[0], blocks_ms[-1]], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_max, ms_best, ms_worst = (float(v) for v in t.tolist())

    # end to end through the host-buffer entry point: pinned host input, results read back every step
    e2e = None
    if not args.skip_e2e:
        Wp = torch.from_numpy(Wh.view(np.int16)).view(torch.bfloat16).pin_memory()
        mask_h = torch.empty((ROWS, tm.tm_mask_words_per_row(COLS)), dtype=torch.int32).pin_memory()
        masked_h = torch.empty_like(Wp).pin_memory()
        e2e_steps = max(2, min(args.steps, 5))
        for _ in range(2):
            tm.tm_find_mask_host(Wp, N_KEEP, M_BLOCK, tm.TM_APPROX, mask_out=mask_h, masked_w_out=masked_h)
        sync()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            _, _, obj_e2e, st_e2e = tm.tm_find_mask_host(Wp, N_KEEP, M_BLOCK, tm.TM_APPROX, mask_out=mask_h, masked_w_out=masked_h)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        te = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
        if world > 1:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        e2e_s = float(te.item())
        e2e = {"value": world * ROWS * COLS / e2e_s, "unit": "weights/s", "h2d_bytes_per_step": int(Wp.numel() * 2),
               "d2h_bytes_per_step": int(masked_h.numel() * 2 + mask_h.numel() * 4 + 8), "ms_per_step": e2e_s * 1e3,
               "objective": obj_e2e, "status": st_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    weights = ROWS * COLS
    peak, peak_src = measured_peak()
    achieved = weights * BYTES_PER_WEIGHT / (ms * 1e-3) / 1e9
    cpu = None
    if not args.skip_cpu and world == 1:
        # the oracle as it stands on this machine's host cores: one thread (the plain definition) and all of them (its OpenMP
        # loop over block rows), each on a bounded strip of the same matrix
        cores = os.cpu_count() or 1
        one_rows = min(768, ROWS)
        one_value, one_dt = time_oracle(Wh, one_rows, 1)
        from oracle import tm_oracle as orc
        threads = orc.max_threads()
        all_rows = min(ROWS, max(one_rows, 512 * threads))
        all_value, all_dt = time_oracle(Wh, all_rows, threads)
        cpu = {"value": all_value, "unit": "weights/s", "cores": threads, "kind": "oracle",
               "sample": "first %d rows of the matrix (%d weights), %d OpenMP threads over block rows, %.1f s" % (all_rows, all_rows * COLS, threads, all_dt),
               "single_thread": {"value": one_value, "unit": "weights/s", "cores": 1,
                                 "sample": "first %d rows of the matrix (%d weights), %.1f s" % (one_rows, one_rows * COLS, one_dt)},
               "host_cores": cores}
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    line = {
        "metric": METRIC, "value": world * weights / (ms_max * 1e-3), "unit": "weights/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD % ROWS, "N": N_KEEP, "M": M_BLOCK, "method": "approx", "outputs": "mask+masked_w+objective",
                   "l2": "inputs (1.2 GB) larger than L2 (126 MB)", "device_status": status,
                   "objective": float(obj.item())},
        "timing": {"blocks_of_K_steps": repeats, "timed_steps": repeats * args.steps, "region_s": region_s, "ms_per_step_median": ms,
                   "ms_per_step_best_block": ms_best, "ms_per_step_worst_block": ms_worst, "warmup_steps_run": warm,
                   "ms_x_sm_mhz": ms * sm_mhz if sm_mhz else None,
                   "note": "value = median over the blocks; every block is exactly K steps, timed with CUDA events on the launching stream"},
        "e2e": e2e,
        "gpu_launches": args.steps * repeats,               # a step is one launch: the search kernel reduces its own objective
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC_BYTES_PER_LAUNCH if ROWS == FULL_ROWS else None, "traffic_source": TRAFFIC_SOURCE,
                     "peak_source": peak_src, "algorithmic_bytes_per_launch": weights * BYTES_PER_WEIGHT,
                     "frac_of_8000": achieved / 8000.0,
                     "cold": {"ms_per_step": ms_cold, "achieved": weights * BYTES_PER_WEIGHT / (ms_cold * 1e-3) / 1e9,
                              "frac": weights * BYTES_PER_WEIGHT / (ms_cold * 1e-3) / 1e9 / peak,
                              "note": "K steps timed right after W warm-up steps, before the sustained warm-up under the clock sampler"},
                     "note": "duration = CUDA-event time of one step = one launch of the search kernel (its last CTA adds up the objective)"},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_dry(args):
    """The multi-rank skeleton of run_gpu() without a GPU: gloo ranks, a host stand-in for the step, the same barrier,
    max-over-ranks reduction and one JSON line from rank 0.  Used by the CPU test of the launcher."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    x = np.ones(1 << 16, np.float32)

    def sync():
        if world > 1:
            dist.barrier()

    for _ in range(max(args.warmup, 3)):
        x += 1.0
    sync()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        x += 1.0
    ms = (time.perf_counter() - t0) * 1e3 / args.steps
    sync()
    t = torch.tensor([ms], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"metric": "dry run of the launcher (no GPU work)", "value": world * x.size / (float(t.item()) * 1e-3), "unit": "elements/s",
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(t.item()), "scaling": "weak",
                          "gpu_launches": 0}))
    if world > 1:
        dist.destroy_process_group()


def launch_ranks(args, argv):
    """`--gpus N` with N > 1 outside a torchrun environment: start N ranks of this script on this node (one per GPU,
    rendezvous on 127.0.0.1) and hand their output through; rank 0 prints the line."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def _block_sums(x, M):
    r, c = x.shape
    return x.reshape(r // M, M, c // M, M).sum(axis=(1, 3))


def quality_numbers(W, cover_bits, approx_bits, exact_bits, M):
    """Per-block quality of the approximation against the optimum (Section 4.1 quotes "within a factor of 1.2" for
    Algorithm 1; the Lemma bounds the factor by 2): pruned-mass ratio W(P) / W* of the cover and of the completed mask,
    kept-mass gap 1 - kept(approx) / kept(exact); mean and maximum over the blocks with W* > 0."""
    mag = np.abs(W.astype(np.float64))
    total = _block_sums(mag, M)
    kept_e, kept_a, kept_c = (_block_sums(mag * b, M) for b in (exact_bits, approx_bits, cover_bits))
    w_star, w_cover, w_approx = total - kept_e, total - kept_c, total - kept_a
    ok = w_star > 0
    return {"blocks": int(ok.sum()),
            "cover_ratio_mean": float((w_cover[ok] / w_star[ok]).mean()), "cover_ratio_max": float((w_cover[ok] / w_star[ok]).max()),
            "approx_ratio_mean": float((w_approx[ok] / w_star[ok]).mean()), "approx_ratio_max": float((w_approx[ok] / w_star[ok]).max()),
            "kept_gap_mean": float((1 - kept_a[ok] / kept_e[ok]).mean()), "kept_gap_max": float((1 - kept_a[ok] / kept_e[ok]).max()),
            "kept_gap_whole_matrix": float(1 - kept_a.sum() / kept_e.sum())}


def run_survey(args):
    """Secondary measurements (one JSON line per case): every named workload x method through a prepared plan.
    Small workloads are L2-resident across repeats, so their GB/s is not an HBM figure; it is labelled so."""
    import torch

    import paper_2102_08124_b200 as tm
    from paper_2102_08124_b200 import build as tm_build
    tm_build.build()
    torch.cuda.set_device(0)
    peak, _ = measured_peak()
    cases = [("config1 256x256 fp32", workloads.config1, 2, 4, ["approx", "cover", "exact"]),
             ("config2 ResNet-50-shaped, 54 matrices fp32", workloads.config2, 2, 4, ["approx", "exact"]),
             ("config3 BERT-large-shaped, 96 matrices bf16", workloads.config3, 2, 4, ["approx"]),
             ("config4 8192x8192 fp32 Laplace", workloads.config4, 4, 8, ["approx", "cover", "exact"]),
             ("config5 12288x49152 bf16 quantised", workloads.config5, 2, 4, ["approx", "cover", "exact"]),
             # two more large cases, so that every (dtype, N:M) pair of the bandwidth kernels has an HBM-sized measurement
             ("config6 (extra) 8192x8192 fp32 Laplace, 2:4", workloads.config4, 2, 4, ["approx", "cover"]),
             ("config7 (extra) 12288x49152 bf16 quantised, 4:8", workloads.config5, 4, 8, ["approx", "cover"])]
    methods = {"approx": tm.TM_APPROX, "cover": tm.TM_APPROX_COVER, "exact": tm.TM_EXACT}
    for name, gen, N, M, ms in cases:
        if args.config and not name.startswith("config%d" % args.config):
            continue
        mats = gen()
        Ws = [torch.from_numpy(m.view(np.int16)).cuda().view(torch.bfloat16) if m.dtype == np.uint16 else torch.from_numpy(m).cuda() for m in mats]
        weights = sum(int(m.size) for m in mats)
        bpw = sum(m.size * (2 * m.itemsize + 0.125) for m in mats) / weights
        batch = tm.TmBatch(Ws)                    # descriptors marshalled once, as a training loop would
        objs, status = batch.objectives, batch.status
        for mname in ms:
            meth = methods[mname]
            # prepared once (descriptors validated, tensor maps built, tables uploaded), then only launched: the refresh loop's way
            plan = tm.tm_plan_create(Ws, N, M, meth, masks=batch.masks, maskeds=batch.maskeds, objectives=batch.objectives,
                                     workspace=batch.workspace, status=batch.status)
            def step():
                tm.tm_plan_run(plan)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            t0 = time.perf_counter(); step(); torch.cuda.synchronize(); once = time.perf_counter() - t0
            steps = args.survey_steps or max(3, min(200, int(0.5 / max(once, 1e-5))))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                step()
            e1.record(); torch.cuda.synchronize()
            msec = e0.elapsed_time(e1) / steps
            gbs = weights * bpw / (msec * 1e-3) / 1e9
            print(json.dumps({"workload": name, "N": N, "M": M, "method": mname, "matrices": len(mats), "weights": weights,
                              "ms_per_call": msec, "weights_per_s": weights / (msec * 1e-3), "algorithmic_GBps": gbs,
                              "frac_of_measured_hbm": gbs / peak, "steps": steps,
                              "resident_in_l2": bool(weights * bpw < 100e6), "status": int(status.item()),
                              "objective_sum": float(objs.sum().item())}), flush=True)
            tm.tm_plan_destroy(plan)
        if name.startswith("config1") or name.startswith("config4"):
            # quality of the approximation against the optimum, per block (masks from the GPU, sums on the host in fp64)
            bits = {}
            for mname in ("cover", "approx", "exact"):
                batch.run(N, M, methods[mname]); torch.cuda.synchronize()
                words = batch.masks[0].cpu().numpy().view(np.uint32)
                bits[mname] = np.unpackbits(words.view(np.uint8), axis=1, bitorder="little")[:, :mats[0].shape[1]]
            print(json.dumps({"workload": name, "N": N, "M": M, "quality": quality_numbers(mats[0], bits["cover"], bits["approx"], bits["exact"], M)}), flush=True)
        del Ws, batch, objs, status
        torch.cuda.empty_cache()


def run_survey_neighbours(args):
    """Secondary measurements of the neighbouring operations (1-D N:M pruning, compression, refresh loop)."""
    import torch

    import paper_2102_08124_b200 as tm
    from paper_2102_08124_b200.refresh import MaskRefresher
    peak, _ = measured_peak()

    def timed(fn, min_steps=5):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter(); fn(); torch.cuda.synchronize(); once = time.perf_counter() - t0
        steps = args.survey_steps or max(min_steps, min(200, int(0.3 / max(once, 1e-5))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record(); torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def emit(name, op, msec, nbytes, weights):
        gbs = nbytes / (msec * 1e-3) / 1e9
        print(json.dumps({"workload": name, "op": op, "ms_per_call": msec, "weights_per_s": weights / (msec * 1e-3),
                          "algorithmic_GBps": gbs, "frac_of_measured_hbm": gbs / peak}), flush=True)

    for name, gen, N, M in (("config5 12288x49152 bf16 quantised", workloads.config5, 2, 4), ("config4 8192x8192 fp32 Laplace", workloads.config4, 4, 8)):
        m = gen()[0]
        W = torch.from_numpy(m.view(np.int16)).cuda().view(torch.bfloat16) if m.dtype == np.uint16 else torch.from_numpy(m).cuda()
        es, n = m.itemsize, m.size
        mask = torch.empty((W.shape[0], tm.tm_mask_words_per_row(W.shape[1])), dtype=torch.int32, device="cuda")
        masked = torch.empty_like(W); obj = torch.zeros(1, dtype=torch.float64, device="cuda"); viol = torch.zeros(1, dtype=torch.int64, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda"); ws = torch.empty(tm.tm_aux_workspace_bytes(), dtype=torch.uint8, device="cuda")
        for absorb in (False, True):
            ms_ = timed(lambda: tm.tm_nm_mask_1d(W, N, M, absorb_mean=absorb, mask_out=mask, masked_w_out=masked, objective_out=obj,
                                                  violations_out=viol, status=st, workspace=ws))
            emit(name, "1-D %d:%d pruning%s" % (N, M, " + mean absorption" if absorb else ""), ms_, n * (2 * es + 0.125), n)
        ms_ = timed(lambda: tm.tm_mask_violations(W, mask, violations_out=viol, workspace=ws))
        emit(name, "mask violations", ms_, n * (es + 0.125), n)
        if M == 4:
            fn = tm.tm_find_mask_bf16 if m.dtype == np.uint16 else tm.tm_find_mask
            fn(W, 2, 4, tm.TM_APPROX, mask_out=mask, masked_w_out=masked, objective_out=obj)
            vals = torch.empty((W.shape[0], W.shape[1] // 2), dtype=W.dtype, device="cuda"); vals_t = torch.empty((W.shape[1], W.shape[0] // 2), dtype=W.dtype, device="cuda")
            meta = torch.empty_like(mask); meta_t = torch.empty((W.shape[1], tm.tm_mask_words_per_row(W.shape[0])), dtype=torch.int32, device="cuda")
            ms_ = timed(lambda: tm.tm_compress_2_4(W, mask, vals, meta, vals_t, meta_t, st))
            emit(name, "2:4 compression of W and W^T", ms_, n * (es + 0.125 + es + 0.25), n)
        mask2 = mask.clone()
        ms_ = timed(lambda: tm.tm_mask_hamming(mask, mask2, distance_out=viol, workspace=ws))
        emit(name, "mask Hamming distance", ms_, n * 0.25, n)
        del W, mask, masked, mask2
        torch.cuda.empty_cache()
    mats = workloads.config3()
    Ws = [torch.from_numpy(m.view(np.int16)).cuda().view(torch.bfloat16) for m in mats]
    n = sum(m.size for m in mats)
    for N, M in ((2, 4), (4, 8)):
        for graph in (False, True):
            r = MaskRefresher(Ws, N=N, M=M, use_graph=graph)
            ms_ = timed(lambda: r.refresh())
            emit("config3 BERT-large-shaped, 96 matrices bf16", "refresh %d:%d (%s): masks + masked weights + changed bits, result read back"
                 % (N, M, "CUDA graph" if graph else "eager"), ms_, n * (4.125 + 0.5), n)
            del r


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="tm", choices=["tm", "reference"])
    # profiling aids (ncu captures want a smaller case and none of the side measurements)
    ap.add_argument("--rows", type=int, default=ROWS, help="rows of the matrix (default: the full workload)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer end-to-end measurement")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--skip-clocks", action="store_true", help="no nvidia-smi sampling and no extended warm-up")
    ap.add_argument("--survey", action="store_true", help="secondary table: all named workloads and methods, one JSON line each")
    ap.add_argument("--config", type=int, default=0, help="with --survey: only this workload (1..5)")
    ap.add_argument("--survey-steps", type=int, default=0, help="with --survey: timed calls per case (default: about 0.5 s worth, at most 200)")
    ap.add_argument("--repeats", type=int, default=0, help="timed blocks of K steps (default: about half a second worth, 10 to 200)")
    ap.add_argument("--dry-run", action="store_true", help="launcher and multi-rank skeleton only: gloo on CPU, no GPU work")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.survey and args.impl != "reference":
        raise SystemExit(launch_ranks(args, sys.argv[1:]))
    if args.dry_run:
        run_dry(args)
    elif args.survey:
        if not args.config:
            run_survey(args)
            run_survey_neighbours(args)
        elif args.config == 8:
            run_survey_neighbours(args)
        else:
            run_survey(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
