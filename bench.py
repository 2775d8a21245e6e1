#!/usr/bin/env python
"""Benchmark of the SKIM row-clustering path on B200.

One step = one pass of the whole path over one synthetic LLaMA-7B down-projection matrix
(4096 x 11008 fp16 weights + fp32 importance): cluster every row at widths {1,2,3,4} for 50
Lloyd iterations, allocate bits greedily at an average of 3.0, emit packed codes and LUTs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded row sample.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2412_04180_b200 import inputs  # noqa: E402

METRIC = "weight rows clustered/sec (all 4 bit-widths, fixed iters), full pipeline"
ROWS, COLS, SEED = 4096, 11008, 3001   # --rows shrinks the row count for profiler captures only
BIT_SET = [1, 2, 3, 4]
ITERS = 50
BUDGET = 3.0
WORKLOAD = "llama7b_down_proj 4096x11008 fp16, importance LogNormal(0,1.5) fp32, bits {1,2,3,4}, 50 iters, budget 3.0"
# Algorithmic bytes of the clustering stage: fp16 weight + fp32 importance in, 4 errors + 30 centroids
# (fp32) out per row.  The stage is two kernels: the row-sorting kernel (the dominant one) reads
# the 6 bytes per element; the Lloyd kernel writes the 136 bytes per row.  The row records that
# pass between them are scratch, not algorithmic bytes.
CLUSTER_BYTES_PER_ELEMENT = 6
CLUSTER_BYTES_PER_ROW = 136
# DRAM traffic of one launch of the dominant kernel per row, from the committed ncu capture
# (bytes), or None when the kernel changed since the counters were taken.
SORT_TRAFFIC_BYTES_PER_ROW = 136_638   # (135.38 MB read + 144.46 MB written) / 2048 rows, profiles/skim_sort16_kernel_2048x11008.md
DOMINANT_KERNEL = "skim_sort16_kernel"
DTYPE = "f64 sums, f32 centroid state (fp16 weights and fp32 importance in)"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ctypes_size(ctx, rows, cols):
    """Scratch bytes of the L-full alpha-update (skim_scale_lfull_bytes)."""
    import ctypes as C
    from paper_2412_04180_b200 import skim
    need = C.c_size_t()
    rc = skim.lib().skim_scale_lfull_bytes(C.c_int64(rows), C.c_int64(cols), C.byref(need))
    assert rc == 0
    return need.value


def measured_tensor_peak():
    """Measured dense bf16 tensor throughput (TFLOP/s) for a kernel timed alone; fp16 runs at the same rate."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (cuBLAS bf16 burst; fp16 has the same nominal rate)"
    except Exception:
        return 1590.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(1.0)   # nvidia-smi needs about a second before its first sample
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _oracle_pass(orc, nrows):
    """One pass of the whole path by the oracle over the first `nrows` rows; returns seconds."""
    w, g = inputs.make_rows(ROWS, COLS, SEED, 0, nrows)
    t0 = time.perf_counter()
    res = orc.cluster_rows(w, g, BIT_SET, ITERS, want_codes=False)
    bits, _ = orc.allocate_bits(res["err"].astype(np.float32), BIT_SET[0], BUDGET)
    orc.emit(w, bits, res["centroids"].astype(np.float32), BIT_SET)
    return time.perf_counter() - t0


def _oracle_sample_rows(orc, target_seconds):
    cores = orc.num_threads()
    probe = _oracle_pass(orc, cores)
    nrows = int(min(ROWS, max(cores, round(cores * target_seconds / max(probe, 1e-3)))))
    return max(cores, nrows // cores * cores)


def cpu_baseline(target_seconds=15.0):
    """The oracle, as it stands, on a bounded row sample of the same workload (all host cores)."""
    from oracle import skim_oracle as orc
    orc.build()
    nrows = _oracle_sample_rows(orc, target_seconds)
    t = _oracle_pass(orc, nrows)
    return {"value": nrows / t, "unit": "rows/s", "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"first {nrows} of {ROWS} rows of the same matrix, full pipeline, {t:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import skim_oracle as orc
    orc.build()
    per_step = max(0.5, min(6.0, 100.0 / max(1, args.steps + args.warmup)))
    nrows = _oracle_sample_rows(orc, per_step)
    times = []
    for i in range(args.warmup + args.steps):
        t = _oracle_pass(orc, nrows)
        if i >= args.warmup:
            times.append(t)
    ms = 1e3 * sum(times) / len(times)
    value = nrows / (ms / 1e3)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "rows/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": WORKLOAD, "rows": ROWS, "cols": COLS, "sample_rows_per_step": nrows},
        "cpu_baseline": {"value": value, "unit": "rows/s", "cores": orc.num_threads(), "kind": "oracle",
                         "sample": f"first {nrows} of {ROWS} rows of the same matrix per step, full pipeline"},
        "e2e": {"value": value, "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_stage(args, ctx, stream, W, G, cent, bits, out):
    """Times one stage outside the benchmark's step: the alpha-update (Algorithm 2, inner repeat) or the
    consumers of the packed form, on the benchmark's matrix after one pipeline step."""
    import torch
    peak, peak_kind = measured_peak()
    with torch.cuda.stream(stream):
        if args.stage == "scale":
            _, labels, _ = ctx.cluster_rows_at(W, G, bits, BIT_SET, ITERS, want_codes=True, centroids=cent.clone())
            alpha = torch.ones(COLS, dtype=torch.float32, device="cuda")
            ctx.scale_update(W, G, labels, alpha, steps=3, want_trace=False)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            trace = ctx.scale_update(W, G, labels, alpha, steps=args.steps)
            e1.record(stream)
            stream.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            nbytes = 2 * 7 * ROWS * COLS
            print(json.dumps({"stage": "scale_update", "workload": WORKLOAD, "adam_steps": args.steps, "ms_per_adam_step": ms,
                              "algorithmic_bytes_per_step": nbytes, "achieved_gbs": nbytes / (ms * 1e-3) / 1e9,
                              "hbm_frac": nbytes / (ms * 1e-3) / 1e9 / peak, "peak_kind": f"of {peak_kind}",
                              "loss_first": float(trace[0]), "loss_last": float(trace[-1]), "kernel_launches_per_step": 3}))
        elif args.stage == "lfull":
            tpeak, tpeak_kind = measured_tensor_peak()
            Hc = torch.from_numpy(inputs.make_gram(COLS, SEED + 7)).cuda()
            Dbuf = torch.empty((ROWS, COLS), dtype=torch.float16, device="cuda")
            scr = torch.empty(ctx.err_lfull_bytes(ROWS, COLS), dtype=torch.uint8, device="cuda")
            col = torch.empty((ROWS,), dtype=torch.float32, device="cuda")
            ctx.residual(W, cent, BIT_SET, width=BIT_SET[-1], out=Dbuf)
            for _ in range(2):
                ctx.err_lfull(Dbuf, Hc, scratch=scr, out=col)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                ctx.err_lfull(Dbuf, Hc, scratch=scr, out=col)
            e1.record(stream)
            stream.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            flops = 2.0 * ROWS * COLS * COLS
            print(json.dumps({"stage": "err_lfull", "workload": WORKLOAD, "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                              "tensor_frac": flops / (ms * 1e-3) / 1e12 / tpeak, "peak_kind": f"of {tpeak_kind}"}))
        elif args.stage == "exact":
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ctx.cluster_rows_exact(W[:64], G[:64], BIT_SET)
            e0.record(stream)
            ctx.cluster_rows_exact(W, G, BIT_SET)
            e1.record(stream)
            stream.synchronize()
            print(json.dumps({"stage": "cluster_rows_exact", "workload": WORKLOAD, "ms": e0.elapsed_time(e1)}))
        else:
            xq = torch.from_numpy(np.random.default_rng(1).standard_normal(COLS).astype(np.float16)).cuda()
            wq = torch.empty((ROWS, COLS), dtype=torch.float16, device="cuda")
            yq = torch.empty((ROWS,), dtype=torch.float32, device="cuda")
            res = {}
            for name, fn in (("dequantize", lambda: ctx.dequantize(out, COLS, BIT_SET, out=wq)),
                             ("matvec", lambda: ctx.matvec(out, COLS, BIT_SET, xq, out=yq))):
                fn()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(args.steps):
                    fn()
                e1.record(stream)
                stream.synchronize()
                res[name + "_ms_incl_launch_gaps"] = e0.elapsed_time(e1) / args.steps
            print(json.dumps({"stage": "consumers", "workload": WORKLOAD, **res}))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2412_04180_b200 import build, shard
    from paper_2412_04180_b200.skim import Skim

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if local == 0:
        build.build()
    if world > 1:
        dist.barrier()

    # every rank clusters a matrix of its own (independent problems: no data-path collective)
    mine = shard.assign_matrices([(ROWS, COLS)] * world, world)[rank]
    assert len(mine) == 1
    w, g = inputs.make_matrix(ROWS, COLS, shard.matrix_seed(SEED, mine[0]))
    stream = torch.cuda.Stream()
    ctx = Skim(device=local, stream=stream)
    ctx.reserve(ROWS, COLS)
    nb, sumk = len(BIT_SET), sum(1 << b for b in BIT_SET)
    with torch.cuda.stream(stream):
        W = torch.from_numpy(w).cuda()
        G = torch.from_numpy(g).cuda()
        cent = torch.empty((ROWS, sumk), dtype=torch.float32, device="cuda")
        err = torch.empty((ROWS, nb), dtype=torch.float32, device="cuda")
        bits = torch.empty((ROWS,), dtype=torch.uint8, device="cuda")
        _, mx = Skim.packed_layout(ROWS, COLS, BIT_SET)
        out = dict(packed=torch.empty(mx // 4, dtype=torch.int32, device="cuda"),
                   row_order=torch.empty(ROWS, dtype=torch.int32, device="cuda"),
                   group_info=torch.empty(2 * (nb + 1), dtype=torch.int64, device="cuda"),
                   lut=torch.empty((ROWS, 1 << BIT_SET[-1]), dtype=torch.int16, device="cuda"))
    stream.synchronize()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        ctx.cluster_rows_into(W, G, BIT_SET, ITERS, cent, err)
        if ev:
            ev[1].record(stream)
        ctx.allocate_bits(err, BIT_SET, BUDGET, out=bits)
        if ev:
            ev[2].record(stream)
        ctx.quantize(W, bits, cent, BIT_SET, out=out)
        if ev:
            ev[3].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if args.stage != "pipeline":
        if rank == 0:
            run_stage(args, ctx, stream, W, G, cent, bits, out)
        if world > 1:
            dist.destroy_process_group()
        return

    def busy(seconds):
        # the same steps, untimed, so that the clock samples around the timed region see this load
        if args.rows:
            return          # profiler captures: keep the launch count small
        t_end = time.perf_counter() + seconds
        while time.perf_counter() < t_end:
            step()
            stream.synchronize()

    busy(0.05)
    sampler = ClockSampler(local) if rank == 0 else None
    busy(0.4)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches0 = ctx.launch_count()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record(stream)
    for k in range(args.steps):
        step()
    end.record(stream)
    barrier()
    total_ms = start.elapsed_time(end)
    launches = ctx.launch_count() - launches0
    # the same K steps once more with events between the stages and between the two clustering kernels
    # (on the same stream): these events keep a kernel from starting under its predecessor's tail and cost
    # about 3 % of a step, so the headline above is timed without them
    ctx.kernel_timing(True)
    for k in range(args.steps):
        step(evs[k])
    stream.synchronize()
    sort_total, lloyd_total, timed_chunks = ctx.kernel_times()
    ctx.kernel_timing(False)
    sort_ms, lloyd_ms = sort_total / max(1, timed_chunks), lloyd_total / max(1, timed_chunks)
    iter_sum, iter_rows = ctx.lloyd_iterations()
    busy(0.4)
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["window"] = "0.4 s of the same steps before and after the timed region, plus the region itself"
    job_rows_per_s, job_rows, total_ms = shard.job_throughput(ROWS * args.steps, total_ms, "cuda")
    ms_step = total_ms / args.steps
    cluster_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    alloc_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    quant_ms = statistics.mean(e[2].elapsed_time(e[3]) for e in evs)
    assert ctx.get_status() == 0
    total_bits = int(bits.sum().item())
    assert total_bits == int(ROWS * BUDGET), total_bits
    mx = Skim.packed_layout(ROWS, COLS, BIT_SET)[1]

    # the same step with the converged-row shortcut off: every row runs all ITERS iterations (same output)
    extra = {}
    if not args.rows:
        ctx.early_exit(False)
        for _ in range(3):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        stream.synchronize()
        ctx.early_exit(True)
        extra["ms_per_step_early_exit_off"] = e0.elapsed_time(e1) / args.steps

        # Algorithm 2 on the same matrix at the allocated widths (outside the timed region): the alpha-update
        # alone, and one whole alternation round = re-clustering at b_i + 120 Adam steps + emission
        peak_s, _ = measured_peak()
        with torch.cuda.stream(stream):
            alpha = torch.ones(COLS, dtype=torch.float32, device="cuda")
            ctx.apply_scale(alpha)
            cent_at = cent.clone()
            _, labels, _ = ctx.cluster_rows_at(W, G, bits, BIT_SET, ITERS, want_codes=True, centroids=cent_at)
            ctx.scale_update(W, G, labels, alpha, steps=3, want_trace=False)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ctx.scale_update(W, G, labels, alpha, steps=40, want_trace=False)
            e1.record(stream)
            stream.synchronize()
            adam_ms = e0.elapsed_time(e1) / 40
            adam_bytes = 2 * 7 * ROWS * COLS          # two passes over fp16 W, fp32 importance and u8 labels
            # two rounds, the second one reported: the first still meets one-time costs (allocator growth for the
            # label matrix, lazily loaded kernels), which once showed as 14.6 ms instead of 2.1 ms of re-clustering
            for _ in range(2):
                r0, r1, r2, r3 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
                r0.record(stream)
                ctx.apply_scale(alpha)
                _, labels, _ = ctx.cluster_rows_at(W, G, bits, BIT_SET, ITERS, want_codes=True, centroids=cent_at)
                r1.record(stream)
                ctx.scale_update(W, G, labels, alpha, steps=120, want_trace=False)
                r2.record(stream)
                ctx.apply_scale(alpha)
                ctx.quantize(W, bits, cent_at, BIT_SET, out=out)
                r3.record(stream)
                stream.synchronize()
            ctx.apply_scale(None)
            assert ctx.get_status() == 0
        extra["scale_update"] = {"ms_per_adam_step": adam_ms, "algorithmic_bytes_per_step": adam_bytes,
                                 "hbm_frac": adam_bytes / (adam_ms * 1e-3) / 1e9 / peak_s, "kernels_per_step": 3}
        extra["alternation_round"] = {"recluster_at_allocated_widths_ms": r0.elapsed_time(r1),
                                      "adam_120_steps_ms": r1.elapsed_time(r2), "emit_ms": r2.elapsed_time(r3),
                                      "total_ms": r0.elapsed_time(r3),
                                      "note": "one round of Algorithm 2 on the same matrix with the scale vector installed "
                                              "(32-bit keys), labels written; the second of two rounds, outside the timed region"}
        # the pipeline's own outputs again (the round above overwrote the packed form with the scaled one)
        step()
        stream.synchronize()

        # the error table in the paper's L-full form on the same matrix (outside the timed region): residual +
        # tcgen05 GEMM with the row-wise dot fused in, once per width, against a synthetic Gram matrix
        tpeak, tpeak_kind = measured_tensor_peak()
        with torch.cuda.stream(stream):
            Hc = torch.from_numpy(inputs.make_gram(COLS, SEED + 7)).cuda()
            Dbuf = torch.empty((ROWS, COLS), dtype=torch.float16, device="cuda")
            lf_scr = torch.empty(ctx.err_lfull_bytes(ROWS, COLS), dtype=torch.uint8, device="cuda")
            table = torch.empty((ROWS, nb), dtype=torch.float32, device="cuda")
            for _ in range(2):
                ctx.residual(W, cent, BIT_SET, width=BIT_SET[-1], out=Dbuf)
                ctx.err_lfull(Dbuf, Hc, scratch=lf_scr, out=table[:, nb - 1], out_stride=nb)
            l0, l1, l2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            res_ms = gemm_ms = 0.0
            for bi, b in enumerate(BIT_SET):
                l0.record(stream)
                ctx.residual(W, cent, BIT_SET, width=b, out=Dbuf)
                l1.record(stream)
                ctx.err_lfull(Dbuf, Hc, scratch=lf_scr, out=table[:, bi], out_stride=nb)
                l2.record(stream)
                stream.synchronize()
                res_ms += l0.elapsed_time(l1)
                gemm_ms += l1.elapsed_time(l2)
            assert ctx.get_status() == 0 and bool(torch.isfinite(table).all())
            # the alpha-update on the L-full loss (Section 4.3): residual, contraction with Y kept, two streaming passes, Adam
            ctx.apply_scale(None)
            _, labels0, _ = ctx.cluster_rows_at(W, G, bits, BIT_SET, ITERS, want_codes=True, centroids=cent.clone())
            alpha_lf = torch.ones(COLS, dtype=torch.float32, device="cuda")
            need_lf = ctypes_size(ctx, ROWS, COLS)
            scr_lf = torch.empty(need_lf, dtype=torch.uint8, device="cuda")
            ctx.scale_update_lfull(W, G, labels0, alpha_lf, Hc, steps=2, want_trace=False, scratch=scr_lf)
            l0.record(stream)
            tr = ctx.scale_update_lfull(W, G, labels0, alpha_lf, Hc, steps=10, scratch=scr_lf)
            l1.record(stream)
            stream.synchronize()
            lf_step_ms = l0.elapsed_time(l1) / 10
            lf_loss = (float(tr[0]), float(tr[-1]))
            assert ctx.get_status() == 0
            del scr_lf, labels0
        flops = 2.0 * ROWS * COLS * COLS
        extra["lfull_table"] = {"residual_ms_per_width": res_ms / nb, "gemm_ms_per_width": gemm_ms / nb,
                                "table_ms_all_widths": res_ms + gemm_ms,
                                "roofline": {"bound": "tensor", "kernel": "skim_lfull_gemm_kernel", "dtype": "fp16 in, fp32 accumulate",
                                             "achieved": flops / (gemm_ms / nb * 1e-3) / 1e12, "peak": tpeak, "peak_kind": f"of {tpeak_kind}",
                                             "unit": "TFLOP/s", "frac": flops / (gemm_ms / nb * 1e-3) / 1e12 / tpeak, "traffic": None},
                                "scale_update_lfull_ms_per_adam_step": lf_step_ms, "scale_update_lfull_loss_first_last": lf_loss,
                                "note": "Section 3.4's L-full error for every row and width: 2*rows*cols^2 flop per width; "
                                        "the alpha-update on the same loss does one such contraction per Adam step"}
        del Hc, Dbuf, lf_scr

        # the optimum of the clustering objective per row (yardstick for the 50 Lloyd iterations)
        with torch.cuda.stream(stream):
            need = torch.empty(0)
            x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ctx.cluster_rows_exact(W[:296], G[:296], BIT_SET)
            x0.record(stream)
            _, err_opt = ctx.cluster_rows_exact(W, G, BIT_SET)
            x1.record(stream)
            stream.synchronize()
            ratio = (err_opt.double() / err.double().clamp_min(1e-300)).cpu().numpy()
        extra["exact_clustering"] = {"ms": x0.elapsed_time(x1),
                                     "optimum_over_lloyd_error_mean_per_width": [float(v) for v in ratio.mean(axis=0)],
                                     "optimum_over_lloyd_error_median_per_width": [float(v) for v in np.median(ratio, axis=0)],
                                     "note": "skim_cluster_rows_exact on the same matrix: the iterations' error table entries "
                                             "divided into the optimum's (1.0 = the iterations found the optimum)"}

    # the consumers of the packed form (outside the timed region; reported beside the step)
    consumers = None
    if not args.rows:
        xq = torch.from_numpy(np.random.default_rng(1).standard_normal(COLS).astype(np.float16)).cuda()
        wq = torch.empty((ROWS, COLS), dtype=torch.float16, device="cuda")
        yq = torch.empty((ROWS,), dtype=torch.float32, device="cuda")
        words = int(out["group_info"][-1].item())
        times = {}
        filler = torch.empty(3 << 30, dtype=torch.uint8, device="cuda")
        with torch.cuda.stream(stream):
            for name, fn in (("dequantize", lambda: ctx.dequantize(out, COLS, BIT_SET, out=wq)),
                             ("matvec", lambda: ctx.matvec(out, COLS, BIT_SET, xq, out=yq))):
                for _ in range(3):
                    fn()
                # long fills first (they also flush L2), so that the launches below queue up behind
                # them and the events see device time only, not the host's launch overhead: the fills
                # must outlast the host's 20 calls (some 20 us each from Python)
                for _ in range(4):
                    filler.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(20):
                    fn()
                e1.record(stream)
                stream.synchronize()
                times[name] = e0.elapsed_time(e1) / 20
        peak_c, _ = measured_peak()
        deq_bytes = words * 4 + ROWS * 32 + COLS * 4 + ROWS * COLS * 2
        mv_bytes = words * 4 + ROWS * 32 + COLS * 2 + ROWS * 4
        consumers = {"dequantize_ms": times["dequantize"], "dequantize_bytes": deq_bytes,
                     "dequantize_hbm_frac": deq_bytes / (times["dequantize"] * 1e-3) / 1e9 / peak_c,
                     "matvec_ms": times["matvec"], "matvec_bytes": mv_bytes,
                     "matvec_hbm_frac": mv_bytes / (times["matvec"] * 1e-3) / 1e9 / peak_c,
                     "note": "skim_dequantize / skim_matvec on the step's packed output; 20 back-to-back launches each, queued behind four 3 GB fills"}
        del filler

    # end to end through the host-buffer entry point: pinned host inputs -> pinned host outputs
    e2e = None
    if not args.no_e2e:
        staging = torch.empty(Skim.host_staging_bytes(ROWS, COLS, BIT_SET), dtype=torch.uint8, device="cuda")
        Wh = torch.from_numpy(w).pin_memory()
        Gh = torch.from_numpy(g).pin_memory()
        hout = dict(err=torch.empty((ROWS, nb), dtype=torch.float32).pin_memory(),
                    bits=torch.empty((ROWS,), dtype=torch.uint8).pin_memory(),
                    packed=torch.empty(mx // 4, dtype=torch.int32).pin_memory(),
                    row_order=torch.empty(ROWS, dtype=torch.int32).pin_memory(),
                    group_info=torch.empty(2 * (nb + 1), dtype=torch.int64).pin_memory(),
                    lut=torch.empty((ROWS, 1 << BIT_SET[-1]), dtype=torch.int16).pin_memory())
        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            ctx.quantize_matrix_host(Wh, Gh, BIT_SET, ITERS, BUDGET, staging, hout)
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            ctx.quantize_matrix_host(Wh, Gh, BIT_SET, ITERS, BUDGET, staging, hout)
        torch.cuda.synchronize()
        e2e_ms = 1e3 * (time.perf_counter() - t0) / n_e2e
        e2e_ms = shard.max_over_ranks(e2e_ms, "cuda")
        words = int(hout["group_info"][-1].item())
        d2h = ROWS * nb * 4 + ROWS + ROWS * 4 + 2 * (nb + 1) * 8 + ROWS * (1 << BIT_SET[-1]) * 2 + words * 4
        e2e = {"value": world * ROWS / (e2e_ms / 1e3), "unit": "rows/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": ROWS * COLS * 6, "d2h_bytes_per_step": d2h, "steps": n_e2e}
        assert int(hout["bits"].sum().item()) == int(ROWS * BUDGET)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    cluster_bytes = ROWS * COLS * CLUSTER_BYTES_PER_ELEMENT + ROWS * CLUSTER_BYTES_PER_ROW
    sort_bytes = ROWS * COLS * CLUSTER_BYTES_PER_ELEMENT
    achieved = sort_bytes / (sort_ms * 1e-3) / 1e9
    pipeline_bytes = ROWS * COLS * (6 + 2 + BUDGET / 8) + ROWS * 170
    result = {
        "metric": METRIC, "value": job_rows_per_s, "unit": "rows/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": WORKLOAD, "rows": ROWS, "cols": COLS, "l2": "inputs 270 MB per step exceed the 126 MB L2",
                   "early_exit": "on (rows stop once no boundary moved; output bit-identical to running all iterations)",
                   "parallelism": f"{world} independent matrices"},
        "lloyd_iterations_mean": (iter_sum / iter_rows) if iter_rows else None, "lloyd_iterations_max": ITERS,
        "weights_per_s": world * ROWS * COLS / (ms_step / 1e3),
        "stage_ms": {"cluster": cluster_ms, "allocate": alloc_ms, "quantize": quant_ms},
        "kernel_ms": {"skim_sort16_kernel": sort_ms, "skim_lloyd_kernel": lloyd_ms, "launches_timed": timed_chunks,
                      "note": "stage_ms and kernel_ms: a second pass of the same steps with CUDA events between the kernels"},
        "pipeline_hbm_frac": pipeline_bytes / (ms_step * 1e-3) / 1e9 / peak,
        "cluster_stage_hbm_frac": cluster_bytes / (cluster_ms * 1e-3) / 1e9 / peak,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "consumers": consumers,
        **extra,
        "roofline": {"bound": "hbm", "limiter": "shared-memory wavefronts and instruction issue (ncu); HBM is the roofline the target names",
                     "kernel": DOMINANT_KERNEL, "achieved": achieved, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "traffic": SORT_TRAFFIC_BYTES_PER_ROW * ROWS if SORT_TRAFFIC_BYTES_PER_ROW else None,
                     "algorithmic_bytes": sort_bytes, "kernel_ms": sort_ms},
    }
    if world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline()
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--rows", type=int, default=0, help="profiling only: use fewer rows of the same matrix")
    ap.add_argument("--stage", default="pipeline", choices=["pipeline", "scale", "consumers", "lfull", "exact"],
                    help="pipeline: the benchmark proper; scale / consumers / lfull / exact: time only the alpha-update, the "
                         "unpacking kernels, the L-full error GEMM or the exact clustering on the same matrix (their own "
                         "JSON line; used for profiler captures)")
    args = ap.parse_args()
    if args.rows:
        global ROWS, WORKLOAD
        ROWS = args.rows
        WORKLOAD += f" [PROFILING SUBSET: {ROWS} rows]"
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
