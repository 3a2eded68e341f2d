#!/usr/bin/env python
"""Benchmark of the f-OPD loss hot path (libfopd) on B200.

One step = one pass of the whole path over one batch of synthetic input:
fopd_token_stats on every chunk, fopd_sample_freshness, fopd_loss_fwd_bwd on
every chunk, fopd_loss_finalize.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl fopd|reference]
                  [--workload reasoning|tiny|tool_use|coding_agent|roofline:<rows>x<V>]
                  [--path cached|standalone]

N > 1 (under torchrun): the path has no exchange step, so every rank runs an
independent replica of the workload (different seed); time is the max over
ranks, value the sum of tokens over ranks divided by it ("weak" scaling).
--impl reference times the fp64 CPU oracle on a bounded sample of the same
workload on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused OPD loss fwd+bwd tokens/s and HBM GB/s (% of ~8 TB/s) at V=151,936"
UNIT = "tokens/s"
# What the top-level `value` covers, and where the metric's own figure sits in the line.
VALUE_IS = ("whole hot path per batch (fopd_token_stats on every chunk, fopd_sample_freshness, fopd_loss_fwd_bwd on "
            "every chunk, fopd_loss_finalize); the metric's own figure is metric_figures.loss_fwd_bwd_cached "
            "(fopd_loss_fwd_bwd given the row statistics fopd_token_stats wrote), with the same call without "
            "cached statistics beside it in metric_figures.loss_fwd_bwd_on_chip")
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of a launch over its algorithmic
# bytes, from ncu captures of a small case of the same kernel (4,096 rows x 151,936: larger than
# L2, a few GB on the device); the traffic of a row does not depend on how many rows there are, so
# the ratio scales to a full launch by the rows processed.  A kernel that has changed since its
# counters were taken is taken out of this table (traffic: null).
NCU_TRAFFIC_RATIO = {"grad_stream_kernel": 0.989, "token_stats_kernel": 1.001, "fused_cluster_kernel": 0.990,
                     "grad_sampled_kernel": 0.979, "token_stats_student_kernel": 1.002}

def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="fopd", choices=["fopd", "reference"])
    ap.add_argument("--workload", default="reasoning")
    ap.add_argument("--path", default="cached", choices=["cached", "standalone"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--vocab-shards", type=int, default=8,
                    help="also time the vocabulary-sharded entry points with this many column ranges (0: skip)")
    ap.add_argument("--max-chunks", type=int, default=0,
                    help="keep only the first K chunks of a chunked workload (0: all)")
    ap.add_argument("--resident-chunks", type=int, default=0,
                    help="chunks of a chunked workload whose logits are generated and kept on the device; the "
                         "other chunks reuse them in turn with their own mask and sample ids (0: as many as fit, at most 3)")
    ap.add_argument("--no-sampled", action="store_true", help="skip the timing of the sampled-token form of the loss")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-on-chip", action="store_true", help="skip the extra timing of the on-chip fwd+bwd kernel")
    ap.add_argument("--cpu-sample-rows", type=int, default=0, help="rows of the CPU-oracle sample (0 = auto)")
    return ap.parse_args()


def make_workload(name: str):
    from paper_2605_17862_b200 import synth

    if name.startswith("roofline:"):
        rows, V = name.split(":")[1].split("x")
        return synth.roofline_point(int(rows), int(V))
    return synth.WORKLOADS[name]()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0=None, t1=None):
        """Summary of the samples taken between wall-clock times t0 and t1 (all samples if none fall there)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for t, r in self.rows if t0 is not None and t0 <= t <= t1 + 0.05]
        for r in inside or [r for _, r in self.rows]:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm),
                "sampled": "during the timed region" if inside else "around the timed region", "reasons": sorted(reasons)}


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def replica_throughput(tokens_per_rank: int, ms_per_step_local: float, device=None):
    """Replicas-only scaling: every rank processes its own copy of the workload, the
    job's time is the slowest rank's, its work the sum over ranks."""
    import torch.distributed as dist

    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = max_over_ranks(ms_per_step_local, device)
    return world * tokens_per_rank / (ms * 1e-3), ms


def algorithmic_bytes(wl, active_rows: int):
    """Minimum bytes: statistics sweep reads S and T of aligned rows; the loss
    fwd+bwd reads S and T of differentiated rows once and writes every dlogits row."""
    e = 2 if str(wl.dtype).endswith("bfloat16") else 4
    aligned = int(wl.mask.sum())
    row = wl.V * e
    stats = 2 * row * aligned
    grad = 3 * row * active_rows + row * (wl.n_rows - active_rows)
    return stats, grad


def run_reference(args, rank: int):
    """CPU oracle on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    import torch
    from oracle import fopd_oracle as orc
    from paper_2605_17862_b200 import synth

    wl = make_workload(args.workload)
    # rows per step sized so that warm-up + steps stay within a few minutes on the host cores
    rows = args.cpu_sample_rows or max(128, min(2048, 40960 // max(1, args.steps + args.warmup)))
    res = time_oracle(wl, rows, steps=args.steps, warmup=args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "rows": wl.n_rows, "vocab": wl.V, "samples": wl.B, "sample": res["sample"]},
        "cpu_baseline": {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.lower().startswith("model name"):
                    return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def time_oracle(wl, sample_rows: int, steps: int = 1, warmup: int = 0, chunk0=None, threads: int = 0):
    """Times the oracle, as it stands, on the first `sample_rows` aligned rows of
    chunk 0: the statistics pass, per-sample sums, freshness, loss and the
    gradient of every sampled row (the same steps the GPU path runs).  The rows
    are copied from `chunk0` (the already generated device chunk) when given,
    else generated on the host; the gradient is taken in blocks of rows so that
    its fp64 output stays small."""
    import numpy as np
    from oracle import fopd_oracle as orc
    from paper_2605_17862_b200 import synth

    lo, hi = wl.chunk_range(0)
    aligned = np.nonzero(wl.mask[lo:hi])[0][:sample_rows]
    n = int(aligned.max()) + 1 if len(aligned) else 0
    if chunk0 is not None:
        ch = {k: v[:n].cpu() for k, v in chunk0.items()}
    else:
        sub = synth.Workload(wl.name, wl.B, wl.V, wl.dtype, n, wl.sample_id[:n], wl.mask[:n], wl.tau, wl.H,
                             wl.sigma_s, wl.boost_frac, wl.boost, wl.sigma_t, wl.sigma_b, wl.seed)
        ch = synth.gen_chunk(sub, 0, "cpu", row_block=64)
    P = synth.DEFAULT_PARAMS
    all_threads = orc.num_threads()
    if threads:
        orc.set_threads(threads)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        r = orc.run_batch([ch], wl.B, wl.tau, wl.H, None, P["alpha"], P["beta"], P["xi"], P["lam"])
        for r0 in range(0, len(aligned), 256):
            orc.grad_rows(ch["student"], ch["teacher"], ch["tokens"], ch["behav_logprob"], ch["mask"],
                          ch["sample_id"], r.fresh.coef, P["lam"], aligned[r0:r0 + 256])
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    dt = sum(times) / len(times)
    cores = orc.num_threads()
    if threads:
        orc.set_threads(all_threads)
    return {"value": len(aligned) / dt, "ms_per_step": dt * 1e3, "cores": cores,
            "sample": f"first {len(aligned)} aligned rows of chunk 0 ({n} rows incl. masked), V={wl.V}, "
                      f"stats + freshness + loss + gradient of every sampled row, {dt:.1f} s per pass"}


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2605_17862_b200 import binding as fb
    from paper_2605_17862_b200 import pipeline as pl
    from paper_2605_17862_b200 import synth

    fb.lib()  # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = make_workload(args.workload)
    wl.seed = wl.seed + 100 * rank  # independent replica per rank
    if args.max_chunks and args.max_chunks < wl.n_chunks:
        import dataclasses
        keep = args.max_chunks * wl.chunk_rows
        wl = dataclasses.replace(wl, name="%s[first %d chunks]" % (wl.name, args.max_chunks),
                                 sample_id=wl.sample_id[:keep], mask=wl.mask[:keep])
    esz = 2 if wl.dtype == torch.bfloat16 else 4
    free_dev, _ = torch.cuda.mem_get_info(dev)
    chunk_bytes = 3 * min(wl.chunk_rows, wl.n_rows) * wl.V * esz   # S, T, dlogits of one chunk
    fit = int((0.85 * free_dev) // chunk_bytes)
    if fit < 1:
        raise SystemExit("workload %s needs %.0f GB per chunk (S, T, dlogits); %.0f GB free"
                         % (wl.name, chunk_bytes / 1e9, free_dev / 1e9))
    # Chunked workloads stream: the logits of the first K chunks stay on the device and chunk j
    # works on the logits, tokens and behaviour log-probs of chunk j % K (rows are i.i.d.) with
    # its OWN mask and sample ids, so the per-sample structure, the number of aligned rows and
    # the gates are the workload's; K x 15 GB cycled through is far larger than L2.
    K = wl.n_chunks if wl.n_chunks <= fit and not args.resident_chunks else min(
        wl.n_chunks, fit, args.resident_chunks or 3)
    slots = [synth.gen_chunk(wl, j, dev) for j in range(K)]
    chunks_d = []
    for j in range(wl.n_chunks):
        lo, hi = wl.chunk_range(j)
        n = hi - lo
        if j < K:
            chunks_d.append(slots[j])
        else:
            base = slots[j % K]
            chunks_d.append(dict(student=base["student"][:n], teacher=base["teacher"][:n], tokens=base["tokens"][:n],
                                 behav_logprob=base["behav_logprob"][:n],
                                 mask=torch.from_numpy(wl.mask[lo:hi].copy()).to(dev),
                                 sample_id=torch.from_numpy(wl.sample_id[lo:hi].copy()).to(dev)))
    chunks = [pl.to_chunk(c) for c in chunks_d]
    dl_slots = [torch.empty_like(c["student"]) for c in slots]
    dlogits = [dl_slots[j % K][:chunks_d[j]["student"].shape[0]] for j in range(wl.n_chunks)]
    rows = [pl.RowOutputs.alloc(c["student"].shape[0], dev) for c in chunks_d]
    buf = pl.BatchBuffers(wl.B, dev)
    P = synth.DEFAULT_PARAMS
    p = fb.params(**P)
    tau = torch.as_tensor(wl.tau, device=dev)
    H = torch.as_tensor(wl.H, device=dev)
    cached = args.path == "cached"

    def one_step(ev=None):
        buf.reset()
        if ev: ev[0].record()
        pl.measure(chunks, buf, rows, keep_row_ws=cached)
        if ev: ev[1].record()
        pl.freshness(buf, tau, H, None, p)
        if ev: ev[2].record()
        pl.optimise(chunks, dlogits, buf, p, rows, use_row_ws=cached)
        if ev: ev[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()
    assert fb.fopd_check_status(buf.status) == 0
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    wall0 = time.time()
    t_begin.record()
    for k in range(args.steps):
        one_step(events[k])
    t_end.record()
    barrier()
    clocks = sampler.stop(wall0, time.time()) if rank == 0 else None
    total_ms = t_begin.elapsed_time(t_end)
    stats_all = [e[0].elapsed_time(e[1]) for e in events]   # all chunks of the batch
    grad_all = [e[2].elapsed_time(e[3]) for e in events]
    stats_ms, grad_ms = statistics.mean(stats_all), statistics.mean(grad_all)

    # the same loss forward + backward without cached row statistics (on-chip kernel), timed
    # on its own after the step timing: what a caller pays when the student logits changed
    # between the measurement and the optimisation phase
    on_chip_ms = None
    if cached and not args.no_on_chip:
        for it in range(3 + args.steps):
            if it == 3:
                torch.cuda.synchronize()
                t_begin.record()
            for j, ch in enumerate(chunks):
                fb.fopd_loss_fwd_bwd(ch, buf.B, buf.coef, p, dlogits[j], buf.loss_acc, status=buf.status)
        t_end.record()
        torch.cuda.synchronize()
        on_chip_ms = t_begin.elapsed_time(t_end) / args.steps

    # the whole step with the fewest bytes: the measurement phase reads the student rows only
    # (all the freshness needs), the loss phase runs without cached statistics
    student_step = None
    if cached and not args.no_on_chip:
        ev_s = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for it in range(3 + args.steps):
            if it == 3:
                torch.cuda.synchronize()
                t_begin.record()
            buf.reset()
            if it == 3 + args.steps - 1: ev_s[0].record()
            pl.measure_student(chunks, buf, None)
            if it == 3 + args.steps - 1: ev_s[1].record()
            pl.freshness(buf, tau, H, None, p)
            pl.optimise(chunks, dlogits, buf, p, None, use_row_ws=False)
        t_end.record()
        torch.cuda.synchronize()
        assert fb.fopd_check_status(buf.status) == 0
        student_step = {"ms_per_batch": t_begin.elapsed_time(t_end) / args.steps,
                        "student_stats_ms_last_step": ev_s[0].elapsed_time(ev_s[1]), "loss": float(buf.loss.cpu()[0])}

    # the sampled-token form of the token loss (importance-weighted reverse KL on the stored token):
    # its own measurement phase for the row statistics and weights, then the timed loss forward +
    # backward, which reads only the student row of a differentiated row
    sampled = None
    if cached and not args.no_sampled:
        s_chunks = [pl.to_chunk(c, loss_kind=fb.LOSS_SAMPLED_KL) for c in chunks_d]
        s_buf = pl.BatchBuffers(wl.B, dev)
        s_rows = rows  # the full-vocabulary statistics are not needed any more
        pl.measure(s_chunks, s_buf, s_rows, keep_row_ws=True)
        pl.freshness(s_buf, tau, H, None, p)
        for it in range(3 + args.steps):
            if it == 3:
                torch.cuda.synchronize()
                t_begin.record()
            pl.optimise(s_chunks, dlogits, s_buf, p, s_rows, use_row_ws=True)
        t_end.record()
        torch.cuda.synchronize()
        s_buf.loss_acc.zero_()  # the timed repetitions all added to it
        pl.optimise(s_chunks, dlogits, s_buf, p, s_rows, use_row_ws=True)
        s_coef = s_buf.coef.cpu().numpy()
        s_active = int(((s_coef[np.clip(wl.sample_id, 0, wl.B - 1)] > 0) & (wl.mask > 0)).sum())
        s_ms = t_begin.elapsed_time(t_end) / args.steps
        s_bytes = wl.V * (2 if wl.dtype == torch.bfloat16 else 4) * (2 * s_active + (wl.n_rows - s_active))
        sampled = {"kernel": "grad_sampled_kernel", "ms_per_batch": s_ms, "differentiated_rows": s_active,
                   "tokens_per_s": s_active / (s_ms * 1e-3), "algorithmic_bytes": s_bytes,
                   "bytes_per_differentiated_row": "2 V e (student read, gradient written)",
                   "loss": float(s_buf.loss.cpu()[0])}

    # the vocabulary-sharded entry points on the same rows: every holder's column range in turn
    # on this one GPU (partial sums of all parts, one merge, every part's gradient), so the sums
    # over the parts compare with the whole-row kernels above
    sharded = None
    if cached and args.vocab_shards > 1 and len(chunks) == 1:
        pl.measure(chunks, buf, rows, keep_row_ws=True)  # (the sampled form above reused the row workspace)
        sharded = time_vocab_sharded(args, wl, chunks_d[0], dlogits[0], rows[0], buf, p, dev)

    coef = buf.coef.cpu().numpy()
    active_rows = int(((coef[np.clip(wl.sample_id, 0, wl.B - 1)] > 0) & (wl.mask > 0)).sum())
    aligned = int(wl.mask.sum())
    stats_bytes, grad_bytes = algorithmic_bytes(wl, active_rows)
    value, ms_per_step = replica_throughput(aligned, total_ms / args.steps, dev)
    peak, peak_src = measured_peak()
    n_chunks = len(chunks)
    # per chunk: statistics sweep (+ 2 row-range kernels) + per-sample reduction; gradient sweep (or
    # row weights + on-chip kernel) (+ 2 row-range kernels) + per-sample reduction; per batch: freshness, finalize
    ranges = 0 if wl.B <= 32 else 2  # (batches of few samples: the reductions find the row ranges themselves)
    kernels_per_step = n_chunks * ((2 + ranges) + ((2 if cached else 3) + ranges)) + 2
    plan = fb.fopd_loss_fwd_bwd_plan(wl.dtype, wl.V)
    on_chip_kernel = "fused_cluster_kernel" if plan["cluster_size"] else "token_stats_kernel+grad_stream_kernel"
    grad_kernel = "grad_stream_kernel" if cached else on_chip_kernel

    def figure(ms, nbytes, rows_done):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"ms_per_batch": ms, "tokens_per_s": rows_done / (ms * 1e-3), "gbs": gbs,
                "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}

    achieved = grad_bytes / (grad_ms * 1e-3) / 1e9
    ratio = NCU_TRAFFIC_RATIO.get(grad_kernel)
    traffic = None if ratio is None else ratio * grad_bytes / n_chunks
    traffic_src = None if ratio is None else (
        "ncu dram__bytes_read.sum + dram__bytes_write.sum of the 4,096 x 151,936 case of the same kernel, over its "
        "algorithmic bytes (%.3f), times the algorithmic bytes of one launch here" % ratio)
    if sampled:
        sampled.update({k: v for k, v in figure(sampled["ms_per_batch"], sampled["algorithmic_bytes"],
                                                sampled["differentiated_rows"]).items() if k != "ms_per_batch"})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "value_is": VALUE_IS,
        "config": {
            "workload": wl.name, "rows": wl.n_rows, "aligned_tokens": aligned, "differentiated_rows": active_rows,
            "vocab": wl.V, "samples": wl.B, "logits_dtype": str(wl.dtype).replace("torch.", ""),
            "chunks": n_chunks, "chunk_rows": wl.chunk_rows, "path": args.path,
            "resident_chunks": K,
            "chunk_streaming": None if K == n_chunks else
            "logits, tokens and behaviour log-probs of chunk j are those of generated chunk j mod %d (rows are "
            "i.i.d.); mask and sample ids are chunk j's own; both loops of Algorithm 1 run over all %d chunks"
            % (K, n_chunks),
            "fused_plan": None if cached else plan, "tokens_counted": "aligned (mask = 1) rows",
            "l2": "%d x 3 x %.2f GB of logits and gradients cycled through, far larger than the 126 MB L2, no flush needed"
                  % (K, min(wl.chunk_rows, wl.n_rows) * wl.V * esz / 1e9),
            "parallelism": "replicas only" if world > 1 else "1 gpu", "params": P,
        },
        "gpu_launches": kernels_per_step * args.steps,
        "phases_ms": {"token_stats_per_batch": stats_ms, "loss_fwd_bwd_per_batch": grad_ms,
                      "token_stats_median_best": [statistics.median(stats_all), min(stats_all)],
                      "loss_fwd_bwd_median_best": [statistics.median(grad_all), min(grad_all)],
                      "freshness": statistics.mean(e[1].elapsed_time(e[2]) for e in events)},
        "metric_figures": {
            "loss_fwd_bwd_cached" if cached else "loss_fwd_bwd_standalone": dict(
                figure(grad_ms, grad_bytes, active_rows), kernel=grad_kernel,
                bytes="3 V e per differentiated row, V e per other row"),
            "whole_step_student_statistics": None if student_step is None else dict(
                figure(student_step["ms_per_batch"], stats_bytes / 2 + grad_bytes, aligned),
                student_stats_ms=student_step["student_stats_ms_last_step"], loss=student_step["loss"],
                calls="fopd_token_stats_student, fopd_sample_freshness, fopd_loss_fwd_bwd(row_ws = NULL), fopd_loss_finalize",
                bytes="V e per aligned row, then 3 V e per differentiated row (V e per other row): 4 V e in all"),
            "loss_fwd_bwd_on_chip": None if on_chip_ms is None else dict(
                figure(on_chip_ms, grad_bytes, active_rows), kernel=on_chip_kernel, plan=plan),
            "loss_fwd_bwd_sampled_token_form": sampled,
            "token_stats": dict(figure(stats_ms, stats_bytes, aligned), bytes="2 V e per aligned row"),
            "whole_step": dict(figure(ms_per_step, stats_bytes + grad_bytes, aligned),
                               bytes="5 V e per differentiated row as run (two sweeps), against 3 V e at the least"),
        },
        "roofline": {"bound": "hbm", "kernel": grad_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src,
                     "traffic": traffic, "traffic_source": traffic_src,
                     "launches_per_step": n_chunks,
                     "algorithmic_bytes_per_launch": grad_bytes / n_chunks},
        "clocks": clocks,
        "loss": float(buf.loss.cpu()[0]),
    }
    if sharded:
        e = 2 if wl.dtype == torch.bfloat16 else 4
        sharded["stats_gbs"] = stats_bytes / (sharded["stats_ms_all_parts"] * 1e-3) / 1e9
        sharded["grad_gbs"] = grad_bytes / (sharded["grad_ms_all_parts"] * 1e-3) / 1e9
        line["vocab_sharded"] = sharded

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    if not args.no_e2e and len(chunks) >= 1:
        try:
            import psutil
            need_host = 3 * sum(c["student"].numel() * c["student"].element_size() for c in slots)
            # from the host's total memory, so that every rank takes the same decision
            if need_host * world > 0.6 * psutil.virtual_memory().total:
                raise MemoryError("pinned host copies of the batch (%.0f GB) would not fit comfortably in host memory"
                                  % (need_host / 1e9))
            line["e2e"] = run_e2e(args, wl, slots, chunks_d, dev, world, aligned)
        except Exception as exc:  # report, never fake
            line["e2e"] = {"value": None, "unit": UNIT, "error": repr(exc)[:200]}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        res = time_oracle(wl, args.cpu_sample_rows or 32768, chunk0=chunks_d[0])
        one = time_oracle(wl, max(64, (args.cpu_sample_rows or 32768) // 24), chunk0=chunks_d[0], threads=1)
        line["cpu_baseline"] = {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                                "sample": res["sample"], "cpu_model": cpu_model(), "host_cores": os.cpu_count(),
                                "single_thread": {"value": one["value"], "sample": one["sample"]}}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_vocab_sharded(args, wl, ch, dlogits, row_out, buf, p, dev):
    """CUDA-event times of fopd_shard_stats (all parts), fopd_shard_merge and
    fopd_shard_loss_fwd_bwd (all parts) on one chunk; buf.coef holds the step's weights."""
    import torch
    from paper_2605_17862_b200 import binding as fb

    K, V, n = args.vocab_shards, wl.V, ch["tokens"].numel()
    per = 16 // (2 if wl.dtype == torch.bfloat16 else 4)
    cuts = [0] + [per * ((V * k // K) // per) for k in range(1, K)] + [V]
    ranges = list(zip(cuts[:-1], cuts[1:]))
    mk = lambda a, b: fb.Chunk(ch["student"][:, a:b], ch["teacher"][:, a:b], ch["behav_logprob"], ch["tokens"],
                               ch["mask"], ch["sample_id"])
    shards = [mk(a, b) for a, b in ranges]
    parts = torch.empty((K, n, 8), dtype=torch.float32, device=dev)
    acc = torch.zeros((wl.B, 4), dtype=torch.float64, device=dev)
    lacc = torch.zeros((wl.B, 2), dtype=torch.float64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    tot = [0.0, 0.0, 0.0]
    for it in range(3 + args.steps):
        ev[0].record()
        for k, (a, b) in enumerate(ranges):
            fb.fopd_shard_stats(shards[k], a, V, parts[k])
        ev[1].record()
        fb.fopd_shard_merge(parts, ch["behav_logprob"], ch["tokens"], ch["mask"], ch["sample_id"], V, wl.B, acc,
                            row_out.row_ws, status=status)
        ev[2].record()
        for k, (a, b) in enumerate(ranges):
            fb.fopd_shard_loss_fwd_bwd(shards[k], a, V, wl.B, buf.coef, row_out.row_ws, p, dlogits[:, a:b],
                                       loss_acc=lacc if k == 0 else None)
        ev[3].record()
        torch.cuda.synchronize()
        if it >= 3:
            for q in range(3):
                tot[q] += ev[q].elapsed_time(ev[q + 1]) / args.steps
    assert fb.fopd_check_status(status) == 0
    return {"parts": K, "columns_per_part": cuts[1], "stats_ms_all_parts": tot[0], "merge_ms": tot[1],
            "grad_ms_all_parts": tot[2], "launches_per_pass": 2 * K + 3}


def run_e2e(args, wl, slots, chunks_d, dev, world, aligned):
    """Same step through fopd_step_host: logits start in pinned host memory, every step
    uploads them, runs the path and downloads dlogits and the per-sample results.  A chunked
    workload whose chunks share the logits of a few generated ones on the device shares them in
    host memory the same way (every chunk is still uploaded, and its gradient downloaded)."""
    import torch
    import torch.distributed as dist
    from paper_2605_17862_b200 import binding as fb
    from paper_2605_17862_b200 import pipeline as pl
    from paper_2605_17862_b200 import synth

    K = len(slots)
    h_slots = [{k: v.cpu().pin_memory() for k, v in c.items()} for c in slots]
    h_dl = [torch.empty_like(c["student"]).pin_memory() for c in h_slots]
    host, hdl = [], []
    for j, c in enumerate(chunks_d):
        n = c["student"].shape[0]
        base = h_slots[j % K]
        if j < K:
            host.append(base)
        else:
            host.append(dict(student=base["student"][:n], teacher=base["teacher"][:n], tokens=base["tokens"][:n],
                             behav_logprob=base["behav_logprob"][:n], mask=c["mask"].cpu().pin_memory(),
                             sample_id=c["sample_id"].cpu().pin_memory()))
        hdl.append(h_dl[j % K][:n])
    hchunks = [pl.to_chunk(c) for c in host]
    need = fb.fopd_step_host_workspace_bytes(hchunks, wl.B, True)
    free, _ = torch.cuda.mem_get_info(dev)
    if need > free - (2 << 30) or K < len(chunks_d):
        need = fb.fopd_step_host_workspace_bytes(hchunks, wl.B, False)
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    tau = torch.as_tensor(wl.tau)
    H = torch.as_tensor(wl.H)
    p = fb.params(**synth.DEFAULT_PARAMS)
    fb.fopd_step_host(hchunks, wl.B, tau, H, None, p, hdl, ws)  # warm-up
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        res = fb.fopd_step_host(hchunks, wl.B, tau, H, None, p, hdl, ws)
    torch.cuda.synchronize()
    dt = max_over_ranks((time.perf_counter() - t0) / args.e2e_steps, dev)
    resident = need == fb.fopd_step_host_workspace_bytes(hchunks, wl.B, True)
    # bytes as counted by the library from the copies it issued: logits of aligned rows only
    # (rows with mask = 0 are never read, so they are not uploaded), every gradient row back
    return {"value": world * aligned / dt, "unit": UNIT, "ms_per_step": dt * 1e3,
            "h2d_bytes_per_step": int(res["copied_bytes"][0]), "d2h_bytes_per_step": int(res["copied_bytes"][1]),
            "steps": args.e2e_steps, "api": "fopd_step_host (pinned host buffers)",
            "mode": "logits resident, uploads / kernels / downloads overlapped" if resident else "two uploads per chunk",
            "loss": float(res["loss"][0])}


if __name__ == "__main__":
    main()
