#!/usr/bin/env python
"""Benchmark: GCN epochs/sec over all extended partitions on one B200.

A step is one epoch of the whole training path: for every extended partition
forward + backward (feature transform, normalized-adjacency SpMM, bias + ReLU,
masked softmax cross-entropy, transposed SpMM, gradient GEMMs), then the
gradient average + Adam.  The workload is the synthetic paper-scale graph
(232 965 vertices, 114.6 M directed non-zeros, 602 features, 41 classes, hidden
128, 5 partitions, overlap 10 %).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload paper_scale|large_sparse|small|tiny] [--scale S]

With N > 1 (launched by torch.distributed.run) every rank trains an independent
replica of the same workload on its own GPU; no collective is on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GCN epochs/sec over all augmented partitions"
# dram__bytes_read.sum + dram__bytes_write.sum per spmm_rows launch (mean over the four launches of one partition in
# an ncu capture of this command on the kernel in use), keyed by (workload, factored_norm); None = not captured for
# that kernel variant.  l1tex__data_pipe_lsu_wavefronts (% of peak) from the same captures.
SPMM_TRAFFIC_BYTES = {("paper_scale", False): 177.0e6, ("paper_scale", True): 97.2e6}
SPMM_L1_PIPE_PCT = {("paper_scale", False): 86.7, ("paper_scale", True): 86.1}
# the same for sage_concat_mean (mean over the hidden-layer and the output-layer launch of a batch)
SAGE_TRAFFIC_BYTES = {"paper_scale": 38.3e6}
UNIT = "epochs/s"
REPEATS = 5   # the K-epoch timed region is repeated; the value is the median repeat


def load_workload(name, scale):
    from gen import configs
    if name in ("paper_scale", "large_sparse"):
        return configs.by_name(name, scale=scale)
    return configs.by_name(name)


def measured_peaks():
    """(HBM copy GB/s, dense bf16 TFLOP/s sustained, max SM MHz, "measured" | "fallback")."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", 1400.0)), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1400.0, 1965.0, "fallback"


def host_threads():
    """Threads the checker's OpenMP loops and numpy's BLAS get on this machine."""
    n = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    for var in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS"):
        if os.environ.get(var, "").isdigit():
            n = min(n, int(os.environ[var]))
    return n


class ClockSampler:
    """nvidia-smi clock / throttle samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.device, self.proc, self.path = device, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.device), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as fh:
            for ln in fh:
                c = [t.strip() for t in ln.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_epochs(w, warmup, steps, budget_s=None):
    """Whole epochs of the fp64 CPU checker as it stands (forward + backward on every extended partition, gradient
    average, Adam), parameters advancing.  Returns (seconds per timed epoch, epochs timed, last loss).  With a
    budget, timing stops after the first epoch that ends beyond it."""
    from oracle import oracle
    _, parts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    xs = [w.x[pt.members].astype(np.float64) for pt in parts]
    ys = [w.y[pt.members] for pt in parts]
    mks = [w.train_mask[pt.members] for pt in parts]
    ws = [a.astype(np.float64) for a in w.w0]
    bs = [b.astype(np.float64) for b in w.b0]
    opt = oracle.Adam(ws + bs, w.lr, w.beta1, w.beta2, w.eps)
    loss = None
    for _ in range(warmup):
        ws, bs, loss, _ = oracle.epoch(parts, xs, ys, mks, ws, bs, opt, w.loss_on_halo)
    done, t0 = 0, time.perf_counter()
    for _ in range(steps):
        ws, bs, loss, _ = oracle.epoch(parts, xs, ys, mks, ws, bs, opt, w.loss_on_halo)
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    return (time.perf_counter() - t0) / max(done, 1), done, loss


def run_reference(args):
    """The reference arm: the fp64 CPU checker, as it stands, on the host cores.  A step is one whole epoch of the
    same workload, so the line's ms_per_step is the time of what a step ran."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = load_workload(args.workload, args.scale)
    s_per_epoch, done, loss = oracle_epochs(w, args.warmup, args.steps)
    value = 1.0 / s_per_epoch
    cores = host_threads()
    sample = f"{done} whole epochs (forward + backward on all {w.m} extended partitions, gradient average, Adam) after {args.warmup} warm-up epochs"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": done,
            "warmup": args.warmup, "ms_per_step": 1e3 * s_per_epoch, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "n": w.n, "nnz": w.nnz, "dims": w.dims, "partitions": w.m,
                       "overlap_ppm": w.overlap_ppm, "final_loss": loss},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def cpu_baseline(w, args):
    """The checker timed on the host cores on the same workload: up to 3 whole epochs (Adam included) within about
    30 s; for the two small workloads also on one thread (a child process with the thread counts set to 1)."""
    s_per_epoch, done, _ = oracle_epochs(w, 0, 3 if w.n > 50_000 else 20, budget_s=30.0)
    out = {"value": 1.0 / s_per_epoch, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
           "sample": f"{done} whole epochs ({done * s_per_epoch:.1f} s) of the same workload, Adam included"}
    if w.name in ("tiny", "small"):
        env = dict(os.environ, OMP_NUM_THREADS="1", OPENBLAS_NUM_THREADS="1", MKL_NUM_THREADS="1")
        try:
            r = subprocess.run([sys.executable, os.path.abspath(__file__), "--impl", "reference", "--workload", w.name,
                                "--steps", "5", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=600)
            one = json.loads(r.stdout.strip().splitlines()[-1])
            out["single_thread"] = {"value": one["value"], "unit": UNIT, "cores": 1}
        except Exception as e:  # noqa: BLE001 - the figure is context only
            out["single_thread"] = {"value": None, "error": str(e)[:200]}
    return out


def run_ours(args):
    import torch
    from paper_2012_04930_b200 import gcnsa
    from paper_2012_04930_b200 import dist as gdist

    rank, world, local = gdist.init_from_env("nccl" if torch.cuda.is_available() else "gloo")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    w = load_workload(args.workload, args.scale)
    if args.graph:
        # a recorded epoch needs a stream of its own (the legacy default stream cannot be recorded); torch's events
        # below time whatever stream is current, so make it current for the rest of the run
        torch.cuda.set_stream(torch.cuda.Stream())
    env = gcnsa.make_env(local)
    t0 = time.perf_counter()
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo, order_window=args.order_window)
    build_s = time.perf_counter() - t0
    gemm_mode = gcnsa.GEMM_FP32 if args.gemm == "fp32" else gcnsa.GEMM_TF32X3
    model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        gemm_mode=gemm_mode, loss_rows_only=1, epoch_graph=int(args.graph),
                        factored_norm=int(args.factored_norm))
    infos = [parts.info(p) for p in range(w.m)]
    loss = torch.zeros(1, device="cuda")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()            # samples cover the warm-up and the timed region (both under load)
    for _ in range(max(args.warmup, 3)):
        model.epoch(loss.data_ptr())
    torch.cuda.synchronize()

    # ---- device-timed region: K epochs, inputs resident in HBM ----
    # Without --graph the per-kernel events are recorded inside this region; with it the region replays the recorded
    # epoch (no events between kernels) and the per-kernel figures come from a second pass of K epochs after it.
    # An epoch reads every partition's feature rows and both CSRs.  Where that is more than L2 holds, consecutive
    # epochs cannot find their inputs cached and the K epochs are timed back to back; otherwise a buffer of twice
    # the L2 size is written before every timed epoch (outside its events) and the K event times are added.
    l2_bytes = int(getattr(torch.cuda.get_device_properties(local), "L2_cache_size", 126 * 2 ** 20))
    epoch_input_bytes = int(sum(i.n * ((w.dims[0] + 15) // 16 * 16) * 4 + 2 * i.nnz * 4 for i in infos))
    flush = None if epoch_input_bytes > l2_bytes else torch.empty(2 * l2_bytes, dtype=torch.uint8, device="cuda")

    def timed_pass():
        gdist.barrier()
        torch.cuda.synchronize()
        n0 = gcnsa.launch_count()
        if flush is None:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for _ in range(args.steps):
                model.epoch(loss.data_ptr())
            ev1.record()
            torch.cuda.synchronize()
            ms_pass = ev0.elapsed_time(ev1)
        else:
            evs = []
            for _ in range(args.steps):
                flush.zero_()
                ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                ev0.record()
                model.epoch(loss.data_ptr())
                ev1.record()
                evs.append((ev0, ev1))
            torch.cuda.synchronize()
            ms_pass = sum(a.elapsed_time(b) for a, b in evs)
        gdist.barrier()
        return gdist.max_over_ranks(ms_pass), gcnsa.launch_count() - n0

    tc0, fb0 = gcnsa.gemm_path_counts()
    if args.graph:
        # the K-epoch region REPEATS times; the value is the median repeat (K epochs each, as --steps says)
        runs = [timed_pass() for _ in range(REPEATS)]
        final_loss = loss.item()
        model.profile(True)
        ms_profiled, _ = timed_pass()
    else:
        model.profile(True)
        runs = [timed_pass()]
        final_loss = loss.item()
        ms_profiled = runs[0][0]
    prof = model.profile_read()
    model.profile(False)
    tc1, fb1 = gcnsa.gemm_path_counts()
    all_ms = sorted(r[0] for r in runs)
    ms, launches = all_ms[len(all_ms) // 2], runs[0][1]
    clocks = sampler.stop() if rank == 0 else {}

    # ---- reported separately: the same training with A_hat X kept across epochs (layer 1 then needs no sparse
    # product in either direction; an algebraic shortcut, so it is not the headline value) ----
    cached = None
    if args.cache_ax_leg:
        model_c = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                              gemm_mode=gemm_mode, loss_rows_only=1, epoch_graph=int(args.graph),
                              factored_norm=int(args.factored_norm), cache_ax=1)
        loss_c = torch.zeros(1, device="cuda")
        for _ in range(max(args.warmup, 3)):
            model_c.epoch(loss_c.data_ptr())
        gdist.barrier()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(args.steps):
            model_c.epoch(loss_c.data_ptr())
        ev1.record()
        torch.cuda.synchronize()
        ms_c = gdist.max_over_ranks(ev0.elapsed_time(ev1))
        cached = {"value": world * args.steps / (ms_c * 1e-3), "unit": UNIT, "ms_per_step": ms_c / args.steps,
                  "final_loss": loss_c.item(),
                  "note": "cache_ax=1: A_hat X computed once per partition, layer 1 runs as (A_hat X) W; "
                          "not the headline (skips the per-epoch layer-1 sparse products)"}
        model_c.close()

    # ---- end to end: the same epochs through the host-buffer entry point ----
    xs = [torch.from_numpy(np.ascontiguousarray(w.x[parts.members(p)])).pin_memory() for p in range(w.m)]
    ptrs = [x.data_ptr() for x in xs]
    loss_h = np.zeros(1, np.float32)
    for _ in range(2):
        model.epoch_host(ptrs, loss_h)
    gdist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        model.epoch_host(ptrs, loss_h)
    e2e_s = gdist.max_over_ranks(time.perf_counter() - t0)
    h2d = int(sum(x.numel() * 4 for x in xs))

    if rank == 0:
        peak_hbm, peak_bf16, sm_max_mhz, peak_kind = measured_peaks()
        props = torch.cuda.get_device_properties(local)
        sp, ge = prof["spmm"], prof["gemm"]
        sp_s = max(sp["ms"] * 1e-3, 1e-12)
        nnz_total = int(sum(i.nnz for i in infos))
        # the sparse products gather rows of an n_p x F' matrix; F' = the narrower side of the layer
        widths = [min(a, b) for a, b in zip(w.dims[:-1], w.dims[1:])]
        gathered_bytes = max(i.n for i in infos) * max(widths) * 4
        l2_bytes = int(getattr(props, "L2_cache_size", 126 * 2 ** 20))
        exceeds_l2 = gathered_bytes > l2_bytes
        # L1 data path of all SMs: 128 bytes per clock each, at the SM clock sampled under load
        sm_mhz = clocks.get("sm_mhz") or sm_max_mhz
        peak_l1 = props.multi_processor_count * 128.0 * sm_mhz * 1e6 / 1e9
        hbm_gbs = sp["alg_bytes"] / sp_s / 1e9
        hbm_gbs_val = sp["alg_bytes_val"] / sp_s / 1e9
        l1_gbs = sp["l1_bytes"] / sp_s / 1e9
        key = (w.name, bool(args.factored_norm))
        # the unit that binds is the one closest to its roof: HBM when the gathers miss L2 (no locality and a gathered
        # matrix beyond L2), the L1 data path of the SMs otherwise
        hbm_bound = hbm_gbs / peak_hbm >= l1_gbs / peak_l1
        roofline = {
            "kernel": "spmm_rows", "bound": "hbm" if hbm_bound else "l1",
            "achieved": hbm_gbs if hbm_bound else l1_gbs, "peak": peak_hbm if hbm_bound else peak_l1, "unit": "GB/s",
            "frac": (hbm_gbs / peak_hbm) if hbm_bound else (l1_gbs / peak_l1),
            "peak_kind": (peak_kind + " HBM copy") if hbm_bound else
                         f"derived: {props.multi_processor_count} SMs x 128 B/clk x {sm_mhz:.0f} MHz (SM clock sampled under load)",
            "why": ("the gathers miss L2: HBM is the unit closest to its roof" if hbm_bound else
                    "the gathers hit L2 (" + ("ids are community-ordered although the gathered matrix exceeds L2"
                                              if exceeds_l2 else "the gathered matrix is L2-resident") +
                    "): HBM carries little more than the compulsory bytes, the L1 data path is the unit closest to its roof"),
            "gathered_matrix_bytes": int(gathered_bytes), "l2_bytes": l2_bytes,
            "frac_l1": l1_gbs / peak_l1,
            "traffic": SPMM_TRAFFIC_BYTES.get(key),
            "traffic_note": None if key in SPMM_TRAFFIC_BYTES else "no ncu capture of this workload / kernel variant",
            "alg_bytes_per_launch": sp["alg_bytes"] / max(sp["launches"], 1),
            "l1_bytes_per_launch": sp["l1_bytes"] / max(sp["launches"], 1),
            # the HBM view of the same launches, with the bytes the kernel in use must move (4 B per stored entry
            # when the normalization is factored out) and with 8 B per stored entry (index + value)
            "frac_hbm": {"peak": peak_hbm, "peak_kind": peak_kind, "achieved": hbm_gbs, "frac": hbm_gbs / peak_hbm,
                         "achieved_8B_per_nnz": hbm_gbs_val, "frac_8B_per_nnz": hbm_gbs_val / peak_hbm},
            "l1_data_pipe_pct_of_peak_ncu": SPMM_L1_PIPE_PCT.get(key),
            "launches": sp["launches"], "avg_launch_ms": sp["ms"] / max(sp["launches"], 1),
            "share_of_step": sp["ms"] / ms_profiled}
        # what the SMs can gather when the indices cost nothing: the library's probe (512-byte rows at indices the
        # warps compute themselves) on a matrix as large as the largest gathered one, measured here with events
        n_probe = int(max(i.n for i in infos))
        xp = torch.zeros((n_probe, 128), device="cuda")
        outp = torch.empty((gcnsa.gather_probe_warps(), 128), device="cuda")
        rounds = 200

        def probe_gbs(hit_every):
            best = 0.0
            for _ in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                gcnsa.op_gather_probe(xp, n_probe, min(64, n_probe), hit_every, rounds, outp)
                e1.record()
                torch.cuda.synchronize()
                best = max(best, outp.shape[0] * rounds * 16 * 512 / (e0.elapsed_time(e1) * 1e-3) / 1e9)
            return best

        ceil_l2, ceil_quarter, ceil_l1 = probe_gbs(0), probe_gbs(4), probe_gbs(1)
        roofline["gather_ceiling"] = {
            "kernel": "gather_probe", "unit": "GB/s", "kind": "measured in this run (CUDA events, best of 4)",
            "matrix_bytes": n_probe * 512, "no_l1_reuse": ceil_l2, "one_l1_hit_in_four": ceil_quarter,
            "all_l1_hits": ceil_l1,
            "note": "24 warps per SM, 16 independent 512-byte gathers in flight each, no index loads; spmm_rows has "
                    "an L1 hit rate of 26 % on paper_scale (ncu), so one hit in four is the comparable line"}
        roofline["frac_of_gather_ceiling"] = l1_gbs / ceil_quarter
        del xp, outp
        ge_s = max(ge["ms"] * 1e-3, 1e-12)
        useful = ge["flops"] / ge_s / 1e12
        terms = 3.0 if gemm_mode else 1.0
        peak_tf32 = peak_bf16 / 2.0
        peak_fma = props.multi_processor_count * 128 * 2 * sm_mhz * 1e6 / 1e12
        gemm_roof = {
            "kernel": "gemm_tf32x3" if gemm_mode else "gemm_tile", "bound": "tensor" if gemm_mode else "alu",
            "achieved": useful, "unit": "TFLOP/s", "peak": peak_tf32 if gemm_mode else peak_fma,
            "frac": useful / (peak_tf32 if gemm_mode else peak_fma),
            "issued": useful * terms, "frac_issued": useful * terms / (peak_tf32 if gemm_mode else peak_fma),
            "peak_kind": (f"{peak_kind} dense bf16 sustained / 2 (nominal tf32 : bf16 ratio)" if gemm_mode else
                          f"derived: {props.multi_processor_count} SMs x 128 lanes x 2 x {sm_mhz:.0f} MHz"),
            "note": "achieved counts each product once; the tensor core issues three TF32 MMAs per product" if gemm_mode else None,
            "launches": ge["launches"], "share_of_step": ge["ms"] / ms_profiled}
        line = {
            "metric": METRIC, "value": world * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "n": w.n, "nnz": w.nnz, "dims": w.dims, "partitions": w.m,
                       "overlap_ppm": w.overlap_ppm, "rows_extended": int(sum(i.n for i in infos)),
                       "nnz_extended": nnz_total, "l2": (f"inputs larger than L2 (CSR + features of an epoch: {epoch_input_bytes / 1e6:.0f} MB)"
                              if flush is None else
                              f"flushed: {2 * l2_bytes >> 20} MiB written before every timed epoch "
                              f"(an epoch's inputs are {epoch_input_bytes / 1e6:.1f} MB)"),
                       "parallelism": "replicas only" if world > 1 else "single GPU", "build_s": round(build_s, 2),
                       "gemm": "tcgen05 tf32 x3 (fp32-level accuracy)" if gemm_mode else "fp32 fma",
                       "gemm_products_on_tensor_cores": tc1 - tc0, "fp32_fallback": fb1 - fb0,
                       "tc_status": gcnsa.tc_status(),
                       "loss_rows_only": True,  # last-layer logits only where the loss reads them; training bit-identical
                       # A_hat T computed as diag(d^-1/2) (A + I) (diag(d^-1/2) T): no value loads in the SpMM
                       "factored_norm": bool(args.factored_norm),
                       "order_window": args.order_window,
                       "epoch_graph": bool(args.graph), "ms_per_step_with_kernel_events": ms_profiled / args.steps,
                       "repeats": {"count": len(all_ms), "ms_per_step": [m_ / args.steps for m_ in all_ms],
                                   "min": all_ms[0] / args.steps, "median": ms / args.steps,
                                   "max": all_ms[-1] / args.steps},
                       "final_loss": final_loss, "with_cached_ax": cached},
            "clocks": clocks,
            "e2e": {"value": world * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": 4},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "roofline_gemm": gemm_roof,
            "kernels": {k: {"ms_per_step": v["ms"] / args.steps, "launches_per_step": v["launches"] / args.steps,
                            "tflops": v["flops"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0}
                        for k, v in prof.items()},
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(w, args)
        print(json.dumps(line), flush=True)
    model.close()
    parts.close()
    gdist.finish()


def sage_cpu_baseline(w, dims, fanout, batch, lr, budget_s=20.0):
    """The GraphSAGE checker on the host cores: whole batches of partition 0 for about budget_s seconds, scaled to an
    epoch by the number of batches of all partitions."""
    from gen import configs
    from oracle import oracle, sage
    ws, wn, bs = configs.sage_weights(dims, w.seed + 77)
    params = [a.astype(np.float64) for pair in zip(ws, wn, bs) for a in pair]
    _, parts = oracle.build_partitions(w.rowptr, w.col, w.m, w.overlap_ppm, w.seed, w.part_mode, w.user_part)
    n_batches = 0
    for pt in parts:
        n_train = int(oracle.train_set(pt, w.train_mask[pt.members], w.loss_on_halo).sum())
        n_batches += (n_train + batch - 1) // batch
    pt = parts[0]
    x, y = w.x[pt.members].astype(np.float64), w.y[pt.members]
    tr = oracle.train_set(pt, w.train_mask[pt.members], w.loss_on_halo)
    opt = oracle.Adam(params, lr)
    done, t0 = 0, time.perf_counter()
    for tg in sage.batches(pt, tr, w.seed, 0, batch):
        fw = sage.batch_forward(pt, x, params, tg, y, w.seed, 0, fanout)
        grads, _ = sage.batch_backward(fw, x, params)
        params = opt.step(params, grads)
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    spent = time.perf_counter() - t0
    return {"value": 1.0 / (spent / done * n_batches), "unit": UNIT, "cores": host_threads(), "kind": "oracle",
            "sample": f"{done} of the {n_batches} batches of one epoch ({spent:.1f} s: sampling, forward, backward, Adam), scaled to an epoch"}


def run_sage(args):
    """The GraphSAGE variant (mean aggregator, fan-outs 25 / 10, batches of 256, hidden 128, per-worker Adam and
    per-epoch parameter averaging) on the same workload; one JSON line.  A step is one epoch over all partitions."""
    import torch
    from gen import configs
    from paper_2012_04930_b200 import gcnsa
    torch.cuda.set_device(0)
    torch.cuda.set_stream(torch.cuda.Stream())   # recorded batches need a stream other than the legacy default one
    w = load_workload(args.workload, args.scale)
    hidden = 128 if w.dims[0] >= 128 else w.dims[1]
    dims, fanout, batch, lr = [w.dims[0], hidden, w.dims[-1]], (25, 10), 256, 1e-4
    ws, wn, bs = configs.sage_weights(dims, w.seed + 77)
    env = gcnsa.make_env(0)
    parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                        w.part_mode, w.user_part, w.loss_on_halo)
    model = gcnsa.Sage(env, parts, dims, ws, wn, bs, fanout=fanout, batch=batch, lr=lr, seed=w.seed,
                       gemm_mode=gcnsa.GEMM_FP32 if args.gemm == "fp32" else gcnsa.GEMM_TF32X3,
                       batch_graph=int(args.graph))
    n_batches = sum(model.n_batches(p) for p in range(w.m))
    loss = torch.zeros(1, device="cuda")
    sampler = ClockSampler(0)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        model.epoch(loss.data_ptr())
    torch.cuda.synchronize()
    n0 = gcnsa.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        model.epoch(loss.data_ptr())
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    launches = gcnsa.launch_count() - n0
    final_loss = loss.item()
    model.profile(True)
    ev0.record()
    model.epoch(loss.data_ptr())
    ev1.record()
    torch.cuda.synchronize()
    ms_prof = ev0.elapsed_time(ev1)
    prof = model.profile_read()
    model.profile(False)
    clocks = sampler.stop()
    # ---- end to end: every epoch uploads each partition's feature rows from pinned host memory
    # (gcnsa_parts_set_features), runs the epoch and reads the loss back ----
    xs = [torch.from_numpy(np.ascontiguousarray(w.x[parts.members(p)])).pin_memory() for p in range(w.m)]
    loss_h = torch.zeros(1).pin_memory()

    def host_epoch():
        for p in range(w.m):
            parts.set_features(p, xs[p].data_ptr())
        model.epoch(loss.data_ptr())
        loss_h.copy_(loss, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    host_epoch()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        host_epoch()
    e2e_s = time.perf_counter() - t0
    h2d = int(sum(x.numel() * 4 for x in xs))
    peak_hbm, peak_bf16, sm_max_mhz, peak_kind = measured_peaks()
    ga, ge = prof["gather"], prof["gemm"]
    gbs = ga["alg_bytes"] / max(ga["ms"] * 1e-3, 1e-12) / 1e9
    line = {"metric": METRIC, "value": args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "variant": "GraphSAGE, mean aggregator (Section 4.1)", "dims": dims,
                       "fanout": list(fanout), "batch": batch, "lr": lr, "partitions": w.m, "batches_per_epoch": n_batches,
                       "ms_per_batch": ms / args.steps / n_batches, "launches_per_batch": launches / args.steps / n_batches,
                       "final_loss": final_loss, "ms_per_step_with_kernel_events": ms_prof,
                       "batch_graph": bool(args.graph),
                       "l2": "the batches of an epoch read every partition's features and CSR (> 2 GB)"},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4},
            "roofline": {"kernel": "sage_concat_mean", "bound": "hbm", "achieved": gbs, "peak": peak_hbm, "unit": "GB/s",
                         "frac": gbs / peak_hbm, "peak_kind": peak_kind + " HBM copy",
                         "traffic": SAGE_TRAFFIC_BYTES.get(w.name),
                         "traffic_note": None if w.name in SAGE_TRAFFIC_BYTES else "no ncu capture of this workload",
                         "alg_bytes_per_launch": ga["alg_bytes"] / max(ga["launches"], 1),
                         "launches": ga["launches"], "avg_launch_ms": ga["ms"] / max(ga["launches"], 1),
                         "share_of_step": ga["ms"] / ms_prof,
                         "note": "source rows are gathered from a partition's feature matrix (125 MB at paper scale, about L2 "
                                 "size); a batch is microsecond-scale work, so launch latency bounds the epoch"},
            "kernels": {k: {"ms_per_step": v["ms"], "launches_per_step": v["launches"],
                            "tflops": v["flops"] / max(v["ms"] * 1e-3, 1e-12) / 1e12} for k, v in prof.items()}}
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = sage_cpu_baseline(w, dims, fanout, batch, lr)
    print(json.dumps(line), flush=True)
    model.close()
    parts.close()


def run_sweep(args):
    """One forward + backward GCN layer (width F -> F) per point; one JSON line
    per point with SpMM and GEMM rates.  Not the headline benchmark."""
    import torch
    from gen import configs
    from paper_2012_04930_b200 import gcnsa
    torch.cuda.set_device(0)
    peak, _, _, peak_kind = measured_peaks()
    pre = configs.sweep_graph(args.sweep, scale=args.scale)
    for m in [int(t) for t in args.sweep_m.split(",")]:
        for f in [int(t) for t in args.sweep_f.split(",")]:
            w = configs.sweep_point(args.sweep, f, m, scale=args.scale, prebuilt=pre)
            env = gcnsa.make_env(0)
            parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], w.m, w.overlap_ppm, w.seed,
                                w.part_mode, w.user_part, w.loss_on_halo)
            model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr,
                                gemm_mode=gcnsa.GEMM_FP32 if args.gemm == "fp32" else gcnsa.GEMM_TF32X3,
                                factored_norm=int(args.factored_norm), loss_rows_only=0, epoch_graph=0)
            infos = [parts.info(p) for p in range(w.m)]
            for _ in range(3):
                model.epoch()
            model.profile(True)
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for _ in range(args.steps):
                model.epoch()
            ev1.record()
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1) / args.steps
            pr = model.profile_read()
            sp, ge = pr["spmm"], pr["gemm"]
            nnz = sum(i.nnz for i in infos)
            rows = sum(i.n for i in infos)
            n_max = max(i.n for i in infos)
            gather_bytes = 2.0 * sp["flops"]                       # 4 F nnz per SpMM, summed
            b_max = sp["alg_bytes"] + gather_bytes - 4.0 * f * rows * 2 * args.steps  # gathers instead of one read
            print(json.dumps({
                "sweep": args.sweep, "width": f, "partitions": m, "factored_norm": bool(args.factored_norm),
                "rows_extended": rows, "nnz_extended": nnz,
                "gathered_matrix_mb": n_max * f * 4 / 1e6, "fits_l2": bool(n_max * f * 4 < 126e6),
                "ms_per_epoch": ms, "spmm_ms": sp["ms"] / args.steps, "gemm_ms": ge["ms"] / args.steps,
                "spmm_alg_gbs": sp["alg_bytes"] / sp["ms"] / 1e6, "spmm_alg_frac_of_hbm": sp["alg_bytes"] / sp["ms"] / 1e6 / peak,
                "spmm_gather_gbs": gather_bytes / sp["ms"] / 1e6, "spmm_bmax_gbs": b_max / sp["ms"] / 1e6,
                "spmm_bmax_frac_of_hbm": b_max / sp["ms"] / 1e6 / peak, "spmm_tflops": sp["flops"] / sp["ms"] / 1e9,
                "gemm_tflops": ge["flops"] / ge["ms"] / 1e9, "peak_gbs": peak, "peak_kind": peak_kind}), flush=True)
            model.close()
            parts.close()


def run_accuracy_study(args):
    """Shape check of the paper's Tables 2-3 on the synthetic `small` workload (not a parity pin): train with M
    range partitions at several overlap thresholds O, evaluate micro-F1 on the held-out vertices of the complete
    graph.  One JSON line per (M, O, aggregation)."""
    import torch
    from gen import configs
    from paper_2012_04930_b200 import gcnsa
    torch.cuda.set_device(0)
    w = configs.small()
    env = gcnsa.make_env(0)
    full = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], 1, 0, w.seed, gcnsa.PART_RANGE)
    test = (1 - w.train_mask).astype(np.uint8)
    for m, o in ((1, 0), (4, 0), (4, 100_000), (4, 250_000), (4, 500_000), (10, 0), (10, 100_000), (10, 250_000),
                 (10, 500_000)):
        parts = gcnsa.Parts(env, w.rowptr, w.col, w.x, w.y, w.train_mask, w.dims[-1], m, o, w.seed, gcnsa.PART_RANGE)
        halo = sum(parts.info(p).n_halo for p in range(m))
        for agg, agg_name in ((gcnsa.AGG_GRAD_AVG, "gradient average"), (gcnsa.AGG_PARAM_AVG, "parameter average")):
            model = gcnsa.Model(env, parts, w.dims, w.w0, w.b0, lr=w.lr, agg_mode=agg, **{**gcnsa.PLAIN, "gemm_mode": gcnsa.GEMM_TF32X3})
            for _ in range(w.epochs):
                model.epoch()
            ev = gcnsa.Model(env, full, w.dims, w.w0, w.b0, **{**gcnsa.PLAIN, "gemm_mode": gcnsa.GEMM_TF32X3})
            ev.copy_params_from(model)
            correct, total, _ = ev.evaluate(full, 0, test)
            print(json.dumps({"workload": w.name, "partitions": m, "overlap_percent": o / 1e4,
                              "overhead_percent_of_n": 100.0 * halo / m / w.n, "aggregation": agg_name,
                              "epochs": w.epochs, "micro_f1": correct / total, "test_vertices": total}), flush=True)
            ev.close()
            model.close()
        parts.close()
    full.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="paper_scale")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm", default="tf32x3", choices=["tf32x3", "fp32"], help="GEMM path of the training step")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="plain launches with per-kernel events inside the timed region (default: the timed region "
                         "replays the recorded epoch, a CUDA graph, and the per-kernel figures come from a second pass)")
    ap.add_argument("--no-factored-norm", dest="factored_norm", action="store_false",
                    help="read the stored A_hat values in every sparse product instead of factoring the normalization out")
    ap.add_argument("--no-cache-ax-leg", dest="cache_ax_leg", action="store_false",
                    help="skip the separately reported run with A_hat X kept across epochs")
    ap.add_argument("--sweep", default=None, choices=["paper", "regular"], help="run the SpMM/GEMM sweep instead")
    ap.add_argument("--sweep-f", default="16,64,128,256,602")
    ap.add_argument("--sweep-m", default="1,5,16")
    ap.add_argument("--accuracy-study", action="store_true", help="micro-F1 vs overlap on the small workload")
    ap.add_argument("--order-window", type=int, default=0,
                    help="rows per window of the processing order (0 = the library's default, -1 = one window)")
    ap.add_argument("--model", default="kw", choices=["kw", "sage"],
                    help="kw: the Kipf-Welling GCN (the headline); sage: the GraphSAGE variant, reported separately")
    args = ap.parse_args()
    if args.accuracy_study:
        run_accuracy_study(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.model == "sage":
        run_sage(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
