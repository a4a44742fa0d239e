#!/usr/bin/env python
"""Benchmark of the fused chunked KL loss (forward + backward over the LM head) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

A step is one kdkl_forward + kdkl_backward over one batch of synthetic input (the paper's
loss-only benchmark shape). Prints ONE JSON line: tokens/s for the whole job, with the
roofline of the dominant kernel (timed live with CUDA events between kernels), an
end-to-end number through the host-buffer entry point, the clocks seen during the timed
region and the fp64 CPU oracle timed on this machine's host cores on a bounded sample.

With N > 1 (launched by torch.distributed.run) every rank runs its own batch of T tokens:
token batches are independent, so there is no data-path collective ("weak" scaling);
torch.distributed is used for the barrier and the max over ranks of the device time.

--impl reference times the CPU oracle (the reference arm for this build: the paper ships no
code to run) on rank 0 and prints the same line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "KL fwd+bwd tokens/s & % of bf16 tensor peak; peak HBM GB vs sequence length"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {}
        for n in dir(nv):
            if n.startswith("nvmlClocksThrottleReason") and isinstance(getattr(nv, n), int):
                names[getattr(nv, n)] = n[len("nvmlClocksThrottleReason"):]
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if bit and (r & bit) == bit and name not in ("None", "All"):
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)

    def summary(self):
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}


def oracle_data(cfg, n_rows: int, dev_tensors=None):
    """The first n_rows tokens of the workload as float64 numpy arrays (prepared once, outside any timing)."""
    import torch
    from paper_2608_03796_b200 import inputs as I
    if dev_tensors is None:
        device = "cuda" if torch.cuda.is_available() else "cpu"
        d = I.make_inputs(cfg, device=device, rows=torch.arange(n_rows, dtype=torch.int64))
    else:
        d = {k: (v if (v is None or k == "weight") else v[:n_rows]) for k, v in dev_tensors.items()}
    out = {"hidden": d["hidden"].cpu().double().numpy(), "weight": d["weight"].cpu().double().numpy(),
           "topk_idx": d["topk_idx"].cpu().numpy(), "topk_val": d["topk_val"].cpu().numpy(),
           "mask": None if d["mask"] is None else d["mask"].cpu().numpy()}
    return out


def oracle_sample(cfg, od):
    """Time the fp64 oracle (forward + gradients) on the prepared sample. Returns (tokens/s, threads, seconds)."""
    from oracle.kdkl_oracle import kdkl_oracle
    n_rows = od["hidden"].shape[0]
    t0 = time.perf_counter()
    kdkl_oracle(od["hidden"], od["weight"], od["topk_idx"], od["topk_val"], tau=cfg.tau, mask=od["mask"],
                want_grads=True)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return n_rows / dt, threads, dt


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_rows = args.ref_rows or 128
    vals = []
    od = oracle_data(cfg, n_rows)
    for i in range(args.warmup + args.steps):
        tps, threads, dt = oracle_sample(cfg, od)
        if i >= args.warmup:
            vals.append((tps, dt))
    tps = sum(v[0] for v in vals) / len(vals)
    ms = 1e3 * sum(v[1] for v in vals) / len(vals)
    sample = f"{n_rows} tokens of {cfg.name} per step, forward + gradients, dense fp64"
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def rank_config(cfg, rank: int):
    """Each rank times its own batch: same shape and generators, seed offset by the rank."""
    import dataclasses
    return dataclasses.replace(cfg, seed=cfg.seed + rank)


def max_over_ranks(value: float, world: int, device) -> float:
    """The slowest rank's time (all-reduce MAX); the job is as slow as its slowest rank."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Aggregate over all ranks: every rank processes tokens_per_rank tokens per step."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def workload_name(cfg):
    return (f"{cfg.name}: T={cfg.T} H={cfg.H} V={cfg.V} K={cfg.K} chunk={cfg.chunk} tau={cfg.tau} "
            f"bf16 hidden/weight, top-K teacher ({cfg.idx_dist} indices)")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="kdkl", choices=["kdkl", "reference"])
    ap.add_argument("--ref-rows", type=int, default=0,
                    help="tokens in the CPU-oracle sample (0: 768 for the cpu_baseline leg, 128 per reference step)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--capture", action="store_true",
                    help="profiler-capture mode: exactly --warmup warm-up steps, no e2e, no CPU baseline, no stage run")
    args = ap.parse_args()

    from paper_2608_03796_b200 import inputs as I
    cfg = I.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_03796_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    import __graft_entry__ as entry
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    B.lib()
    peaks = load_peaks()

    # every rank: its own batch (seed offset by rank), generated on the device
    d = I.make_inputs(rank_config(cfg, rank), device=dev)
    T, H, V, K = cfg.T, cfg.H, cfg.V, cfg.K
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    base_mem = torch.cuda.memory_allocated()
    torch.cuda.empty_cache()                        # idle blocks left by the input generators go back first
    free_before = torch.cuda.mem_get_info()[0]      # driver's view, for a cross-check of the allocator's peak
    op = B.FusedChunkedKL(T, H, V, K, chunk=cfg.chunk, temperature=cfg.tau, device=dev)

    def step():
        op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], loss_mask=d["mask"])
        op.backward(d["hidden"], d["weight"], loss_mask=d["mask"])

    n_warm = args.warmup if args.capture else max(args.warmup, 3)
    for _ in range(n_warm):
        step()
    torch.cuda.synchronize()
    code, detail = op.status()
    if code != 0:
        raise SystemExit(f"device status {code} {detail}")
    launches_per_step = op.launches

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    with ClockSampler(local_rank) as clk:
        ev0.record()
        for i in range(args.steps):
            step()
            step_ev[i].record()
        ev1.record()
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    marks = [ev0] + step_ev
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps))
    ms_median, ms_min = per_step[len(per_step) // 2], per_step[0]
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    loss_val = float(op.loss.item())
    peak_mem = torch.cuda.max_memory_allocated()
    driver_delta = free_before - torch.cuda.mem_get_info()[0]   # what the op's buffers took from the device
    ws_bytes = op.workspace.numel()

    # peak memory versus sequence length for this shape, from the allocation sizes alone (inputs + outputs +
    # workspace; the measured sweep is in profiles/): the vocabulary-sized part does not grow with T
    def allocation_gb(tokens):
        mask_bytes = tokens if d["mask"] is not None else 0
        fixed = V * H * 2 + V * H * 4 + 4
        per_t = tokens * (H * 2 + K * 8 + H * 2) + mask_bytes
        return (fixed + per_t + B.kdkl_workspace_bytes(tokens, H, V, K, cfg.chunk)) / 1e9
    mem_model = {str(t): round(allocation_gb(t), 3) for t in (4096, 32768, 65536, 131072, 262144)}

    # the single-pass step (kdkl_forward_backward: three projections instead of four, same memory, same outputs up
    # to one more bf16 rounding inside G), timed like the headline; reported beside it, not instead of it
    def step1():
        op.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], loss_mask=d["mask"])
    for _ in range(n_warm):
        step1()
    sp0, sp1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sp0.record()
    for _ in range(args.steps):
        step1()
    sp1.record()
    barrier()
    sp_ms = max_over_ranks(sp0.elapsed_time(sp1), world, dev) / args.steps
    assert op.status()[0] == 0 and abs(float(op.loss.item()) - loss_val) <= 1e-6 * abs(loss_val)
    sp_acc = {}
    n_sp_prof = 1 if args.capture else 3
    for _ in range(n_sp_prof):
        for k, (ms, n) in B.kdkl_profile_single_pass(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"],
                                                      op.workspace, op.loss, op.dhidden, op.dweight,
                                                      loss_mask=d["mask"], chunk=cfg.chunk,
                                                      temperature=cfg.tau).items():
            a = sp_acc.setdefault(k, [0.0, 0])
            a[0] += ms
            a[1] += n
    sp_stages = {k: {"ms_per_step": v[0] / n_sp_prof, "launches_per_step": v[1] // n_sp_prof,
                     "ms_per_launch": v[0] / v[1]} for k, v in sp_acc.items()}
    single_pass = {"ms_per_step": sp_ms, "stages": sp_stages, "tokens_per_s": whole_job_tokens_per_s(T, world, sp_ms),
                   "flops_executed": 0.75 * cfg.flops, "tflops_executed_per_gpu": 0.75 * cfg.flops / (sp_ms * 1e-3) / 1e12,
                   "launches_per_step": op.launches,
                   "what": "forward + backward in one call without the second projection (6*T*H*V flops)"}

    # per-kernel times, live, with an event between kernels (a separate short run)
    stage_acc = {}
    n_prof = 1 if args.capture else 3
    for _ in range(n_prof):
        st = B.kdkl_profile_stages(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], op.workspace, op.loss,
                                   op.dhidden, op.dweight, loss_mask=d["mask"], chunk=cfg.chunk, temperature=cfg.tau)
        for k, (ms, n) in st.items():
            a = stage_acc.setdefault(k, [0.0, 0])
            a[0] += ms
            a[1] += n
    stages = {k: {"ms_per_step": v[0] / n_prof, "launches_per_step": v[1] // n_prof,
                  "ms_per_launch": (v[0] / v[1] if v[1] else 0.0)} for k, v in stage_acc.items()}
    gemm_stages = ["fwd_gemm_lse", "bwd_gemm_dlogits", "dhidden_gemm", "dweight_gemm"]
    dom = max(gemm_stages, key=lambda k: stages[k]["ms_per_step"])
    # DRAM bytes per launch from one ncu capture at chunk=4096, H=4096, V=131072 (read + write); null elsewhere
    measured_traffic = {"fwd_gemm_lse": 1118791680 + 25831168, "bwd_gemm_dlogits": 1249679104 + 1053059584,
                        "dhidden_gemm": 5458027520 + 117394432, "dweight_gemm": 1551928576 + 2114988800}
    C = min(cfg.chunk, T)
    traffic = measured_traffic[dom] if (C, H, V) == (4096, 4096, 131072) else None
    flops_per_launch = 2.0 * C * H * V             # each of the four GEMMs: 2 * chunk * H * V per launch
    dom_tflops = flops_per_launch / (stages[dom]["ms_per_launch"] * 1e-3) / 1e12
    long_step = ms_total > 1000.0
    peak_key = "bf16_tflops_sustained" if long_step else "bf16_tflops"
    peak = float(peaks.get(peak_key, FALLBACK_PEAKS[peak_key]))
    for k in gemm_stages:
        stages[k]["tflops"] = flops_per_launch / (stages[k]["ms_per_launch"] * 1e-3) / 1e12

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e and not args.capture:
        opt = None
        arena = torch.empty(B.kdkl_host_arena_bytes(T, H, V, K, cfg.chunk), dtype=torch.uint8, device=dev)
        hh = {k: (v.cpu().pin_memory() if v is not None else None) for k, v in d.items()}
        loss_h = torch.zeros(1, dtype=torch.float32).pin_memory()
        dh_h = torch.empty(T, H, dtype=torch.bfloat16).pin_memory()
        dw_h = torch.empty(V, H, dtype=torch.float32).pin_memory()

        def e2e_step():
            B.kdkl_forward_backward_host(hh["hidden"], hh["weight"], hh["topk_idx"], hh["topk_val"], arena, loss_h,
                                         dh_h, dw_h, loss_mask=hh["mask"], chunk=cfg.chunk, temperature=cfg.tau,
                                         opt=opt)
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e_ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0)) / args.e2e_steps
        e_ms = max_over_ranks(e_ms, world, dev)
        h2d = sum(v.numel() * v.element_size() for v in hh.values() if v is not None)
        d2h = 4 + dh_h.numel() * 2 + dw_h.numel() * 4
        assert abs(float(loss_h.item()) - loss_val) <= 1e-5 * abs(loss_val)
        e2e = {"value": whole_job_tokens_per_s(T, world, e_ms), "unit": "tokens/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "what": "every input (hidden, weight, teacher record, mask) from pinned host memory and loss, dHidden, "
                       "dWeight back to the host each step: bound by the host link"}
        del arena

    # the HBM-bound companion op (hidden-state feature loss, one pass: 2 reads + 1 write of [T,H] bf16), timed at
    # 32768 tokens so that its 6*T*H bytes are several times the L2 whatever T the main workload has
    feature = None
    if rank == 0:
        fT = 32768
        fcfg = I.Config("feature", T=fT, H=H, V=V, K=K, chunk=cfg.chunk)
        fs, fr = I.hidden(fcfg, device=dev), I.teacher_hidden(fcfg, device=dev)
        fws = torch.empty(B.kdkl_feature_loss_workspace_bytes(fT), dtype=torch.uint8, device=dev)
        fl, fd = torch.zeros(1, device=dev), torch.empty_like(fs)
        feature = {"T": fT, "H": H, "algorithmic_bytes": 6 * fT * H,
                   "hbm_peak_GBps": float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))}
        for kind, kname in ((B.FEATURE_MSE, "mse"), (B.FEATURE_COSINE, "cosine")):
            for _ in range(3):
                B.kdkl_feature_loss(fs, fr, fws, fl, kind=kind, dstudent=fd)
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record()
            f_iters = 2 if args.capture else 20
            for _ in range(f_iters):
                B.kdkl_feature_loss(fs, fr, fws, fl, kind=kind, dstudent=fd)
            f1.record()
            torch.cuda.synchronize()
            f_ms = f0.elapsed_time(f1) / f_iters
            gbps = 6 * fT * H / (f_ms * 1e-3) / 1e9
            feature[kname] = {"ms": f_ms, "GBps": gbps, "frac_of_hbm_copy": gbps / feature["hbm_peak_GBps"],
                              "loss": float(fl.item())}
        del fs, fr, fd, fws

    # the step as the offline pipeline feeds it: only the batch's cached teacher record (and mask) comes from the
    # host every step; hidden states, weight and gradients stay on the device, as in a training loop
    e2e_record = None
    if not args.no_e2e and not args.capture:
        staging = torch.empty(B.kdkl_record_staging_bytes(T, K), dtype=torch.uint8, device=dev)
        rec = {k: (d[k].cpu().pin_memory() if d[k] is not None else None) for k in ("topk_idx", "topk_val", "mask")}
        loss_h2 = torch.zeros(1, dtype=torch.float32).pin_memory()

        def record_step():
            B.kdkl_step_host_record(d["hidden"], d["weight"], rec["topk_idx"], rec["topk_val"], staging, op.workspace,
                                    loss_h2, op.dhidden, op.dweight, loss_mask_host=rec["mask"], chunk=cfg.chunk,
                                    temperature=cfg.tau)
        record_step()
        barrier()
        t0 = time.perf_counter()
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(args.steps):
            record_step()
        r1.record()
        barrier()
        r_ms = max(r0.elapsed_time(r1), 1e3 * (time.perf_counter() - t0)) / args.steps
        r_ms = max_over_ranks(r_ms, world, dev)
        assert abs(float(loss_h2.item()) - loss_val) <= 1e-5 * abs(loss_val)
        e2e_record = {"value": whole_job_tokens_per_s(T, world, r_ms), "unit": "tokens/s", "ms_per_step": r_ms,
                      "h2d_bytes_per_step": sum(v.numel() * v.element_size() for v in rec.values() if v is not None),
                      "d2h_bytes_per_step": 4, "steps": args.steps,
                      "what": "teacher record (+ mask) from pinned host memory each step; hidden, weight, gradients resident"}
        del staging

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline and not args.capture and world == 1:
        tps, threads, dt = oracle_sample(cfg, oracle_data(cfg, args.ref_rows or 768, d))
        cpu_baseline = {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                        "sample": f"{args.ref_rows or 768} tokens of {cfg.name}, forward + gradients, dense fp64, {dt:.1f} s"}

    tokens_per_s = whole_job_tokens_per_s(T, world, ms_step)
    step_tflops = cfg.flops / (ms_step * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": tokens_per_s, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": ms_step, "ms_per_step_median": ms_median, "ms_per_step_min": ms_min,
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "l2": f"inputs larger than L2 (weight {V * H * 2 / 2**20:.0f} MiB, dW {V * H * 4 / 2**20:.0f} MiB per step)",
                   "per_rank_tokens": T, "parallelism": f"independent batches x{world}"},
        "tflops_per_gpu": step_tflops,
        "frac_of_bf16_burst_peak": step_tflops / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])),
        "frac_of_bf16_sustained_peak": step_tflops / float(peaks.get("bf16_tflops_sustained",
                                                                     FALLBACK_PEAKS["bf16_tflops_sustained"])),
        "peaks": peaks.get("_source"),
        "peak_mem_gb": peak_mem / 1e9, "workspace_gb": ws_bytes / 1e9, "input_mem_gb": base_mem / 1e9,
        "op_mem_gb_allocator": (peak_mem - base_mem) / 1e9, "op_mem_gb_driver": driver_delta / 1e9,
        "peak_mem_gb_vs_tokens": mem_model,
        "loss": loss_val,
        "clocks": clk.summary(),
        "gpu_launches": launches_per_step * args.steps,
        "single_pass": single_pass,
        "e2e": e2e,
        "e2e_record_from_host": e2e_record,
        "roofline": {"bound": "tensor", "kernel": dom, "achieved": dom_tflops, "peak": peak, "unit": "TFLOP/s",
                     "frac": dom_tflops / peak, "peak_kind": f"{peak_key} ({peaks.get('_source')})",
                     "traffic": traffic, "ms_per_launch": stages[dom]["ms_per_launch"],
                     "flops_per_launch": flops_per_launch},
        "stages": stages,
        "feature_loss": feature,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
