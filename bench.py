#!/usr/bin/env python
"""Benchmark of the verify step on the headline workload (B=256, K=3, V=151936, bf16).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" = one bebop_verify call over one batch (every row of the hot path:
temperature softmax of both logit rows, accept scan, TV, residual / bonus draw,
compaction).  Prints ONE JSON line (rank 0).  `value` is positions/s with the
inputs resident in HBM; `e2e` is the same metric through the same C-ABI call but
with the inputs in pinned host memory and the results read back, copies inside
the timed region.  `--impl reference` times the fp64 CPU oracle on a bounded
sample of the same workload instead (host cores only).
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verify positions/s at V=151936 bf16 (B=256,K=3); HBM GB/s as % of peak"
WORKLOAD = "headline"
FALLBACK_HBM_GBS = 6650.0
NORTH_STAR_PEAK_GBS = 8000.0


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


KERNEL_OF_PATH = {0: "k_pipe"}


def ncu_traffic(kernel):
    """DRAM bytes per launch of the dominant kernel on the headline workload, from the committed ncu summary."""
    try:
        for ln in open(os.path.join(ROOT, "profiles", kernel + "_headline.md")):
            if ln.startswith("traffic_bytes_per_launch"):
                return int(ln.split("=")[1].split()[0])
    except Exception:
        pass
    return None


def roofline(alg_bytes, kern_ms, peak, peak_kind, headline, kernel, timed_launches):
    """HBM roofline of the dominant kernel: algorithmic bytes of one launch over its CUDA-event
    duration measured inside the timed region."""
    gbs = alg_bytes / (kern_ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
            "traffic": ncu_traffic(kernel) if headline else None, "peak_kind": "of " + peak_kind,
            "kernel": kernel, "kernel_ms": kern_ms, "kernel_launches_timed": timed_launches,
            "algorithmic_bytes_per_launch": alg_bytes,
            "pct_of_8tbs": 100.0 * gbs / NORTH_STAR_PEAK_GBS}


class ClockSampler:
    """Polls SM clock, power and throttle reasons through NVML (read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, uuid=None):
        self.samples, self.max_mhz, self.ok = [], None, False
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-%s" % uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                mhz = self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)
                rs = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                pw = self.nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), mhz, rs, pw))
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.ok:
            self.t.start()

    def stop(self):
        self._stop.set()
        if self.ok:
            self.t.join(timeout=1.0)

    def summary(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        where = "timed region"
        if not inside:
            inside, where = self.samples, "warm-up and timed region (timed region shorter than one sample)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        mhz = sorted(s[1] for s in inside)
        bits = 0
        for s in inside:
            bits |= s[2]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz,
                "reasons": sorted(n for b, n in self.REASONS.items() if bits & b),
                "power_w_max": round(max(s[3] for s in inside), 1), "samples": len(inside),
                "window": where}


def oracle_sample_rate(x_cpu, nseq, nthreads=0):
    """positions/s of the oracle on the first nseq sequences of a CPU-resident input set."""
    import oracle
    sl = slice(0, nseq)
    tgt = x_cpu["target"][sl].float().numpy()
    drf = x_cpu["draft"][sl].float().numpy()
    t0 = time.perf_counter()
    oracle.verify(tgt, drf, x_cpu["draft_tokens"][sl].numpy(), x_cpu["u_accept"][sl].numpy(),
                  x_cpu["u_final"][sl].numpy(), temperature_all=x_cpu["temperature_all"], nthreads=nthreads)
    dt = time.perf_counter() - t0
    return nseq * x_cpu["cfg"].K / dt, dt


def run_reference(args):
    """The reference arm: the oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import bebop_gen as G
    import oracle
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    cores = oracle.num_threads()
    nseq = max(2 * cores, 8)
    cfg = G.get_config(WORKLOAD, B=nseq)
    x = G.make_inputs(cfg, "cpu")
    for _ in range(warmup):
        oracle_sample_rate(x, nseq)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_rate(x, nseq)
    dt = (time.perf_counter() - t0) / steps
    val = nseq * cfg.K / dt
    sample = "%d of the workload's 256 sequences per step (same recipe, seed %d)" % (nseq, cfg.seed)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "positions/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "headline: B=256 K=3 V=151936 bf16 logits, tau=1 (oracle sample)"},
        "cpu_baseline": {"value": val, "unit": "positions/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "positions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    import bebop_gen as G
    import paper_2606_12370_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    steps = args.steps if args.steps is not None else 2000
    warmup = max(3, args.warmup if args.warmup is not None else 20)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    P.load_library()
    P.bebop_debug_force_general_path(args.path)

    # weak scaling: every rank verifies its own batch of the headline shape (seed offset by rank)
    cfg = G.get_config(WORKLOAD)
    over = {"B": args.batch} if args.batch else {}
    cfg = G.get_config(WORKLOAD, seed=cfg.seed + 1000 * rank, **over)
    x = G.make_inputs(cfg, dev)
    B, K, V = cfg.B, cfg.K, cfg.V
    es = 2 if cfg.dtype == "bf16" else 4
    rows = G.rows_read(cfg, x["draft_len"])
    alg_bytes = rows * V * es
    positions = B * K
    ws = torch.empty(P.bebop_workspace_bytes(B, K, V, P.BEBOP_BF16), dtype=torch.uint8, device=dev)
    out = dict(accept_len=torch.empty(B, dtype=torch.int32, device=dev),
               out_tokens=torch.empty((B, K + 1), dtype=torch.int32, device=dev),
               tv=torch.empty((B, K), dtype=torch.float32, device=dev),
               p_draft=torch.empty((B, K), dtype=torch.float32, device=dev),
               q_draft=torch.empty((B, K), dtype=torch.float32, device=dev),
               row_status=torch.empty(B, dtype=torch.int32, device=dev))

    def step(inp=x):
        return P.bebop_verify(inp["target"], inp["draft"], inp["draft_tokens"], inp["u_accept"], inp["u_final"],
                              draft_len=inp["draft_len"], temperature=inp["temperature"],
                              temperature_all=inp["temperature_all"], out=out, workspace=ws)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local, getattr(torch.cuda.get_device_properties(dev), "uuid", None))
    sampler.start()
    for _ in range(warmup):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # events around the dominant kernel (k_pipe) inside the timed region: the library records
    # them on the launching stream.  Every fourth step at most, and at most 32 steps, carry a pair: an
    # event between the main kernel and its dependent kernels costs that step about 5 us
    stride = max(4, (steps + 31) // 32)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range((steps + stride - 1) // stride)]
    for a_, b_ in pairs:            # a torch event owns a CUDA event only after its first record
        a_.record(); b_.record()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for i in range(steps):
        if i % stride == 0:
            P.bebop_debug_set_timing_events(*pairs[i // stride])
        else:
            P.bebop_debug_set_timing_events(None, None)
        step()
    e1.record()
    barrier()
    t1 = time.perf_counter()
    P.bebop_debug_set_timing_events(None, None)
    ms = e0.elapsed_time(e1)
    kern_ms = [a_.elapsed_time(b_) for a_, b_ in pairs]
    kern_ms = sum(kern_ms) / len(kern_ms)
    clocks = sampler.summary(t0, t1)
    launches_per_call = 6 if args.path == 1 else 2      # main kernel, fp64 re-draw kernel | 6 general kernels

    # the same call without a TV output (the second sweep then reads only the rows a token is drawn from): not the
    # headline, which emits TV; reported beside it
    notv_steps = max(1, min(steps, 200))
    out_notv = {k: v for k, v in out.items() if k != "tv"}

    def step_notv():
        return P.bebop_verify(x["target"], x["draft"], x["draft_tokens"], x["u_accept"], x["u_final"],
                              draft_len=x["draft_len"], temperature=x["temperature"],
                              temperature_all=x["temperature_all"], out=out_notv, workspace=ws, want_tv=False)

    for _ in range(3):
        step_notv()
    barrier()
    n0, n1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0.record()
    for _ in range(notv_steps):
        step_notv()
    n1.record()
    barrier()
    notv_ms = n0.elapsed_time(n1) / notv_steps

    # the two other entry points on the same logits (reported beside the headline, not part of it)
    def timed(fn, n):
        for _ in range(3):
            fn()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(n):
            fn()
        a1.record()
        barrier()
        return a0.elapsed_time(a1) / n

    other_steps = max(1, min(steps, 50))
    tv_t = x["target"][:, :K].reshape(B * K, V)
    tv_d = x["draft"].reshape(B * K, V)
    tv_ms = timed(lambda: P.bebop_tv(tv_t, tv_d, temperature_all=1.0), other_steps)
    gr_ms = timed(lambda: P.bebop_greedy_verify(x["target"], x["draft_tokens"]), other_steps)

    # end to end: pinned host inputs -> device, same C-ABI call, results back to the host
    e2e_steps = 0 if args.no_e2e else max(1, min(steps, 10))
    host = {k: x[k].cpu().pin_memory() for k in ("target", "draft", "draft_tokens", "u_accept", "u_final")}
    dev_in = {k: torch.empty_like(x[k]) for k in host}
    host_out = {k: torch.empty(out[k].shape, dtype=out[k].dtype).pin_memory() for k in ("accept_len", "out_tokens", "tv")}
    staged = dict(x)
    staged.update(dev_in)

    def e2e_step():
        for k in host:
            dev_in[k].copy_(host[k], non_blocking=True)
        step(staged)
        for k in host_out:
            host_out[k].copy_(out[k], non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for _ in range(2 if e2e_steps else 0):
        e2e_step()
    barrier()
    w0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = (time.perf_counter() - w0) / max(e2e_steps, 1) if e2e_steps else float("inf")
    h2d = sum(host[k].numel() * host[k].element_size() for k in host)
    d2h = sum(host_out[k].numel() * host_out[k].element_size() for k in host_out)

    # max over ranks
    from paper_2606_12370_b200.shard import max_over_ranks
    ms, e2e_s, notv_ms, tv_ms, gr_ms = max_over_ranks([ms, e2e_s, notv_ms, tv_ms, gr_ms], dist, dev)
    sampler.stop()

    if rank == 0:
        ms_step = ms / steps
        peak, peak_kind = measured_peak()
        gbs = alg_bytes / (ms_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": world * positions / (ms_step * 1e-3), "unit": "positions/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "headline: B=%d K=3 V=151936 bf16 logits, tau=1, N(0,3^2)+8 Zipf peaks, "
                                   "draft=target+N(0,1), per GPU" % B,
                       "global_batch": world * B, "positions_per_step": world * positions,
                       "l2": "inputs (%.0f MB per GPU) larger than the 126 MB L2; no flush" % (alg_bytes / 1e6),
                       "draw": "fp32 inverse CDF kept when it clears the error bound, else re-drawn in fp64",
                       "parallelism": "dp%d" % world},
            "clocks": clocks,
            "e2e": {"value": world * positions / e2e_s, "unit": "positions/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_s * 1e3},
            "gpu_launches": steps * launches_per_call,
            "other_entry_points": {
                "bebop_tv": {"ms_per_call": tv_ms, "row_pairs": world * B * K, "steps": other_steps,
                             "algorithmic_gbs": world * B * K * 2 * V * es / (tv_ms * 1e-3) / 1e9},
                "bebop_greedy_verify": {"ms_per_call": gr_ms, "steps": other_steps,
                                        "algorithmic_gbs": world * B * (K + 1) * V * es / (gr_ms * 1e-3) / 1e9}},
            "without_tv": {"value": world * positions / (notv_ms * 1e-3), "unit": "positions/s", "ms_per_step": notv_ms,
                           "steps": notv_steps, "note": "same call with tv = NULL; not the headline"},
            "hbm_gbs": gbs, "hbm_pct_of_8tbs": 100.0 * gbs / NORTH_STAR_PEAK_GBS,
            "roofline": roofline(alg_bytes, kern_ms, peak, peak_kind, B == 256, KERNEL_OF_PATH.get(args.path, "general kernels"), len(pairs)),
        }
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            cores = oracle.num_threads()
            nseq = min(64, B)
            xc = {k: (v[:nseq].cpu() if hasattr(v, "cpu") else v) for k, v in x.items()}
            oracle_sample_rate(xc, min(8, nseq))
            reps, spent = 0, 0.0
            while spent < 10.0 and reps < 1000:
                _, dt = oracle_sample_rate(xc, nseq)
                spent += dt
                reps += 1
            line["cpu_baseline"] = {"value": reps * nseq * K / spent, "unit": "positions/s", "cores": cores,
                                    "kind": "oracle",
                                    "sample": "first %d of the step's %d sequences, %d passes, %.1f s" % (nseq, B, reps, spent)}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0,
                    help="profiling aid: sequences per GPU instead of the workload's 256 (not a bench line)")
    ap.add_argument("--no-e2e", action="store_true", help="profiling aid: skip the host-buffer leg")
    ap.add_argument("--path", type=int, default=0, help="profiling aid: kernel path (0 default: pipelined kernel, 1 general kernels)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
