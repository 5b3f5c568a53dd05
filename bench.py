#!/usr/bin/env python
"""Benchmark of the verify step on the headline workload (B=256, K=3, V=151936, bf16).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--scaling weak|strong]

One "step" = one bebop_verify call over one batch (every row of the hot path:
temperature softmax of both logit rows, accept scan, TV, residual / bonus draw,
compaction).  Prints ONE JSON line (rank 0).  `value` is positions/s with the
inputs resident in HBM; `e2e` is the same metric through the same C-ABI call but
with the inputs in pinned host memory and the results read back, copies inside
the timed region.  Beside the headline the line carries the five benchmark
configurations (`configs`: time per call, bandwidth, and a sampled comparison
with the oracle outside the timed region).  `--impl reference` times the fp64 CPU
oracle on the same workload instead (host cores only).

With --gpus N > 1 and no launcher (WORLD_SIZE unset) the script starts the N ranks
itself, one per GPU.  Sequences are independent, so the ranks share nothing on the
data path: `--scaling weak` (default) gives every rank its own headline batch,
`--scaling strong` cuts the full rollout batch (config 5, ragged) into contiguous
blocks balanced by the rows each rank has to read.
"""
import argparse
import json
import math
import os
import socket
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verify positions/s at V=151936 bf16 (B=256,K=3); HBM GB/s as % of peak"
WORKLOAD = "headline"
WORKLOAD_STR = "headline: B=256 K=3 V=151936 bf16 logits, tau=1, N(0,3^2)+8 Zipf peaks, draft=target+N(0,1), per GPU"
STRONG_WORKLOAD = "full_batch"
FALLBACK_HBM_GBS = 6650.0
NORTH_STAR_PEAK_GBS = 8000.0
L2_BYTES = 126e6


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


KERNEL_NAME = {1: "general kernels", 2: "k_pipe", 3: "k_fuse"}      # by bebop_debug_last_kernel()


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


# ------------------------------------------------------------------------------- workload of a rank
def slice_inputs(x, begin, end):
    """Sequences [begin, end) of a generated input set (views, nothing is copied)."""
    out = dict(x)
    for k in ("target", "draft", "draft_tokens", "u_accept", "u_final", "draft_len", "temperature"):
        if x.get(k) is not None:
            out[k] = x[k][begin:end]
    return out


def rank_workload(rank, world, scaling, device, overrides=None, config=None):
    """What rank `rank` of `world` verifies.  weak: its own batch of the headline shape (seed offset by the rank).
    strong: its contiguous block of the one full rollout batch (config 5), cut so that every rank reads about the same
    number of logit rows.  Returns the rank's inputs and the sizes the metric needs."""
    import bebop_gen as G
    from paper_2606_12370_b200.shard import shard_range
    over = dict(overrides or {})
    if scaling == "strong":
        cfg = G.get_config(config or STRONG_WORKLOAD, **over)
        full = G.make_inputs(cfg, device)                           # same seed on every rank: the same batch
        lens = None if full["draft_len"] is None else [int(v) for v in full["draft_len"].cpu()]
        begin, end = shard_range(cfg.B, rank, world, lens)
        x = slice_inputs(full, begin, end)
    else:
        base = G.get_config(config or WORKLOAD)
        cfg = G.get_config(config or WORKLOAD, seed=base.seed + 1000 * rank, **over)
        x = G.make_inputs(cfg, device)
        begin, end = 0, cfg.B
    n = end - begin
    dl = x["draft_len"]
    positions = n * cfg.K if dl is None else int(dl.sum().item())
    rows = n * (2 * cfg.K + 1) if dl is None else int((2 * dl.to("cpu").long() + 1).sum().item())
    es = 2 if cfg.dtype == "bf16" else 4
    return dict(x=x, cfg=cfg, begin=begin, end=end, nseq=n, positions=positions, rows=rows,
                alg_bytes=rows * cfg.V * es)


def oracle_rate(x_cpu, nthreads=0):
    """positions/s of the oracle on a CPU-resident input set (all its sequences), and the seconds it took."""
    import oracle
    cfg = x_cpu["cfg"]
    tgt = x_cpu["target"].float().numpy()
    drf = x_cpu["draft"].float().numpy()
    dl = None if x_cpu["draft_len"] is None else x_cpu["draft_len"].numpy()
    tp = None if x_cpu["temperature"] is None else x_cpu["temperature"].numpy()
    t0 = time.perf_counter()
    oracle.verify(tgt, drf, x_cpu["draft_tokens"].numpy(), x_cpu["u_accept"].numpy(), x_cpu["u_final"].numpy(),
                  draft_len=dl, temperature=tp, temperature_all=x_cpu["temperature_all"], nthreads=nthreads)
    dt = time.perf_counter() - t0
    n = tgt.shape[0]
    return (n * cfg.K if dl is None else int(dl.sum())) / dt, dt


def run_reference(args):
    """The reference arm: the oracle, as it stands, on the host cores, on the whole headline batch per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import bebop_gen as G
    import oracle
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    steps, warmup = min(steps, 40), min(warmup, 5)          # a step is a quarter of a second on 16 cores
    cores = oracle.num_threads()
    cfg = G.get_config(WORKLOAD)
    x = G.make_inputs(cfg, "cpu")
    for _ in range(warmup):
        oracle_rate(x)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_rate(x)
    dt = (time.perf_counter() - t0) / steps
    val = cfg.B * cfg.K / dt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "positions/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_STR, "global_batch": cfg.B, "positions_per_step": cfg.B * cfg.K,
                   "parallelism": "host cores"},
        "cpu_baseline": {"value": val, "unit": "positions/s", "cores": cores, "kind": "oracle",
                         "sample": "all %d sequences of the workload per step (seed %d)" % (cfg.B, cfg.seed)},
        "e2e": {"value": val, "unit": "positions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------- timing helpers
def per_call_ms(torch, fns, n, barrier):
    """n calls, cycling through `fns`, an event pair around each: the list of per-call milliseconds."""
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    barrier()
    for i, (a, b) in enumerate(pairs):
        a.record()
        fns[i % len(fns)]()
        b.record()
    barrier()
    return [a.elapsed_time(b) for a, b in pairs]


def stats(ms):
    s = sorted(ms)
    return {"mean": sum(s) / len(s), "median": s[len(s) // 2], "best": s[0], "calls": len(s)}


def checksums(G, x):
    return {k: G.checksum(x[k]) for k in ("target", "draft", "draft_tokens", "u_accept", "u_final", "draft_len", "temperature")
            if x.get(k) is not None}


def config_line(torch, P, G, name, dev, barrier, calls):
    """One of the five benchmark configurations: per-call time over inputs rotated through distinct buffers (so that the
    working set is at least four times the L2), and a comparison with the oracle on a sample, outside the timed region."""
    import numpy as np
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    cfg = G.get_config(name)
    x = G.make_inputs(cfg, dev)
    B, K, V = cfg.B, cfg.K, cfg.V
    es = 2 if cfg.dtype == "bf16" else 4
    dt = P.BEBOP_BF16 if cfg.dtype == "bf16" else P.BEBOP_F32
    rows = G.rows_read(cfg, x["draft_len"])
    alg = rows * V * es
    positions = B * K if x["draft_len"] is None else int(x["draft_len"].sum().item())
    nrot = max(1, min(int(math.ceil(4 * L2_BYTES / alg)), 8192))
    sets = [x]
    for _ in range(nrot - 1):                       # the same values at other addresses
        c = dict(x); c["target"] = x["target"].clone(); c["draft"] = x["draft"].clone()
        sets.append(c)
    ws = torch.empty(P.bebop_workspace_bytes(B, K, V, dt), dtype=torch.uint8, device=dev)
    out = dict(accept_len=torch.empty(B, dtype=torch.int32, device=dev),
               out_tokens=torch.empty((B, K + 1), dtype=torch.int32, device=dev),
               tv=torch.empty((B, K), dtype=torch.float32, device=dev),
               p_draft=torch.empty((B, K), dtype=torch.float32, device=dev),
               q_draft=torch.empty((B, K), dtype=torch.float32, device=dev),
               row_status=torch.empty(B, dtype=torch.int32, device=dev))

    def call(inp):
        return lambda: P.bebop_verify(inp["target"], inp["draft"], inp["draft_tokens"], inp["u_accept"], inp["u_final"],
                                      draft_len=inp["draft_len"], temperature=inp["temperature"],
                                      temperature_all=inp["temperature_all"], out=out, workspace=ws)
    fns = [call(s) for s in sets]
    for f in fns[:3] + fns[:1]:
        f()
    st = stats(per_call_ms(torch, fns, min(max(calls, nrot), 5000), barrier))     # every buffer is visited at least once
    fns[0]()
    torch.cuda.synchronize()
    # sampled comparison with the oracle
    idx = np.unique(np.linspace(0, B - 1, min(B, 16)).astype(np.int64))
    sel = torch.as_tensor(idx, device=dev)
    pick = lambda t: None if t is None else t[sel].cpu().numpy()
    ref = oracle.verify(x["target"][sel].float().cpu().numpy(), x["draft"][sel].float().cpu().numpy(), pick(x["draft_tokens"]),
                        pick(x["u_accept"]), pick(x["u_final"]), draft_len=pick(x["draft_len"]),
                        temperature=pick(x["temperature"]), temperature_all=x["temperature_all"])
    got_len, got_tok = out["accept_len"][sel].cpu().numpy(), out["out_tokens"][sel].cpu().numpy()
    differ = (got_len != ref["accept_len"]) | (got_tok != ref["out_tokens"]).any(axis=1)
    line = {"shape": "B=%d K=%d V=%d %s%s" % (B, K, V, cfg.dtype, " ragged" if cfg.ragged else ""),
            "kernel": KERNEL_NAME.get(P.bebop_debug_last_kernel()),
            "ms_per_call": st, "positions_per_s": positions / (st["mean"] * 1e-3),
            "algorithmic_bytes": alg, "algorithmic_gbs": alg / (st["mean"] * 1e-3) / 1e9,
            "pct_of_8tbs": 100.0 * alg / (st["mean"] * 1e-3) / 1e9 / NORTH_STAR_PEAK_GBS,
            "buffers_rotated": nrot, "working_set_mb": nrot * alg / 1e6,
            "parity_sample": {"sequences": int(len(idx)), "flagged": int(ref["flagged"].sum()),
                              "mismatch_unflagged": int((differ & ~ref["flagged"]).sum()),
                              "tv_max_err": float(np.abs(out["tv"][sel].cpu().numpy() - ref["tv"]).max())},
            "mean_accept_len": float(out["accept_len"].float().mean().item()),
            "checksums": checksums(G, x)}
    if name == "high_entropy":
        # the same shape in the greedy-draft mode: drafts are argmax q, acceptance is x = argmax p
        del sets, fns
        gx = G.make_inputs(cfg, dev, draft_mode="argmax")
        gsets = [gx] + [dict(gx, target=gx["target"].clone()) for _ in range(max(0, int(math.ceil(4 * L2_BYTES / (B * (K + 1) * V * es))) - 1))]
        gout = {}

        def gcall(inp):
            def f():
                gout.update(P.bebop_greedy_verify(inp["target"], inp["draft_tokens"], workspace=ws))
            return f
        gf = [gcall(s) for s in gsets]
        for f in gf[:1] * 3:
            f()
        gst = stats(per_call_ms(torch, gf, calls, barrier))
        gf[0]()
        torch.cuda.synchronize()
        gref = oracle.greedy_verify(gx["target"][sel].float().cpu().numpy(), gx["draft_tokens"][sel].cpu().numpy())
        gdiff = (gout["accept_len"][sel].cpu().numpy() != gref["accept_len"]) | \
                (gout["out_tokens"][sel].cpu().numpy() != gref["out_tokens"]).any(axis=1)
        galg = B * (K + 1) * V * es
        line["greedy_mode"] = {"ms_per_call": gst, "algorithmic_gbs": galg / (gst["mean"] * 1e-3) / 1e9,
                               "pct_of_8tbs": 100.0 * galg / (gst["mean"] * 1e-3) / 1e9 / NORTH_STAR_PEAK_GBS,
                               "mean_accept_len": float(gout["accept_len"].float().mean().item()),
                               "parity_sample": {"sequences": int(len(idx)), "mismatch": int(gdiff.sum())}}
    return line


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

    wl = rank_workload(rank, world, args.scaling, dev, {"B": args.batch} if args.batch else None)
    x, cfg = wl["x"], wl["cfg"]
    B, K, V = wl["nseq"], cfg.K, cfg.V
    es = 2 if cfg.dtype == "bf16" else 4
    alg_bytes, positions = wl["alg_bytes"], wl["positions"]
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
    main_kernel = P.bebop_debug_last_kernel()           # what the timed calls ran: the library chooses by shape
    launches_per_call = 6 if main_kernel == 1 else 2    # main kernel, fp64 re-draw kernel | 6 general kernels

    # median and best of single calls (an event pair around each call, so a little above the back-to-back mean)
    single = stats(per_call_ms(torch, [step], max(10, min(steps, 100)), barrier))

    # the same call without a TV output (the second sweep then reads only the rows a token is drawn from): not the
    # headline, which emits TV; reported beside it
    notv_steps = max(1, min(steps, 200))
    out_notv = {k: v for k, v in out.items() if k != "tv"}

    def step_notv():
        return P.bebop_verify(x["target"], x["draft"], x["draft_tokens"], x["u_accept"], x["u_final"],
                              draft_len=x["draft_len"], temperature=x["temperature"],
                              temperature_all=x["temperature_all"], out=out_notv, workspace=ws, want_tv=False)

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

    notv_ms = timed(step_notv, notv_steps)

    # the two other entry points on the same logits (reported beside the headline, not part of it)
    other_steps = max(1, min(steps, 50))
    tv_ms = gr_ms = float("nan")
    tv_kernel = 0
    if x["draft_len"] is None:
        tv_t = x["target"][:, :K].reshape(B * K, V)
        tv_d = x["draft"].reshape(B * K, V)
        tvws = torch.empty(P.bebop_workspace_bytes(B * K, 1, V, P.BEBOP_BF16), dtype=torch.uint8, device=dev)
        tv_ms = timed(lambda: P.bebop_tv(tv_t, tv_d, temperature_all=1.0, workspace=tvws), other_steps)
        tv_kernel = P.bebop_debug_last_kernel()
        gr_ms = timed(lambda: P.bebop_greedy_verify(x["target"], x["draft_tokens"], workspace=ws), other_steps)

    # end to end: pinned host inputs -> device, same C-ABI call, results back to the host
    e2e_steps = 0 if args.no_e2e else max(1, min(steps, 10))
    names = [k for k in ("target", "draft", "draft_tokens", "u_accept", "u_final", "draft_len", "temperature") if x.get(k) is not None]
    host = {k: x[k].cpu().pin_memory() for k in names} if e2e_steps else {}
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

    # totals over the ranks (work adds up, the job is as slow as its slowest rank)
    from paper_2606_12370_b200.shard import max_over_ranks
    ms, e2e_s, notv_ms, tv_ms, gr_ms = max_over_ranks([ms, e2e_s, notv_ms, tv_ms, gr_ms], dist, dev)
    tot = torch.tensor([positions, alg_bytes, B], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(tot)
    all_pos, all_bytes, all_seq = (float(v) for v in tot.cpu())
    sampler.stop()

    if rank == 0:
        ms_step = ms / steps
        peak, peak_kind = measured_peak()
        gbs = all_bytes / (ms_step * 1e-3) / 1e9
        headline = args.scaling == "weak" and B == 256 and cfg.name == WORKLOAD
        if args.scaling == "weak":
            workload = WORKLOAD_STR if B == 256 else WORKLOAD_STR.replace("B=256", "B=%d" % B)
        else:
            workload = ("full rollout batch (config 5): B=1024 K=4 V=151936 bf16, draft_len ~ U{1..4}, tau ~ U(0.6,1.2), cut into "
                        "%d contiguous blocks balanced by rows read" % world)
        line = {
            "metric": METRIC, "value": all_pos / (ms_step * 1e-3), "unit": "positions/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": workload,
                       "global_batch": int(all_seq), "positions_per_step": int(all_pos),
                       "l2": "inputs (%.0f MB per GPU) larger than the 126 MB L2; no flush" % (alg_bytes / 1e6),
                       "draw": "fp32 inverse CDF kept when it clears the error bound, else re-drawn in fp64",
                       "parallelism": "dp%d" % world},
            "clocks": clocks,
            "e2e": {"value": all_pos / e2e_s, "unit": "positions/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_s * 1e3},
            "gpu_launches": steps * launches_per_call,
            "single_call_ms": single,
            "other_entry_points": {
                "bebop_tv": {"ms_per_call": tv_ms, "row_pairs": world * B * K, "steps": other_steps, "kernel": KERNEL_NAME.get(tv_kernel),
                             "algorithmic_gbs": world * B * K * 2 * V * es / (tv_ms * 1e-3) / 1e9},
                "bebop_greedy_verify": {"ms_per_call": gr_ms, "steps": other_steps,
                                        "algorithmic_gbs": world * B * (K + 1) * V * es / (gr_ms * 1e-3) / 1e9}},
            "without_tv": {"value": all_pos / (notv_ms * 1e-3), "unit": "positions/s", "ms_per_step": notv_ms,
                           "steps": notv_steps, "note": "same call with tv = NULL; not the headline"},
            "hbm_gbs": gbs, "hbm_pct_of_8tbs": 100.0 * gbs / NORTH_STAR_PEAK_GBS,
            "target": "70 % of 8 TB/s for the fused kernel (north star): not met",
            "input_checksums": checksums(G, x),
            "roofline": roofline(alg_bytes, kern_ms, peak, peak_kind, headline, KERNEL_NAME.get(main_kernel, "general kernels"), len(pairs)),
        }
        if world == 1 and not args.no_configs:
            del host, dev_in, staged
            torch.cuda.empty_cache()
            line["configs"] = {}
            for i, name in enumerate(("tiny", "rollout", "high_entropy", "large_vocab", "full_batch")):
                line["configs"]["config%d_%s" % (i + 1, name)] = config_line(torch, P, G, name, dev, barrier, max(20, min(steps, 40)))
                torch.cuda.empty_cache()
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            cores = oracle.num_threads()
            nseq = min(64, B)
            xc = {k: (v[:nseq].cpu() if hasattr(v, "cpu") else v) for k, v in x.items()}
            oracle_rate(slice_inputs(xc, 0, min(8, nseq)))
            reps, spent = 0, 0.0
            while spent < 10.0 and reps < 1000:
                _, dt = oracle_rate(xc)
                spent += dt
                reps += 1
            line["cpu_baseline"] = {"value": reps * nseq * K / spent, "unit": "positions/s", "cores": cores,
                                    "kind": "oracle",
                                    "sample": "first %d of the step's %d sequences, %d passes, %.1f s" % (nseq, B, reps, spent)}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------- launching the ranks ourselves
def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _spawned(local_rank, args, port):
    os.environ.update(RANK=str(local_rank), LOCAL_RANK=str(local_rank), WORLD_SIZE=str(args.gpus),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    (run_reference if args.impl == "reference" else run_ours)(args)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: a headline batch per GPU; strong: the full rollout batch (config 5) cut across the GPUs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the block of the five benchmark configurations")
    ap.add_argument("--batch", type=int, default=0,
                    help="profiling aid: sequences per GPU instead of the workload's 256 (not a bench line)")
    ap.add_argument("--no-e2e", action="store_true", help="profiling aid: skip the host-buffer leg")
    ap.add_argument("--path", type=int, default=0, help="profiling aid: kernel path (0 default: chosen by shape, 1 general kernels, 2 pipelined kernel, 3 fused kernel)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # no launcher: start the ranks here, one per GPU
        import torch
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit("bench.py --gpus %d: only %d CUDA device(s) visible" % (args.gpus, torch.cuda.device_count()))
        import torch.multiprocessing as mp
        mp.spawn(_spawned, args=(args, _free_port()), nprocs=args.gpus, join=True)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
