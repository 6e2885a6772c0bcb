#!/usr/bin/env python
"""Benchmark of the sparse secret-shared FFN path on B200.

One "step" is one pass of the whole path for both parties over one batch of
synthetic input: mask compaction, up-projection (open, exchange, combine),
truncation, down-projection, truncation.  Default workload: the OPT-1.3B-shaped
FFN (tokens 512, d_model 2048, d_ff 8192, 16 fractional bits) at 90 % block
sparsity.  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload opt1.3b] [--sparsity 0.9] [--path auto|simt|limb]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2505_07239_b200 import ranks  # noqa: E402
from paper_2505_07239_b200 import workloads as wl  # noqa: E402

METRIC = "sparse shared-FFN Z_2^64 MACs/s"
UNIT = "MAC64/s"
L2_FLUSH_BYTES = 512 << 20

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the tensor-core combine kernel on the
# default workload, from the committed ncu summary of that kernel (average of the up- and the down-projection
# launch).  Valid only for the kernel source it was taken on: keyed by the SHA-256 of the kernel's part of
# kernels_limb.cuh.
COMBINE_LIMB_TRAFFIC = {
    "workload": ("opt1.3b", 0.9),
    "kernel_sha256": "0f2e1699f0109bf7b914f0fe698b6c08b30d5eb70620faf5cffb1cb7cfccd669",
    "bytes_per_launch": 132884480,
}


def combine_traffic(workload, sparsity, used_path):
    """The stored ncu DRAM traffic of the dominant kernel, or None when it does not apply any more."""
    import hashlib

    if used_path != "limb" or (workload, round(sparsity, 4)) != COMBINE_LIMB_TRAFFIC["workload"]:
        return None
    src = os.path.join(ROOT, "paper_2505_07239_b200", "csrc", "kernels_limb.cuh")
    try:
        with open(src) as fh:
            text = fh.read()
        # the kernel proper: from its argument block to the banner of the next kernel in the file
        text = text[text.index("struct LimbArgs {"):text.index("// Few tokens (M <= 32")]
        digest = hashlib.sha256(text.encode()).hexdigest()
    except (OSError, ValueError):
        return None
    return COMBINE_LIMB_TRAFFIC["bytes_per_launch"] if digest == COMBINE_LIMB_TRAFFIC["kernel_sha256"] else None


def ffn_macs(cfg, T, n):
    """Algorithmic ring MACs of one step, both parties: 2*T*K*N per party per product."""
    g = cfg.groups
    return 2 * (2 * T * cfg.d_model * g * n) + 2 * (2 * T * n * cfg.d_model)


def ffn_bytes(cfg, T, n):
    """Algorithmic bytes of one step, both parties: 8*(6KN + 6TK + 2TN) per party per product."""
    d, g = cfg.d_model, cfg.groups
    up = 8 * (6 * d * g * n + 6 * T * d + 2 * T * g * n)
    dn = 8 * (6 * n * d + 6 * T * n + 2 * T * d)
    return 2 * (up + dn)


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """`nvidia-smi` polled every 20 ms by a child process for the whole run; every sample is stamped on arrival and
    a timed region is summarised from the samples that fell inside it.  The child is started long before the first
    timed region (its start-up takes longer than a region lasts) and adds no work to the device."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.samples.append((time.perf_counter(), line.strip()))

    def wait_ready(self, limit_s: float = 5.0):
        """Wait (device idle) until the first sample has arrived."""
        t0 = time.perf_counter()
        while self.proc is not None and not self.samples and time.perf_counter() - t0 < limit_s:
            time.sleep(0.01)

    def region(self, t0: float, t1: float) -> dict:
        """Summary of the samples taken between the host times t0 and t1 (a sample shows up some milliseconds after
        it was taken, so arrivals up to 30 ms after t1 count, and a region shorter than the polling period takes
        the first sample after it began)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        inside = [ln for t, ln in list(self.samples) if t0 <= t <= t1 + 0.03]
        if not inside:
            inside = [ln for t, ln in list(self.samples) if t >= t0][:1]
        sm, mx, reasons = [], [], set()
        for line in inside:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()


# --------------------------------------------------------------------------- inputs
def make_inputs(cfg, seed, sparsity, step, T):
    """One batch in the paper's shapes: mask, X shares, triples, synthetic hidden state."""
    mask = wl.block_mask(cfg, seed, sparsity, step)
    n = int(mask.sum()) * cfg.block
    g, d = cfg.groups, cfg.d_model
    _, X0, X1 = wl.activation_shares(cfg, seed, step=step, tokens=T)
    up = wl.dealer_triple(seed, f"bench/up/{step}", T, d, g * n, valid=False)
    dn = wl.dealer_triple(seed, f"bench/dn/{step}", T, n, d, valid=False)
    _, H0, H1 = wl.hidden_shares(cfg, seed, n, step=step, tokens=T)
    return {"mask": mask, "n": n, "X": (X0, X1), "up": up, "dn": dn, "H": (H0, H1)}


def lib_tensors(inp):
    """Per party, (tensor id -> numpy array in the library's storage layout)."""
    from paper_2505_07239_b200 import binding as cb

    out = []
    for p in (0, 1):
        out.append({
            cb.X: inp["X"][p], cb.A_UP: inp["up"]["A"][1 + p], cb.B_UP: wl.lib_layout(inp["up"]["B"][1 + p]),
            cb.C_UP: inp["up"]["C"][1 + p], cb.H: inp["H"][p], cb.A_DN: inp["dn"]["A"][1 + p],
            cb.B_DN: wl.lib_layout(inp["dn"]["B"][1 + p]), cb.C_DN: inp["dn"]["C"][1 + p]})
    return out


# --------------------------------------------------------------------------- CPU oracle leg
def time_oracle(cfg, seed, sparsity, budget_s=15.0):
    """The oracle as it stands, single thread, on a bounded sample (a prefix of
    the token rows) of the same workload: SOMM, truncate, SIMM, truncate."""
    import oracle

    W = wl.model_shares(cfg, seed, plain=False)
    g = cfg.groups

    def run(T):
        inp = make_inputs(cfg, seed, sparsity, 0, T)
        I1 = oracle.index_set(inp["mask"], cfg.block, 1)
        Ig = oracle.index_set(inp["mask"], cfg.block, g)
        Wup = tuple(np.concatenate([W["WG"][s], W["W1"][s]], axis=1) if cfg.gated else W["W1"][s] for s in (1, 2))
        t0 = time.perf_counter()
        oracle.index_set(inp["mask"], cfg.block, g)
        r = oracle.somm(inp["X"], Wup, Ig, inp["up"]["A"][1:], inp["up"]["B"][1:], inp["up"]["C"][1:])
        for p in (0, 1):
            oracle.truncate(p, r["Z"][p], cfg.frac_bits)
        y = oracle.simm(inp["H"], W["W2"][1:], I1, inp["dn"]["A"][1:], inp["dn"]["B"][1:], inp["dn"]["C"][1:])
        for p in (0, 1):
            oracle.truncate(p, y["Z"][p], cfg.frac_bits)
        dt = time.perf_counter() - t0
        return dt, ffn_macs(cfg, T, inp["n"])

    probe_T = min(cfg.tokens, 8)
    dt, macs = run(probe_T)
    T = int(max(probe_T, min(cfg.tokens, probe_T * budget_s / max(dt, 1e-6))))
    if T > probe_T:
        dt, macs = run(T)
    return {"value": macs / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": round(dt, 3),
            "sample": f"first {T} of {cfg.tokens} token rows of the same workload, whole path, both parties",
            "host": host_cpu()}


def bf16_sustained_derived(peaks: dict) -> float:
    """Ring multiply-adds per second (in T) the sustained bf16 GEMM figure implies at the nominal int8 : bf16 ratio."""
    return peaks.get("bf16_tflops_sustained", 1400.0) * 1e12 / 2 * 2 / 36 / 1e12


def host_cpu() -> dict:
    """The machine the oracle was timed on: model name and the number of cores it offers (the oracle uses one)."""
    model = None
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.lower().startswith("model name"):
                    model = ln.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"model": model, "logical_cores": os.cpu_count()}


def run_reference(args, cfg, sparsity):
    rank, _, _ = ranks.rank_world_local()
    if rank != 0:
        return          # under a multi-process launch rank 0 alone times the oracle; the others leave with status 0
    steps = max(1, args.steps)
    per = max(2.0, min(30.0, 120.0 / (steps + args.warmup)))
    vals = []
    for s in range(args.warmup + steps):
        r = time_oracle(cfg, 1234 + s, sparsity, budget_s=per)
        if s >= args.warmup:
            vals.append(r)
    value = float(np.mean([v["value"] for v in vals]))
    n = cfg.n_active_blocks(sparsity) * cfg.block
    ms = ffn_macs(cfg, cfg.tokens, n) / value * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, sparsity), "note": "CPU oracle, one thread, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": vals[-1]["sample"],
                         "host": host_cpu()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_name(cfg, sparsity):
    n = cfg.n_active_blocks(sparsity) * cfg.block
    return (f"{cfg.name} FFN tokens={cfg.tokens} d_model={cfg.d_model} d_ff={cfg.d_ff} f={cfg.frac_bits} "
            f"block={cfg.block} sparsity={sparsity:.2f} n_active={n}")


# --------------------------------------------------------------------------- oblivious shuffle (secondary line)
def run_shuffle(args, cfg):
    """`--op shuffle`: the online stage of the oblivious shuffle (Protocol 1) on the workload's activation matrix
    [tokens, d_model], both parties, against the HBM roofline.  Algorithmic bytes per party: read x, a, the
    received y and b, write y and z = 48 bytes per word, plus the two index arrays."""
    import torch

    from paper_2505_07239_b200 import binding as cb

    rank, world, local = ranks.rank_world_local()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rows, cols = cfg.tokens, cfg.d_model
    if args.shuffle_rows:
        rows = args.shuffle_rows
    seed = ranks.rank_seed(2000, rank)
    sets = max(4, int((2 * L2_FLUSH_BYTES) // (6 * 8 * rows * cols)) + 1)      # rotating sets well beyond L2
    sets = min(sets, 64)
    data = []
    for s in range(sets):
        m = wl.dealer_shuffle(seed, f"bench/shuffle/{s % 4}", rows, cols)      # 4 distinct draws, copied to fresh memory
        x = wl.random_u64(seed, f"bench/shuffle/x/{s % 4}", rows * cols).reshape(rows, cols)
        xs = wl.split_shares(x, seed, f"bench/shuffle/x/{s % 4}")
        d64 = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int64)).to(dev)   # noqa: E731
        d32 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)                  # noqa: E731
        data.append(([d64(v) for v in xs], [d32(v) for v in m["tau"]], [d32(v) for v in m["rho"]],
                     [d64(v) for v in m["a"]], [d64(v) for v in m["b"]]))
    stream = torch.cuda.Stream(device=dev)
    bytes_step = 2 * (48 * rows * cols + 8 * rows)
    for s in range(max(3, args.warmup)):
        cb.shuffle(*data[s % sets], stream=stream)
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_ready()
    evs = []
    host0 = time.perf_counter()
    for s in range(args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        cb.shuffle(*data[s % sets], stream=stream)
        e1.record(stream)
        evs.append((e0, e1))
    torch.cuda.synchronize(dev)
    clocks = sampler.region(host0, time.perf_counter()) if rank == 0 else None
    sampler.stop()
    total_ms = float(sum(a.elapsed_time(b) for a, b in evs))
    (total_ms,) = ranks.max_over_ranks([total_ms], dev)
    if rank != 0:
        return
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    hbm = peaks.get("hbm_gbs", 6650.0)
    gbs = ranks.whole_job_throughput(bytes_step, world, args.steps, total_ms) / 1e9
    print(json.dumps({
        "metric": "oblivious shuffle online stage, algorithmic GB/s", "value": gbs, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": f"rows={rows} cols={cols} (activation matrix of {cfg.name}), both parties",
                   "l2": f"{sets} rotating input sets, {sets * 6 * 8 * rows * cols >> 20} MiB in total"},
        "gpu_launches": 2 * args.steps, "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": gbs / world, "peak": hbm, "unit": "GB/s",
                     "frac": gbs / world / hbm, "traffic": None, "kernel": "shuffle_rows_kernel (2 launches per step)",
                     "peak_source": "measured" if peaks else "fallback"}}))


# --------------------------------------------------------------------------- one layer sharded over the neurons
def run_sharded(args, cfg, sparsity):
    """`--shard neurons`: ONE FFN problem per step for the whole job, its neurons dealt to the ranks block by block
    (rank r owns blocks r, r + N, ...; it stores only its slice of the weights).  The up-projection needs no
    exchange; every rank's down-projection is a partial sum of Eq. 1, the partial shares are added over the ranks
    with one integer all-reduce per party, and the sum is truncated.  Strong scaling: the work per step is fixed."""
    import torch
    import torch.distributed as dist

    from paper_2505_07239_b200 import binding as cb
    from paper_2505_07239_b200 import shard

    rank, world, local = ranks.rank_world_local()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    assert cfg.n_blocks % world == 0, "the block count must be a multiple of the number of ranks"
    if args.warmup < 3:
        args.warmup = 3
    T, d, g, f = cfg.tokens, cfg.d_model, cfg.groups, cfg.frac_bits
    seed = 1000                                       # the same layer on every rank
    stream = torch.cuda.Stream(device=dev)
    n_glob = cfg.n_active_blocks(sparsity) * cfg.block
    ctx = cb.Comet(T, d, cfg.d_ff // world, cfg.block, f, cfg.groups - 1, local, 0, cb.PATH_AUTO, stream)
    W = wl.model_shares(cfg, seed, plain=False)
    with torch.cuda.stream(stream):
        for p in (0, 1):
            w1, w2 = shard.slice_stored_weights(wl.lib_layout(W["W1"][1 + p]), wl.lib_layout(W["W2"][1 + p]),
                                                cfg.block, rank, world)
            ctx.load_shares(p, cb.W1, cb.to_device(w1, dev))
            ctx.load_shares(p, cb.W2, cb.to_device(w2, dev))
            if cfg.gated:
                wg, _ = shard.slice_stored_weights(wl.lib_layout(W["WG"][1 + p]), wl.lib_layout(W["W2"][1 + p]),
                                                   cfg.block, rank, world)
                ctx.load_shares(p, cb.WG, cb.to_device(wg, dev))
    ctx.synchronize()
    del W
    sets = []
    for s_ in range(4):
        inp = make_inputs(cfg, seed, sparsity, s_, T)
        cols = shard.local_columns(inp["mask"], cfg.block, rank, world)
        gcols = np.concatenate([cols + k * inp["n"] for k in range(g)])          # [gate(I_r) || up(I_r)]
        zero = np.zeros((T, d), np.uint64)
        per = []
        for p in (0, 1):
            per.append({k: cb.to_device(np.ascontiguousarray(v), dev) for k, v in {
                cb.X: inp["X"][p], cb.A_UP: inp["up"]["A"][1 + p],
                cb.B_UP: wl.lib_layout(inp["up"]["B"][1 + p][:, gcols]), cb.C_UP: inp["up"]["C"][1 + p][:, gcols],
                cb.H: inp["H"][p][:, cols], cb.A_DN: inp["dn"]["A"][1 + p][:, cols],
                cb.B_DN: wl.lib_layout(inp["dn"]["B"][1 + p][cols, :]),
                cb.C_DN: inp["dn"]["C"][1 + p] if rank == 0 else zero}.items()})    # C' enters the sum once
        sets.append({"mask": torch.from_numpy(shard.local_mask(inp["mask"], rank, world)).to(dev), "dev": per,
                     "n_local": cols.size})
    torch.cuda.synchronize(dev)
    macs = ffn_macs(cfg, T, n_glob)
    y_view = [ctx.result_view(p, cb.Y, (T, d)) for p in (0, 1)]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def step(k):
        st = sets[k % 4]
        with torch.cuda.stream(stream):
            ctx.set_mask(st["mask"])
            for p in (0, 1):
                for tid, t in st["dev"][p].items():
                    if t.numel() and tid != cb.H:
                        ctx.bind_shares(p, tid, t)
            if st["n_local"]:
                ctx.ffn_up(T)
                ctx.truncate(cb.Z_UP)
                for p in (0, 1):
                    ctx.bind_shares(p, cb.H, st["dev"][p][cb.H])
            ctx.ffn_down(T)
            for p in (0, 1):
                shard.add_over_ranks(y_view[p])            # the exchange: partial shares added over the ranks
            ctx.truncate(cb.Y)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for k in range(args.warmup):
        step(k)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_ready()
    launches0 = ctx.stats().kernel_launches
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    host0 = time.perf_counter()
    with torch.cuda.stream(stream):
        flush.zero_()
        e0.record(stream)
    for k in range(args.steps):
        step(args.warmup + k)
    with torch.cuda.stream(stream):
        e1.record(stream)
    barrier()
    clocks = sampler.region(host0, time.perf_counter()) if rank == 0 else None
    sampler.stop()
    (ms,) = ranks.max_over_ranks([e0.elapsed_time(e1)], dev)
    launches = ctx.stats().kernel_launches - launches0
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": macs * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": workload_name(cfg, sparsity), "parallelism": f"neurons sharded over {world} rank(s), "
                       "one int64 all-reduce of Y_i per party per step", "l2": "4 rotating input sets with different "
                       "masks; 512 MiB flushed before the region", "timed": "region of exactly K steps between two "
                       "CUDA events on the library stream, collectives included, max over ranks"},
            "gpu_launches": int(launches), "clocks": clocks}))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- measured peaks of the multiply pipes
def measure_pipe_peaks(sampler, tensor_launches=24, alu_launches=12):
    """The rate of the int8 tensor pipe (the instruction the limb kernel issues, operands resident in shared
    memory) and of the 64-bit multiply-add loop on the integer ALUs, each as a run of back-to-back launches of
    about 25 ms: `burst` is the best of the first three launches, `sustained` the median of the last third (the
    part settles under its power limit within a few hundred milliseconds).  Rates in multiply-adds per second: 8-bit
    ones for the tensor pipe (a ring multiply-add costs 36 of them), 64-bit ones for the ALUs."""
    from paper_2505_07239_b200 import binding as cb

    out = {}
    for name, pipe, launches, work in (("tensor_i8", cb.PIPE_TENSOR_I8, tensor_launches, 10000),
                                       ("alu_u64", cb.PIPE_ALU_U64, alu_launches, 40000)):
        cb.pipe_probe(pipe, 2, max(1, work // 50))                         # load the module, touch the clocks
        t0 = time.perf_counter()
        ms, macs = cb.pipe_probe(pipe, launches, work)
        t1 = time.perf_counter()
        rates = [macs / (m * 1e-3) for m in ms]
        tail = rates[-max(1, launches // 3):]
        out[name] = {"burst": max(rates[:3]), "sustained": float(np.median(tail)), "unit": "MAC/s",
                     "launches": launches, "ms_per_launch": [round(m, 3) for m in ms],
                     "clocks": sampler.region(t0, t1) if sampler is not None else None}
        time.sleep(0.5)                                                    # let the part cool before the next probe
    t = out["tensor_i8"]
    t["ring_mac_burst"], t["ring_mac_sustained"] = t["burst"] / 36, t["sustained"] / 36
    if t["clocks"] and t["clocks"].get("sm_mhz"):
        # 8-bit multiply-adds per SM and clock at the sampled median clock (the pipe's nominal figure is 8192)
        t["macs_per_sm_clk_at_sampled_clock"] = t["sustained"] / 148 / (t["clocks"]["sm_mhz"] * 1e6)
    return out


def run_peak(args):
    """`--op peak`: only the measured pipe peaks, one JSON line."""
    import torch

    rank, world, local = ranks.rank_world_local()
    if rank != 0:
        return
    torch.cuda.set_device(local)
    sampler = ClockSampler(local)
    sampler.start()
    sampler.wait_ready()
    peaks = measure_pipe_peaks(sampler, tensor_launches=max(24, args.steps // 4), alu_launches=12)
    sampler.stop()
    print(json.dumps({"metric": "measured peak of the multiply pipes", "value": peaks["tensor_i8"]["ring_mac_burst"],
                      "unit": UNIT, "n_gpus": 1, "steps": peaks["tensor_i8"]["launches"], "warmup": 2,
                      "higher_is_better": True, "dtype": "u8 x u8 -> s32 (tensor), u64 (ALU)", "data": "synthetic",
                      "config": {"workload": "tcgen05.mma kind::i8 M128 N256 K32 loop, 148 CTAs, operands in shared "
                                             "memory; 64-bit multiply-add chains, 2 x 1024 threads per SM"},
                      "peaks": peaks}))


# --------------------------------------------------------------------------- GPU leg
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="opt1.3b", choices=sorted(wl.CONFIGS))
    ap.add_argument("--sparsity", type=float, default=None)
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "limb"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-peak-probe", action="store_true",
                    help="skip the measurement of the multiply pipes' peaks (the roofline then falls back to figures "
                         "derived from the bf16 GEMM peak / the unit counts)")
    ap.add_argument("--token-masks", type=float, default=0.0, metavar="P",
                    help="give every token its own Bernoulli(P) mask over the active blocks (Protocols 2 and 3 in "
                         "general: connected components, per-column row sets); set_token_mask is timed with set_mask")
    ap.add_argument("--clusters", type=int, default=0, metavar="G",
                    help="with --token-masks: deal tokens and active blocks to G groups of requests with disjoint "
                         "blocks (at least G connected components, members scattered); the up-projection then "
                         "computes the component rectangles only")
    ap.add_argument("--in-flight", type=int, default=4, metavar="C",
                    help="independent FFN problems in flight (contexts, one stream each, inputs bound in place); the "
                         "headline throughput is measured that way when C > 1, the one-problem-at-a-time figures are "
                         "reported beside it; 1 = only the latter")
    ap.add_argument("--op", default="ffn", choices=["ffn", "shuffle", "peak"],
                    help="ffn: the sparse FFN path (the headline); shuffle: the oblivious shuffle's online stage; "
                         "peak: the measured rates of the int8 tensor pipe and of the 64-bit ALU loop alone")
    ap.add_argument("--mask-location", default="host", choices=["host", "device"],
                    help="where the block mask (public, one byte per block) is when set_mask is called in the "
                         "device-resident timing: host memory (counted on the host, no round trip) or device memory "
                         "(the count comes back from the compaction kernel)")
    ap.add_argument("--shard", default="problems", choices=["problems", "neurons"],
                    help="how --gpus N > 1 divides the work: problems = every rank runs its own independent FFN "
                         "problems (no collective, weak scaling; the default); neurons = one problem per step, its "
                         "neurons dealt to the ranks, the down-projection's partial shares summed by an all-reduce "
                         "(strong scaling)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="the timed region of K steps is repeated until the device has been under load for this "
                         "long; the first (burst), median and last (sustained) region are reported")
    ap.add_argument("--shuffle-rows", type=int, default=0, help="--op shuffle: rows instead of the workload's tokens")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.workload]
    sparsity = args.sparsity
    if sparsity is None:
        sparsity = 0.9 if args.workload == "opt1.3b" else 1.0 - cfg.active_fraction
    if args.impl == "reference":
        return run_reference(args, cfg, sparsity)
    if args.op == "shuffle":
        return run_shuffle(args, cfg)
    if args.op == "peak":
        return run_peak(args)
    if args.shard == "neurons":
        return run_sharded(args, cfg, sparsity)
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist

    from paper_2505_07239_b200 import binding as cb

    rank, world, local = ranks.rank_world_local()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    T, d, g = cfg.tokens, cfg.d_model, cfg.groups
    sampler = ClockSampler(local)        # polls for the whole run; the timed regions pick their samples by time
    if rank == 0:
        sampler.start()
    seed = ranks.rank_seed(1000, rank)   # every rank runs its own independent FFN problems (weak scaling, no collective)
    path = {"auto": cb.PATH_AUTO, "simt": cb.PATH_SIMT, "limb": cb.PATH_LIMB}[args.path]
    stream = torch.cuda.Stream(device=dev)
    n_cap = cfg.n_active_blocks(sparsity) * cfg.block
    ctx = cb.Comet(T, d, cfg.d_ff, cfg.block, cfg.frac_bits, cfg.groups - 1, local, n_cap, path, stream)
    W = wl.model_shares(cfg, seed, plain=False)
    with torch.cuda.stream(stream):
        for p in (0, 1):
            ctx.load_shares(p, cb.W1, cb.to_device(wl.lib_layout(W["W1"][1 + p]), dev))
            ctx.load_shares(p, cb.W2, cb.to_device(wl.lib_layout(W["W2"][1 + p]), dev))
            if cfg.gated:
                ctx.load_shares(p, cb.WG, cb.to_device(wl.lib_layout(W["WG"][1 + p]), dev))
    ctx.synchronize()

    # rotating input sets: a fresh mask (so different weight rows), X, triples and H each
    R = 4

    def token_mask_for(inp, stream_name):
        """The per-token mask of one input set (None without --token-masks)."""
        if args.token_masks <= 0:
            return None
        nab = int(inp["mask"].sum())
        return torch.from_numpy(
            wl.token_block_masks_clustered(seed, stream_name, T, nab, args.clusters, args.token_masks)
            if args.clusters > 1 else wl.token_block_masks(seed, stream_name, T, nab, args.token_masks))

    sets = []
    for s in range(R):
        inp = make_inputs(cfg, seed, sparsity, s, T)
        host = lib_tensors(inp)
        pinned = [{k: torch.from_numpy(v.view(np.int64)).pin_memory() for k, v in hp.items()} for hp in host]
        devt = [{k: v.to(dev) for k, v in hp.items()} for hp in pinned]
        tm = token_mask_for(inp, f"bench/tm/{s}")
        sets.append({"n": inp["n"], "tm_host": tm.pin_memory() if tm is not None else None,
                     "tm_dev": tm.to(dev) if tm is not None else None,
                     "mask_host": torch.from_numpy(inp["mask"]).pin_memory(),
                     "mask_dev": torch.from_numpy(inp["mask"]).to(dev), "pinned": pinned, "dev": devt})
    torch.cuda.synchronize(dev)
    n = sets[0]["n"]
    macs = ffn_macs(cfg, T, n)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    y_host = [torch.empty((T, d), dtype=torch.int64).pin_memory() for _ in (0, 1)]
    # everything except the hidden state is known before the up-projection starts (the down-projection's
    # triple included); H stands for the output of the activation step that sits between the projections
    UP_IDS = (cb.X, cb.A_UP, cb.B_UP, cb.C_UP, cb.A_DN, cb.B_DN, cb.C_DN)
    DN_IDS = (cb.H,)

    # The block mask is the public sparsity distribution (one byte per block): by default it is handed over in host
    # memory, where the library counts it without a device round trip (its copy to the device and the compaction
    # kernel are inside the timed region); every share, triple and weight is resident in HBM.
    mask_key = "mask_host" if args.mask_location == "host" else "mask_dev"

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def device_step(s, timed):
        """Inputs resident in HBM: only the path's own calls sit between the event pairs."""
        st = sets[s % R]
        with torch.cuda.stream(stream):
            flush.zero_()                                  # evict L2 between steps
            e = [ev() for _ in range(6)]
            e[0].record(stream)
            ctx.set_mask(st[mask_key])
            if st["tm_dev"] is not None:
                ctx.set_token_mask(st["tm_dev"])
            e[1].record(stream)
            for p in (0, 1):
                for tid in UP_IDS:
                    ctx.load_shares(p, tid, st["dev"][p][tid])
            e[2].record(stream)
            ctx.ffn_up(T)
            ctx.truncate(cb.Z_UP)
            e[3].record(stream)
            for p in (0, 1):
                for tid in DN_IDS:
                    ctx.load_shares(p, tid, st["dev"][p][tid])
            e[4].record(stream)
            ctx.ffn_down(T)
            ctx.truncate(cb.Y)
            e[5].record(stream)
        return e if timed else None

    def e2e_step(s):
        """Through the C ABI with HOST buffers: H2D of every per-step input and D2H of the result inside."""
        st = sets[s % R]
        with torch.cuda.stream(stream):
            flush.zero_()
            e0, e1 = ev(), ev()
            e0.record(stream)
            ctx.set_mask(st["mask_host"].numpy())
            if st["tm_host"] is not None:
                ctx.set_token_mask(st["tm_host"].numpy())
            for p in (0, 1):
                for tid in UP_IDS:
                    ctx.load_shares(p, tid, st["pinned"][p][tid])
            ctx.ffn_up(T)
            ctx.truncate(cb.Z_UP)
            for p in (0, 1):
                for tid in DN_IDS:
                    ctx.load_shares(p, tid, st["pinned"][p][tid])
            ctx.ffn_down(T)
            ctx.truncate(cb.Y)
            for p in (0, 1):
                ctx.get_into(p, cb.Y, y_host[p])
            e1.record(stream)
        return e0, e1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing (the headline): per-phase timers off, nothing but the path between the events
    def repeat_regions(one_region):
        """Runs `one_region(index)` (exactly K timed steps; returns its device milliseconds) again and again until
        the device has been under load for --min-seconds, every rank the same number of times.  Returns the regions
        as dicts {ms (max over ranks), t0, t1 (host times, for the clock samples)}."""
        regions, busy = [], 0.0
        while True:
            t0 = time.perf_counter()
            ms = one_region(len(regions))
            t1 = time.perf_counter()
            regions.append({"ms": ms, "t0": t0, "t1": t1})
            busy += t1 - t0
            (busy_max,) = ranks.max_over_ranks([busy], dev)
            if busy_max >= args.min_seconds or len(regions) >= 5000:
                break
        for r, m in zip(regions, ranks.max_over_ranks([r["ms"] for r in regions], dev)):
            r["ms"] = m
        return regions

    def summarise(regions):
        """First (burst), median and last (sustained) region of a run, each with the clocks sampled while it ran."""
        order = sorted(range(len(regions)), key=lambda k: regions[k]["ms"])
        picks = {"first": regions[0], "median": regions[order[len(order) // 2]], "last": regions[-1]}
        out = {"regions": len(regions), "steps_per_region": args.steps,
               "seconds_under_load": round(regions[-1]["t1"] - regions[0]["t0"], 3)}
        for name, r in picks.items():
            out[name] = {"ms_per_step": r["ms"] / args.steps,
                         "value": ranks.whole_job_throughput(macs, world, args.steps, r["ms"]),
                         "clocks": sampler.region(r["t0"], r["t1"]) if rank == 0 else None}
        return out

    for s in range(args.warmup):
        device_step(s, False)
    barrier()
    launches0 = ctx.stats().kernel_launches
    if rank == 0:
        sampler.wait_ready()
    barrier()

    def single_region(index):
        first = args.warmup + index * args.steps
        events = [device_step(first + s, True) for s in range(args.steps)]
        barrier()
        return float(sum(e[0].elapsed_time(e[1]) + e[2].elapsed_time(e[3]) + e[4].elapsed_time(e[5]) for e in events))

    wall0 = time.perf_counter()
    single_regions = repeat_regions(single_region)
    wall = (time.perf_counter() - wall0) / len(single_regions)
    launches = (ctx.stats().kernel_launches - launches0) // len(single_regions)
    single_sum = summarise(single_regions)

    # ---- the same steps again with the library's per-phase event timers on: kernel time of each phase
    #      (the timers add two event records per phase, so this pass is slower and is not the headline)
    prof_steps = min(args.steps, 50)
    ctx.set_profiling(True)
    for s in range(prof_steps):
        device_step(s, False)
    barrier()
    stats = ctx.stats()
    ctx.set_profiling(False)
    up_counts = None
    if args.token_masks > 0:                    # what the up-projection of input set 0 covers under its token mask
        st0 = sets[0]
        ctx.set_mask(st0["mask_dev"])
        ctx.set_token_mask(st0["tm_dev"])
        for p in (0, 1):
            for tid in UP_IDS:
                ctx.load_shares(p, tid, st0["dev"][p][tid])
        ctx.ffn_up(T)
        su = ctx.stats()
        up_counts = {"components": su.n_components, "theorem1_macs": su.ring_macs,
                     "union_macs": 2 * 2 * T * d * cfg.groups * st0["n"], "tensor_tile_macs": su.tensor_tile_macs}
        barrier()

    # ---- several independent problems in flight (throughput mode): C contexts with their own weights, stream and
    #      two input sets each, inputs bound in place (no copies), steps issued round-robin; the region is timed
    #      as a whole on the device.  No flush here: consecutive uses of a context see different masks and inputs,
    #      and the contexts together hold far more than the L2.
    piped = None
    if args.in_flight > 1:
        C = args.in_flight
        tstream = torch.cuda.Stream(device=dev)
        pctx, psets = [], []
        for k in range(C):
            sk = torch.cuda.Stream(device=dev)
            cx = cb.Comet(T, d, cfg.d_ff, cfg.block, cfg.frac_bits, cfg.groups - 1, local, n_cap, path, sk)
            with torch.cuda.stream(sk):
                for p in (0, 1):
                    cx.load_shares(p, cb.W1, cb.to_device(wl.lib_layout(W["W1"][1 + p]), dev))
                    cx.load_shares(p, cb.W2, cb.to_device(wl.lib_layout(W["W2"][1 + p]), dev))
                    if cfg.gated:
                        cx.load_shares(p, cb.WG, cb.to_device(wl.lib_layout(W["WG"][1 + p]), dev))
            cx.synchronize()
            mine = []
            for j in range(2):
                inp = make_inputs(cfg, seed, sparsity, 100 + 2 * k + j, T)
                pinned = [{kk: torch.from_numpy(v.view(np.int64)).pin_memory() for kk, v in hp.items()}
                          for hp in lib_tensors(inp)]
                devt = [{kk: v.to(dev) for kk, v in hp.items()} for hp in pinned]
                tmk = token_mask_for(inp, f"bench/tm/p{k}/{j}")
                mine.append({"mask_dev": torch.from_numpy(inp["mask"]).to(dev), "dev": devt, "pinned": pinned,
                             "tm_dev": tmk.to(dev) if tmk is not None else None,
                             "tm_host": tmk.pin_memory() if tmk is not None else None,
                             "mask_host": torch.from_numpy(inp["mask"]).pin_memory(),
                             "y_host": [torch.empty((T, d), dtype=torch.int64).pin_memory() for _ in (0, 1)]})
            pctx.append((cx, sk))
            psets.append(mine)

        def piped_step(s):
            cx, sk = pctx[s % C]
            st = psets[s % C][(s // C) % 2]
            with torch.cuda.stream(sk):
                cx.set_mask(st[mask_key])
                if st["tm_dev"] is not None:
                    cx.set_token_mask(st["tm_dev"])
                for p in (0, 1):
                    for tid in UP_IDS:
                        cx.bind_shares(p, tid, st["dev"][p][tid])
                cx.ffn_up(T)
                cx.truncate(cb.Z_UP)
                for p in (0, 1):
                    cx.bind_shares(p, cb.H, st["dev"][p][cb.H])
                cx.ffn_down(T)
                cx.truncate(cb.Y)

        for s in range(max(2 * C, args.warmup)):
            piped_step(s)
        barrier()
        launched0 = sum(cx.stats().kernel_launches for cx, _ in pctx)

        def piped_region(index):
            p0, p1 = ev(), ev()
            p0.record(tstream)
            for s in range(args.steps):
                piped_step(index * args.steps + s)
            for cx, sk in pctx:
                done = torch.cuda.Event()
                done.record(sk)
                tstream.wait_event(done)
            p1.record(tstream)
            barrier()
            return float(p0.elapsed_time(p1))

        piped_regions = repeat_regions(piped_region)
        piped_sum = summarise(piped_regions)
        piped = {"in_flight": C, "ms_per_step": piped_sum["median"]["ms_per_step"],
                 "launches": int(sum(cx.stats().kernel_launches for cx, _ in pctx) - launched0) // len(piped_regions),
                 "value": piped_sum["median"]["value"], "unit": UNIT, "timed_regions": piped_sum,
                 "note": "C independent problems on C streams, inputs bound in place, every region of K steps timed "
                         "as a whole on the device; the median region is the figure"}

        # ---- the same C problems in flight end to end: every step copies its inputs from pinned host memory and
        #      its result back, on its context's stream, so one problem's copies run under another's kernels
        def piped_e2e_step(s):
            cx, sk = pctx[s % C]
            st = psets[s % C][(s // C) % 2]
            with torch.cuda.stream(sk):
                cx.set_mask(st["mask_host"].numpy())
                if st["tm_host"] is not None:
                    cx.set_token_mask(st["tm_host"].numpy())
                for p in (0, 1):
                    for tid in UP_IDS:
                        cx.load_shares(p, tid, st["pinned"][p][tid])
                cx.ffn_up(T)
                cx.truncate(cb.Z_UP)
                for p in (0, 1):
                    cx.load_shares(p, cb.H, st["pinned"][p][cb.H])
                cx.ffn_down(T)
                cx.truncate(cb.Y)
                for p in (0, 1):
                    cx.get_into(p, cb.Y, st["y_host"][p])

        for s in range(2 * C):
            piped_e2e_step(s)
        barrier()
        q0, q1 = ev(), ev()
        q0.record(tstream)
        for s in range(args.steps):
            piped_e2e_step(s)
        for cx, sk in pctx:
            done = torch.cuda.Event()
            done.record(sk)
            tstream.wait_event(done)
        q1.record(tstream)
        barrier()
        (piped_e2e_ms,) = ranks.max_over_ranks([q0.elapsed_time(q1)], dev)
        for cx, _ in pctx:
            cx.close()
    del W

    # ---- end-to-end timing (host buffers)
    for s in range(3):
        e2e_step(s)
    barrier()
    pairs = [e2e_step(3 + s) for s in range(args.steps)]
    barrier()
    e2e_ms = float(sum(a.elapsed_time(b) for a, b in pairs))
    h2d = sum(t.numel() * 8 for p in (0, 1) for t in sets[0]["pinned"][p].values()) + sets[0]["mask_host"].numel()
    d2h = 2 * T * d * 8 + 4

    (e2e_ms,) = ranks.max_over_ranks([e2e_ms], dev)
    e2e_single_ms = e2e_ms
    e2e_in_flight = piped is not None and piped_e2e_ms < e2e_ms
    if e2e_in_flight:
        e2e_ms = piped_e2e_ms

    # ---- measured peaks of the two multiply pipes, after the path's own timing (the probes heat the part)
    pipe_peaks = None
    if rank == 0 and not args.no_peak_probe:
        torch.cuda.synchronize(dev)
        time.sleep(1.0)
        pipe_peaks = measure_pipe_peaks(sampler)
    sampler.stop()

    if rank == 0:
        single = {"ms_per_step": single_sum["median"]["ms_per_step"], "value": single_sum["median"]["value"],
                  "unit": UNIT, "timed_regions": single_sum,
                  "note": "one problem at a time on one stream; sum over set_mask, ffn_up + truncate, ffn_down + "
                          "truncate of CUDA-event pairs; 512 MiB written between steps to flush L2; the median "
                          "region of K steps is the figure"}
        # Two issue policies are measured in this run; the headline is the faster one (large dense problems gain
        # nothing from sharing the GPU, small sparse ones hide their memory-side kernels under another problem's
        # tensor-core kernel), and both are reported.
        use_piped = piped is not None and piped["value"] > single["value"]
        chosen = piped_sum if use_piped else single_sum
        ms_per_step, value = chosen["median"]["ms_per_step"], chosen["median"]["value"]
        phase = {name: {"ms_per_step": stats.phase_ms[k] / prof_steps, "launches_per_step":
                        stats.phase_launches[k] / prof_steps} for k, name in enumerate(cb.PHASE_NAMES)}
        comb_launch_ms = stats.phase_ms[3] / max(1, stats.phase_launches[3])
        comb_macs_per_launch = macs / 2          # up and down combine launches carry half the MACs each here
        used_path = {cb.PATH_SIMT: "simt", cb.PATH_LIMB: "limb"}.get(stats.matmul_path, "?")
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except OSError:
            pass
        hbm = peaks.get("hbm_gbs", 6650.0)
        bf16 = peaks.get("bf16_tflops", 1590.0)
        src = "measured" if peaks else "fallback"
        achieved = comb_macs_per_launch / (comb_launch_ms * 1e-3) / 1e12
        # per launch, both parties: planes of both operand pairs read once, Z read and written once (average of the
        # up- and the down-projection launch)
        comb_bytes_per_launch = 8 * ((2 * T * d + 2 * d * g * n + 2 * T * g * n) + (2 * T * n + 2 * n * d + 2 * T * d))
        if used_path == "limb":
            # The pipe's peak in ring multiply-adds: the measured rate of the tensor instruction the kernel issues,
            # over 36 limb products.  Beside it, what the measured bf16 GEMM peak would imply at the nominal int8 :
            # bf16 ratio of 2 (the figure used before the pipe itself was measured).
            derived = bf16 * 1e12 / 2 * 2 / 36 / 1e12
            if pipe_peaks is not None:
                peak = pipe_peaks["tensor_i8"]["ring_mac_burst"] / 1e12
                peak_sustained = pipe_peaks["tensor_i8"]["ring_mac_sustained"] / 1e12
                peak_source = ("measured in this run: tcgen05.mma kind::i8 M128 N256 K32 loop on 148 SMs, operands in "
                               "shared memory, best of the first three 25 ms launches, / 36 limb products")
            else:
                peak, peak_sustained = derived, bf16_sustained_derived(peaks)
                peak_source = f"{src} bf16 GEMM peak x2 (int8 nominal ratio), as MAC/s, / 36 limb products"
            t_tensor = comb_macs_per_launch / (peak * 1e12)
            t_hbm = comb_bytes_per_launch / (hbm * 1e9)
            if t_hbm > t_tensor:
                # few tokens: the kernel streams the weight-side planes once and is bound by that traffic
                roof = {"bound": "hbm", "achieved": comb_bytes_per_launch / (comb_launch_ms * 1e-3) / 1e9, "peak": hbm,
                        "unit": "GB/s", "peak_source": f"{src} HBM copy peak"}
            else:
                roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TMAC64/s",
                        "peak_source": peak_source, "peak_sustained": peak_sustained,
                        "frac_of_sustained_peak": achieved / peak_sustained,
                        "peak_from_bf16_gemm": derived, "frac_of_peak_from_bf16_gemm": achieved / derived}
        else:
            # 148 SMs x 64 32-bit integer multiply-add lanes per clock x max SM clock / 4 issue slots per ring MAC
            derived = 148 * 64 * 1.965e9 / 4 / 1e12
            if pipe_peaks is not None:
                peak = pipe_peaks["alu_u64"]["burst"] / 1e12
                peak_sustained = pipe_peaks["alu_u64"]["sustained"] / 1e12
                peak_source = ("measured in this run: eight 64-bit multiply-add chains per thread, 2 x 1024 threads per "
                               "SM, best of the first three 25 ms launches")
            else:
                peak = peak_sustained = derived
                peak_source = "148 SM x 64 int32 mul-add lanes/clk x 1.965 GHz / 4 issue slots per 64-bit MAC"
            roof = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TMAC64/s", "peak_source": peak_source,
                    "peak_sustained": peak_sustained, "frac_of_sustained_peak": achieved / peak_sustained,
                    "peak_from_unit_counts": derived}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["kernel"] = "combine_" + used_path + ("_few" if used_path == "limb" and T <= 32 else "")
        roof["traffic"] = combine_traffic(args.workload, sparsity, used_path)
        roof["traffic_unit"] = "bytes per launch (ncu dram read+write); algorithmic: planes once + Z read-modify-write"
        roof["algorithmic_bytes_per_launch"] = comb_bytes_per_launch
        roof["timed"] = "kernel time per launch from the per-phase CUDA-event pass, one problem at a time"

        def t_roof_ms(pipe_peak):                 # slower of bytes at the HBM peak and MACs at the pipe's peak
            return max(ffn_bytes(cfg, T, n) / (hbm * 1e9), macs / (pipe_peak * 1e12)) * 1e3

        path_roof = {"algorithmic_bytes": ffn_bytes(cfg, T, n), "algorithmic_macs": macs, "hbm_gbs": hbm,
                     "hbm_source": src, "pipe_peak": peak, "pipe_peak_sustained": peak_sustained,
                     "roofline_ms": t_roof_ms(peak), "roofline_ms_sustained_peak": t_roof_ms(peak_sustained),
                     "frac": t_roof_ms(peak) / ms_per_step,
                     "note": "frac = roofline at the burst peak over the median region of the reported policy; below, "
                             "first region against the burst peak and last region (after --min-seconds of load) "
                             "against the sustained peak, for both policies"}
        for name, summ in (("single_problem", single_sum), ("problems_in_flight", piped_sum if piped else None)):
            if summ is not None:
                path_roof[name] = {
                    "frac_first_region_burst_peak": t_roof_ms(peak) / summ["first"]["ms_per_step"],
                    "frac_median_region_burst_peak": t_roof_ms(peak) / summ["median"]["ms_per_step"],
                    "frac_last_region_sustained_peak": t_roof_ms(peak_sustained) / summ["last"]["ms_per_step"]}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": workload_name(cfg, sparsity), "matmul_path": used_path,
                       "in_flight": args.in_flight if use_piped else 1,
                       "block_mask": f"{cfg.n_blocks} bytes, passed from {args.mask_location} memory; all shares, "
                                     "triples and weights resident in HBM",
                       "l2": (f"{args.in_flight} contexts x 2 input sets with different masks rotate (inputs, gathered "
                              "weight rows and intermediates of consecutive steps far exceed the L2); no flush"
                              if use_piped else
                              "512 MiB buffer written between steps, and 4 rotating input sets with different masks"),
                       "timed": ("every step = set_mask + bind inputs + ffn_up + truncate + ffn_down + truncate; a region "
                                 "of exactly K steps between two CUDA events" if use_piped else
                                 "set_mask + ffn_up + truncate + ffn_down + truncate, CUDA events on the library stream, "
                                 "summed over a region of exactly K steps") +
                                f"; the region is repeated for {args.min_seconds} s of load and the median region is "
                                "the value (first and last regions under timed_regions)",
                       "token_masks": (f"per-token Bernoulli({args.token_masks}) masks over the active blocks, "
                                       f"{stats.n_components} component(s)"
                                       + (f", {args.clusters} groups of requests" if args.clusters > 1 else "")
                                       if args.token_masks > 0 else "none"),
                       "up_projection_under_token_mask": up_counts,
                       "parallelism": f"independent FFN per GPU x{world}"},
            "gpu_launches": int(piped["launches"] if use_piped else launches),
            "clocks": chosen["median"]["clocks"],
            "timed_regions": chosen,
            "e2e": {"value": ranks.whole_job_throughput(macs, world, args.steps, e2e_ms), "unit": UNIT,
                    "ms_per_step": e2e_ms / args.steps, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "in_flight": args.in_flight if e2e_in_flight else 1,
                    "single_problem_ms_per_step": e2e_single_ms / args.steps,
                    "in_flight_ms_per_step": piped_e2e_ms / args.steps if piped is not None else None,
                    "note": "host buffers through the C ABI: H2D of every per-step input from pinned memory and D2H of "
                            "the result inside the timed region; the faster of one problem at a time and C in flight"},
            "roofline": roof,
            "path_roofline": path_roof,
            "pipe_peaks": pipe_peaks,
            "single_problem": single,
            "problems_in_flight": piped,
            "phases": phase,
            "phases_note": f"separate pass of {prof_steps} steps with the per-phase event timers on",
            "wall_ms_per_step_incl_untimed": wall / args.steps * 1e3,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = time_oracle(cfg, 1234, sparsity)
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
