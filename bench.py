#!/usr/bin/env python
"""Benchmark of the outer synchronisation round (one JSON line on stdout).

A "step" is one whole outer round of the headline workload (K=16 workers, P=300M fp32
parameters each): per-round mix descriptors built on the host, Mix1 = global average launched
on a side stream, then on the main stream the fused outer step (outer gradient + ring Mix2 +
Nesterov update + consensus partial sums) updating theta and the momentum in place, with the
per-round consensus sums kept in a device log.  theta_local (the result of the workers' inner
steps) is the step's input and is resident in HBM when the timed region starts.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 1..5]

N > 1 (launched by torch.distributed.run, one rank per GPU) runs N independent replicas of the
same workload -- the path has no exchange between GPUs -- and reports the aggregate.
--impl reference times the float64 CPU oracle on a bounded column sample of the same workload.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "outer_round_worker_params_per_s"
UNIT = "worker-params/s"
FALLBACK_HBM_GBS = 6650.0

# the five benchmark configurations (1-based)
CONFIGS = {
    1: dict(K=4, P=1 << 20, mix1=("mean",), mix2=("ring",), sig=(1e-3, 1e-3), p_fail=0.0,
            name="cfg1 K=4 P=2^20 Mix1=mean Mix2=ring"),
    2: dict(K=8, P=150_000_000, mix1=("mean",), mix2=("xor",), sig=(1e-3, 1e-3), p_fail=0.0,
            name="cfg2 K=8 P=150M Mix1=mean Mix2=one-peer-xor"),
    3: dict(K=16, P=300_000_000, mix1=("mean",), mix2=("ring",), sig=(5e-4, 2e-3), p_fail=0.0,
            name="cfg3 K=16 P=300M Mix1=mean(side stream) Mix2=ring"),
    4: dict(K=16, P=300_000_000, mix1=("hypercube",), mix2=("hypercube",), sig=(1e-3, 1e-3), p_fail=0.1,
            name="cfg4 K=16 P=300M Mix1=Mix2=hypercube gossip, p_fail=0.1 Metropolis"),
    5: dict(K=64, P=50_000_000, mix1=("mean",), mix2=("dense",), sig=(1e-3, 1e-3), p_fail=0.0,
            name="cfg5 K=64 P=50M Mix1=mean Mix2=dense Sinkhorn"),
    # beyond the five: the paper's own experimental scale (Sec. 5: 8 workers, a 1.5 B-parameter model,
    # non-blocking global average + blocking pairwise gossip, 5 % failed exchanges), 150 GB of state
    6: dict(K=8, P=1_500_000_000, mix1=("mean",), mix2=("matching",), sig=(1e-3, 1e-3), p_fail=0.05,
            name="cfg6 K=8 P=1.5B Mix1=mean Mix2=random pairwise gossip, p_fail=0.05 (the paper's scale)"),
}

# DRAM bytes per worker-parameter of the fused outer-step kernel measured with ncu
# (dram__bytes_read.sum + dram__bytes_write.sum over one launch / (K*P) of that launch); the
# capture it comes from is summarised under profiles/.  None = not captured yet.
NCU_TRAFFIC_BYTES_PER_WORKER_PARAM = {2: 20.29, 3: 20.04, 4: 23.81, 5: 19.85, 6: 20.29}   # 6 runs config 2's kernel
NCU_TRAFFIC_FUSED_MIX1 = {4: 19.79}   # the same with --fuse-mix1


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=sorted(CONFIGS))
    ap.add_argument("--cols", type=int, default=0,
                    help="profiling only: shrink P to this many columns (same kernels, smaller launch)")
    ap.add_argument("--subset-frac", type=float, default=0.0,
                    help="variant: restrict Mix2 to about this fraction of the columns (three blocks)")
    ap.add_argument("--average-momentum", action="store_true", help="variant: GlobalM1S (needs Mix1 = mean)")
    ap.add_argument("--chain-mix1", action="store_true",
                    help="variant: the fused step also writes next round's global-average Mix1 (no Mix1 kernel)")
    ap.add_argument("--fuse-mix1", action="store_true",
                    help="variant: Mix1 computed inside the fused step from the staged theta_prev (one launch per round, 20 B per worker-parameter)")
    ap.add_argument("--graph", action="store_true",
                    help="variant: capture the round (Mix1 + fused step) into one CUDA graph and time its replays")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the round: the fused step across worker counts and mix kinds (4 GB per tensor)")
    ap.add_argument("--sweep-ks", default="", help="with --sweep: comma-separated worker counts (default: the full list)")
    ap.add_argument("--sweep-bytes", type=int, default=4_000_000_000, help="with --sweep: bytes per [K,P] tensor (smaller for an ncu capture)")
    ap.add_argument("--sweep-standalone", action="store_true", help="with --sweep: time the stand-alone calls (fgd_mix ring / mean, fgd_consensus_distance) instead of the fused step")
    ap.add_argument("--kernels", action="store_true",
                    help="instead of the round: time every stand-alone C-ABI kernel of the config alone")
    ap.add_argument("--js", action="store_true",
                    help="instead of the round: time the JS functional-disagreement metric on synthetic logits")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the block of --steps rounds until the timed region lasts at least this long (0: exactly --steps rounds)")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration table the default run appends")
    ap.add_argument("--js-positions", type=int, default=4096, help="with --js: token positions U (reduce for profiling)")
    ap.add_argument("--jsonl", default="", help="write one JSON record per round of the untimed consensus trajectory to this file")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true")
    return ap.parse_args()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------- mixes per round
def mix_desc(fgd, spec, cfg, rnd, seed, mix_id, dense_W):
    K = cfg["K"]
    kind = spec[0]
    if kind == "mean":
        return fgd.MixDesc.mean(K)
    if kind == "identity":
        return fgd.MixDesc.identity(K)
    if kind == "dense":
        return fgd.MixDesc.dense(dense_W)
    d = {"ring": lambda: fgd.MixDesc.ring(K), "xor": lambda: fgd.MixDesc.onepeer_xor(K, rnd),
         "hypercube": lambda: fgd.MixDesc.hypercube(K),
         "matching": lambda: fgd.MixDesc.random_matching(K, seed, rnd, mix_id)}[kind]()
    if cfg["p_fail"] > 0.0:
        d = d.with_failures(seed, rnd, mix_id, cfg["p_fail"], fgd.FGD_RENORM_METROPOLIS)
    return d


# ---------------------------------------------------------------------- clocks sampling
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------- CPU oracle leg
def oracle_leg(cfg, steps, warmup, seed=0, sample_cols=1 << 23, threads=0):
    """Times the float64 oracle, as it stands, on a bounded column sample of the workload."""
    import oracle
    from fgd_inputs import gen
    from oracle import topology as T
    K = cfg["K"]
    Ps = min(cfg["P"], sample_cols)
    all_threads = oracle.num_threads()
    if threads > 0:
        oracle.set_num_threads(threads)
    sig = gen.drift_sigmas(seed, K, *cfg["sig"]) if cfg["sig"][0] != cfg["sig"][1] else np.full(K, cfg["sig"][0], np.float32)
    theta = gen.theta0(seed, K, Ps).astype(np.float64)
    v = np.zeros((K, Ps))
    dense = gen.sinkhorn_W(seed, K).astype(np.float64) if "dense" in (cfg["mix1"][0], cfg["mix2"][0]) else None

    def W_of(spec, rnd, mix_id):
        kind = spec[0]
        if kind in ("mean", "identity"):
            return oracle.dense_W(kind, K)
        if kind == "dense":
            return dense
        nbr, w, ws = {"ring": lambda: T.ring(K), "xor": lambda: T.onepeer_xor(K, rnd),
                      "hypercube": lambda: T.hypercube(K),
                      "matching": lambda: T.random_matching(K, seed, rnd, mix_id)}[kind]()
        mask, renorm = None, T.RENORM_NONE
        if cfg["p_fail"] > 0.0:
            mask, renorm = T.edge_mask(seed, rnd, mix_id, cfg["p_fail"], nbr), T.RENORM_METROPOLIS
        return np.array(T.dense_from_sparse(nbr, *T.effective_weights(nbr, w, ws, mask, renorm)))

    times = []
    for r in range(warmup + steps):
        local = theta + gen.scaled_normal(seed, gen.TENSOR_DRIFT, r, K, Ps, sig).astype(np.float64)
        t0 = time.perf_counter()
        W1, W2 = W_of(cfg["mix1"], r, 1), W_of(cfg["mix2"], r, 2)
        theta, v = oracle.outer_round(W1, W2, theta, local, v, 0.7, 0.9)
        oracle.consensus_sumsq(theta)
        if r >= warmup:
            times.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    used = oracle.num_threads()
    oracle.set_num_threads(all_threads)
    return {"value": K * Ps / sec, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"first {Ps} of {cfg['P']} columns, all K={K} workers, {len(times)} round(s), "
                      f"{sec:.3f} s per round (round arithmetic + consensus sums only)"}, sec


def run_reference(args):
    cfg = CONFIGS[args.config]
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, min(args.steps, 3)), max(0, min(args.warmup, 1))
    base, sec = oracle_leg(cfg, steps, warmup)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg["name"], "note": "CPU oracle on a bounded column sample; steps/warmup clamped"},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------- N > 1: replicas
def aggregate(dist, elapsed_ms: float, units: int, device=None):
    """Whole-job figures of N independent replicas: the slowest rank's time and the sum of the
    units all ranks processed.  `dist` is torch.distributed (any backend) or None for N = 1."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


# ---------------------------------------------------------------------- our arm
class RoundState:
    """Tensors, driver and per-round launch logic of one configuration."""

    def __init__(self, torch, fgd, gen, inputs_gpu, OuterRound, cfg, dev, local_rank, flags, log_rounds, seed=0):
        self.torch, self.fgd, self.cfg, self.flags, self.seed = torch, fgd, cfg, flags, seed
        K, P = cfg["K"], cfg["P"]
        self.K, self.P = K, P
        self.sig = (gen.drift_sigmas(seed, K, *cfg["sig"]) if cfg["sig"][0] != cfg["sig"][1]
                    else np.full(K, cfg["sig"][0], np.float32))
        self.dense_W = gen.sinkhorn_W(seed, K) if "dense" in (cfg["mix1"][0], cfg["mix2"][0]) else None
        self.theta = torch.empty((K, P), dtype=torch.float32, device=dev)
        self.local = torch.empty_like(self.theta)
        self.mom = torch.zeros_like(self.theta)
        inputs_gpu.theta0(self.theta, seed)
        inputs_gpu.local_steps(self.local, self.theta, self.sig, seed, 0)
        self.drv = OuterRound(K, P, device=local_rank)
        self.cd_log = torch.zeros((log_rounds, K), dtype=torch.float64, device=dev)
        self.main = torch.cuda.current_stream(dev)
        self.ranges = None
        if flags.subset_frac > 0.0:      # three blocks (embeddings, LM head, first layers), 4-column bounds
            f = flags.subset_frac
            q = lambda t: int(t * P) // 4 * 4
            self.ranges = [(0, q(0.4 * f)), (q(0.5), q(0.5 + 0.3 * f)), (q(1.0 - 0.3 * f), P)]

    def mix(self, which, rnd):
        return mix_desc(self.fgd, self.cfg[which], self.cfg, rnd, self.seed, 1 if which == "mix1" else 2, self.dense_W)

    def one_round(self, r, ev_pair=None):
        """Host mix build, side-stream Mix1, fused step in place.  ev_pair brackets the step kernel alone."""
        fl, drv, main = self.flags, self.drv, self.main
        m1, m2 = self.mix("mix1", r), self.mix("mix2", r)
        drv.cd_sumsq = self.cd_log[r % self.cd_log.shape[0]]
        if fl.fuse_mix1:
            if ev_pair is not None:
                ev_pair[0].record(main)
            drv.step(m2, self.local, self.theta, self.mom, self.theta, 0.7, 0.9, mix1_fused=m1, mix2_ranges=self.ranges,
                     average_momentum=fl.average_momentum)
            if ev_pair is not None:
                ev_pair[1].record(main)
            return
        if not (fl.chain_mix1 and drv._pending is not None):
            drv.launch_mix1(m1, self.theta)
        if ev_pair is not None:
            main.wait_event(drv._pending[0])     # keep the Mix1 wait out of the kernel's event pair
            ev_pair[0].record(main)
        drv.step(m2, self.local, self.theta, self.mom, self.theta, 0.7, 0.9, mix2_ranges=self.ranges,
                 average_momentum=fl.average_momentum, emit_next_mix1=fl.chain_mix1)
        if ev_pair is not None:
            ev_pair[1].record(main)

    def free(self):
        self.theta = self.local = self.mom = self.cd_log = None
        self.drv.close()
        self.drv = None
        self.torch.cuda.empty_cache()


class Flags:
    def __init__(self, subset_frac=0.0, average_momentum=False, chain_mix1=False, fuse_mix1=False, graph=False):
        self.subset_frac, self.average_momentum = subset_frac, average_momentum
        self.chain_mix1, self.fuse_mix1, self.graph = chain_mix1, fuse_mix1, graph


MAX_TIMED_ROUNDS = 4000     # bound on the rounds (and event pairs) of one timed region


def time_rounds(torch, st, steps, warmup, min_seconds=0.0, graph=None, barrier=None, make_sampler=None):
    """`warmup` untimed rounds, then the timed region: the block of `steps` rounds, repeated as often
    as it takes to fill `min_seconds` (so that the clock sampler sees the load), bracketed by
    synchronisation on both sides; CUDA events on the launching stream around the region and around
    every fused-step launch.  Returns the elapsed ms, the per-launch kernel ms, rounds timed, launches."""
    main = st.main
    probe = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    for r in range(warmup):
        if r == warmup - 1:
            probe[0].record(main)
        if graph is not None:
            graph.replay()
        else:
            st.one_round(r)
        if r == warmup - 1:
            probe[1].record(main)
    torch.cuda.synchronize()
    est_ms = max(probe[0].elapsed_time(probe[1]), 1e-3)
    repeats = 1
    if min_seconds > 0.0:
        repeats = max(1, int(np.ceil(min_seconds * 1e3 / (est_ms * steps))))
        repeats = min(repeats, max(1, MAX_TIMED_ROUNDS // steps))
    total = steps * repeats
    if barrier is not None:
        barrier()
    torch.cuda.synchronize()
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(total)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = st.drv.ctx.launch_count
    sampler = make_sampler() if make_sampler is not None else None     # clocks DURING the timed region only
    t_begin.record(main)
    for i in range(total):
        if graph is not None:
            pairs[i][0].record(main)
            graph.replay()
            pairs[i][1].record(main)
        else:
            st.one_round(warmup + i, pairs[i])
    t_end.record(main)
    torch.cuda.synchronize()
    launches = st.drv.ctx.launch_count - launches0 if graph is None else 2 * total   # Mix1 kernel and fused step per replay
    clocks = sampler.stop() if sampler is not None else None
    return {"elapsed_ms": t_begin.elapsed_time(t_end), "kernel_ms": [a.elapsed_time(b) for a, b in pairs],
            "rounds": total, "repeats": repeats, "launches": int(launches), "last_round": warmup + total - 1,
            "clocks": clocks}


def pattern_probe(torch, fgd, st, reps=5):
    """Time of the arithmetic-free tile copy that moves the fused step's bytes (3 [K,P] tensors read,
    2 written, the step's own tile shape) on this configuration's tensors, in this run: the roofline
    of the step's access pattern on this machine.  None for worker counts the probe is not built for."""
    if st.K not in (4, 8, 16, 32, 64):
        return None
    f = lambda: fgd.fgd_debug_stream_pattern(st.drv.ctx, st.local, st.theta, st.mom, st.theta)
    for _ in range(2):
        f()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(st.main)
        f()
        b.record(st.main)
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = statistics.mean(ts)
    return {"ms": ms, "ms_min": min(ts), "bytes": 20 * st.K * st.P, "gbs": 20 * st.K * st.P / (ms * 1e-3) / 1e9,
            "what": "fgd_debug_stream_pattern: the step's tiles and TMA ring, no arithmetic, in place"}


def roofline_of(cfg, cfg_id, K, P, kern_times, fuse_mix1, peak, peak_kind, traffic_ok=True):
    x_vec = cfg["mix1"][0] == "mean"
    step_bytes = (20 * K * P + 4 * P) if x_vec else 24 * K * P      # outer-step kernel, algorithmic
    mix1_bytes = (4 * K * P + 4 * P) if x_vec else 8 * K * P
    if fuse_mix1:
        step_bytes, mix1_bytes = 20 * K * P, 0
    kern_ms = statistics.mean(kern_times)
    achieved = step_bytes / (kern_ms * 1e-3) / 1e9
    tr = (NCU_TRAFFIC_FUSED_MIX1 if fuse_mix1 else NCU_TRAFFIC_BYTES_PER_WORKER_PARAM).get(cfg_id) if traffic_ok else None
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": None if tr is None else tr * K * P,
            "kernel": "outer_step_dense_tc_kernel" if K == 64 else "outer_step_tma_kernel",
            "kernel_ms": kern_ms, "kernel_ms_median": statistics.median(kern_times),
            "kernel_ms_min": min(kern_times), "kernel_ms_max": max(kern_times),
            "algorithmic_bytes": step_bytes, "peak_kind": f"of {peak_kind}",
            "frac_of_nominal_8000": achieved / 8000.0}
    return roof, step_bytes, mix1_bytes


def consensus_trajectory(torch, fgd, inputs_gpu, st, rounds, jsonl_path=None):
    """The configuration's own rounds from its initial state with a fresh drift every round (untimed):
    the consensus distance (Sec. 4.4 definition) after each.  Restores nothing: call it last.
    With `jsonl_path` one record per round goes to that file: the per-worker sums of squares, both
    consensus distances, the fused step's time and bandwidth, and how many edges each mix lost."""
    inputs_gpu.theta0(st.theta, st.seed)
    st.mom.zero_()
    st.drv._pending = None
    out, records = [], []
    K, P = st.K, st.P
    x_vec = st.cfg["mix1"][0] == "mean"
    step_bytes = 20 * K * P if st.flags.fuse_mix1 else ((20 * K * P + 4 * P) if x_vec else 24 * K * P)

    def dropped(m):          # undirected edges the round's mask took out of a sparse mix
        return 0 if m.edge_mask is None else int(((m.edge_mask == 0) & (m.nbr >= 0)).sum()) // 2

    for r in range(rounds):
        m1, m2 = st.mix("mix1", r), st.mix("mix2", r)
        if not st.flags.fuse_mix1:
            st.drv.launch_mix1(m1, st.theta)
            st.main.wait_event(st.drv._pending[0])
        inputs_gpu.local_steps(st.local, st.theta, st.sig, st.seed, r)
        st.drv.cd_sumsq = st.cd_log[r % st.cd_log.shape[0]]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st.main)
        st.drv.step(m2, st.local, st.theta, st.mom, st.theta, 0.7, 0.9, mix1_fused=m1 if st.flags.fuse_mix1 else None)
        e1.record(st.main)
        torch.cuda.synchronize()
        s = st.drv.cd_sumsq.cpu().numpy()
        cd_norm, cd_sq = fgd.fgd_cd_finalize(s)
        out.append(cd_norm)
        ms = e0.elapsed_time(e1)
        records.append({"round": r, "sumsq": [float(v) for v in s], "cd_norm": cd_norm, "cd_sq": cd_sq, "step_ms": ms,
                        "step_gbs": step_bytes / (ms * 1e-3) / 1e9, "worker_params_per_s_step": K * P / (ms * 1e-3),
                        "mix1_edges_dropped": dropped(m1), "mix2_edges_dropped": dropped(m2)})
    if jsonl_path:
        with open(jsonl_path, "w") as f:
            for rec in records:
                f.write(json.dumps(rec) + "\n")
    return out


CONFIG_ROUNDS = {1: 1, 2: 10, 3: 10, 4: 20, 5: 5, 6: 3}     # rounds each configuration asks for


def extra_configs(torch, fgd, gen, inputs_gpu, OuterRound, dev, local_rank, peak, peak_kind, rounds=10):
    """Configurations 1, 2, 4 (factored and with Mix1 fused) and 5 at full size, `rounds` timed
    rounds each after 3 warm-up rounds: the fused-step kernel's time and roofline figures."""
    out = {}
    for key, cfg_id, fuse in (("1", 1, False), ("2", 2, False), ("4", 4, False), ("4_fused", 4, True), ("5", 5, False)):
        cfg = CONFIGS[cfg_id]
        st = RoundState(torch, fgd, gen, inputs_gpu, OuterRound, cfg, dev, local_rank, Flags(fuse_mix1=fuse), 64)
        n = 200 if cfg_id == 1 else rounds
        t = time_rounds(torch, st, n, 3)
        roof, step_bytes, mix1_bytes = roofline_of(cfg, cfg_id, st.K, st.P, t["kernel_ms"], fuse, peak, peak_kind)
        ms_round = t["elapsed_ms"] / t["rounds"]
        entry = {"workload": cfg["name"] + (" [Mix1 fused into the step kernel]" if fuse else ""),
                 "kernel": roof["kernel"],
                 "kernel_ms": {"mean": roof["kernel_ms"], "median": roof["kernel_ms_median"], "min": roof["kernel_ms_min"],
                               "max": roof["kernel_ms_max"]},
                 "algorithmic_bytes": step_bytes, "achieved": roof["achieved"], "frac": roof["frac"],
                 "frac_of_nominal_8000": roof["frac_of_nominal_8000"], "traffic": roof["traffic"],
                 "ms_per_round": ms_round, "rounds_timed": t["rounds"], "gpu_launches": t["launches"],
                 "worker_params_per_s": st.K * st.P / (ms_round * 1e-3)}
        if cfg_id != 1:
            entry["pattern"] = pattern_probe(torch, fgd, st)
            if entry["pattern"]:
                entry["frac_of_pattern"] = entry["pattern"]["gbs"] and entry["achieved"] / entry["pattern"]["gbs"]
        if cfg_id == 1:
            entry["note"] = "working set fits in L2: a latency configuration, achieved/frac are not HBM figures"
            entry["latency"] = latency_leg(torch, fgd, st.drv, cfg, st.theta, st.local, st.mom, st.seed, st.dense_W, dev)
        out[key] = entry
        st.free()
        del st
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2606_22768_b200 as fgd
    from fgd_inputs import gen, gpu as inputs_gpu
    from paper_2606_22768_b200.round import OuterRound

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    if args.js:
        if rank == 0:
            print(json.dumps(js_table(torch, fgd, dev, measured_peak(), U=args.js_positions)), flush=True)
        return
    if args.sweep:
        if rank == 0:
            ks = tuple(int(k) for k in args.sweep_ks.split(",")) if args.sweep_ks else None
            print(json.dumps(sweep_table(torch, fgd, gen, dev, measured_peak(), tensor_bytes=args.sweep_bytes,
                                         standalone=args.sweep_standalone, **({"Ks": ks} if ks else {}))), flush=True)
        return
    cfg = dict(CONFIGS[args.config])
    if args.cols:
        cfg["P"] = args.cols
        cfg["name"] += f" [REDUCED to P={args.cols} for profiling: not a benchmark number]"
    K, P, seed = cfg["K"], cfg["P"], 0
    steps, warmup = args.steps, max(args.warmup, 3)
    flags = Flags(args.subset_frac, args.average_momentum, args.chain_mix1, args.fuse_mix1, args.graph)
    if args.fuse_mix1 and (args.chain_mix1 or args.graph or cfg["mix1"][0] == "dense"):
        raise SystemExit("--fuse-mix1 excludes --chain-mix1 / --graph and needs a mean or sparse Mix1")
    st = RoundState(torch, fgd, gen, inputs_gpu, OuterRound, cfg, dev, local_rank, flags, 64, seed)
    drv, theta, local, mom, dense_W, sig = st.drv, st.theta, st.local, st.mom, st.dense_W, st.sig
    if st.ranges is not None:
        cfg["name"] += f" [variant: Mix2 on {sum(b - a for a, b in st.ranges) / P:.0%} of the columns]"
    if args.average_momentum:
        cfg["name"] += " [variant: momentum averaged (GlobalM1S)]"
    if args.chain_mix1:
        cfg["name"] += " [variant: Mix1 (mean) of round r+1 emitted by the fused step of round r]"
    if args.fuse_mix1:
        cfg["name"] += " [variant: Mix1 fused into the step kernel]"

    if args.kernels:
        if rank == 0:
            print(json.dumps(kernel_table(torch, fgd, drv, cfg, theta, local, mom, seed, dense_W, measured_peak())), flush=True)
        return

    graph = None
    if args.graph:      # the whole round as ONE graph launch (static topologies only: descriptors are frozen in)
        if cfg["p_fail"] > 0.0 or "xor" in (cfg["mix1"][0], cfg["mix2"][0]) or args.chain_mix1:
            raise SystemExit("--graph needs the same Mix1 / Mix2 every round (configs 1, 3, 5)")
        for r in range(2):
            st.one_round(r)         # eager calls size the launches and create the Mix1 buffer
        torch.cuda.synchronize()
        drv.cd_sumsq = st.cd_log[0]
        graph = drv.capture(lambda: (drv.launch_mix1(st.mix("mix1", 0), theta),
                                     drv.step(st.mix("mix2", 0), local, theta, mom, theta,
                                              0.7, 0.9, mix2_ranges=st.ranges, average_momentum=args.average_momentum)))
        cfg["name"] += " [whole round replayed from one CUDA graph]"

    t = time_rounds(torch, st, steps, warmup, min_seconds=args.min_seconds, graph=graph,
                    barrier=dist.barrier if world > 1 else None,
                    make_sampler=(lambda: ClockSampler(local_rank)) if rank == 0 else None)
    clocks = t["clocks"]
    if world > 1:
        dist.barrier()
    elapsed_ms, units = aggregate(dist if world > 1 else None, t["elapsed_ms"], K * P, dev)
    kern_times = t["kernel_ms"]

    ms_per_step = elapsed_ms / t["rounds"]
    value = units / (ms_per_step * 1e-3)
    peak, peak_kind = measured_peak()
    variant = args.subset_frac > 0.0 or args.average_momentum or args.chain_mix1 or args.graph   # not captured with ncu
    roofline, step_bytes, mix1_bytes = roofline_of(cfg, args.config, K, P, kern_times, args.fuse_mix1, peak, peak_kind,
                                                   traffic_ok=not variant)
    if graph is not None:
        roofline["note"] = "graph variant: the event pair spans the whole replay (Mix1 kernel included), so achieved understates the step kernel"

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": cfg["name"], "K": K, "P": P, "rounds_timed": t["rounds"],
                       "timed_region": (f"the block of {steps} rounds repeated {t['repeats']} time(s) back to back "
                                        f"({t['rounds']} rounds, {elapsed_ms / 1e3:.2f} s) so that the clock samples cover it; "
                                        "ms_per_step is the mean over all of them"),
                       "l2": (f"inputs {(3 * K * P * 4) / 1e9:.1f} GB per round, larger than the 126 MB L2"
                              if 3 * K * P * 4 > 4 * 126e6 else "working set fits in L2: latency config, not an HBM number"),
                       "replicas": world, "step": "host mix build + side-stream Mix1 + fused outer step with consensus sums"},
            "hbm_gbs_whole_step": (step_bytes + mix1_bytes) / (ms_per_step * 1e-3) / 1e9,
            "roofline": roofline, "gpu_launches": t["launches"], "clocks": clocks}

    if rank == 0:
        # context: the same STREAM-style copy the pool's peak was measured with, on THIS box, now
        roofline["copy_gbs_this_box"] = copy_bandwidth(torch, dev)
        roofline["pattern"] = pattern_probe(torch, fgd, st)      # and the step's own access pattern without arithmetic
    if rank == 0 and 3 * K * P * 4 <= 4 * 126e6:
        line["latency"] = latency_leg(torch, fgd, drv, cfg, theta, local, mom, seed, dense_W, dev)
    if rank == 0 and not args.no_overlap:
        line["overlap"] = overlap_model(torch, fgd, inputs_gpu, drv, cfg, theta, local, sig, seed, dense_W)
    if K * P * 4 > (32 << 30):
        line["e2e"] = None          # a pinned host copy of theta_local would take more host memory than is safe to assume
        line["config"]["e2e_note"] = "skipped: theta_local is %.0f GB, too large to pin on the host" % (K * P * 4 / 1e9)
    elif not args.no_e2e:
        line["e2e"] = e2e_leg(torch, dist, fgd, drv, cfg, theta, local, mom, st.cd_log, seed, dense_W, world, dev)
    if rank == 0 and graph is None and not args.chain_mix1:
        n = CONFIG_ROUNDS[args.config]
        line["consensus"] = {"cd_norm_per_round": consensus_trajectory(torch, fgd, inputs_gpu, st, n, args.jsonl or None), "rounds": n,
                             "note": "separate untimed run of the configuration's own rounds from its initial state, fresh "
                                     "drift every round (the timed rounds reuse one theta_local: bandwidth only)"}
    del drv, theta, local, mom
    st.free()
    del st
    if rank == 0 and world == 1 and args.config == 3 and not args.cols and not args.no_configs and not variant and not args.fuse_mix1:
        line["configs"] = extra_configs(torch, fgd, gen, inputs_gpu, OuterRound, dev, local_rank, peak, peak_kind)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_leg(cfg, 4, 1)[0]
        line["cpu_baseline"]["value_1thread"] = oracle_leg(cfg, 1, 0, sample_cols=1 << 19, threads=1)[0]["value"]
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def kernel_table(torch, fgd, drv, cfg, theta, local, mom, seed, dense_W, peak, reps=10):
    """Each C-ABI kernel of this config timed alone (CUDA events, mean of `reps` after 3 warm-ups),
    with its algorithmic bytes: GB/s and fraction of the measured HBM peak."""
    K, P = cfg["K"], cfg["P"]
    dev = theta.device
    ctx = drv.ctx
    scratch = torch.empty_like(theta)
    xvec = torch.empty(P, dtype=torch.float32, device=dev)
    cd = torch.zeros(K, dtype=torch.float64, device=dev)
    m1 = mix_desc(fgd, cfg["mix1"], cfg, 0, seed, 1, dense_W)
    m2 = mix_desc(fgd, cfg["mix2"], cfg, 0, seed, 2, dense_W)
    mean = fgd.MixDesc.mean(K)
    fgd.fgd_mix(ctx, mean, theta, xvec, out_is_vector=True)
    WP = K * P
    cases = {
        "fgd_outer_grad": (lambda: fgd.fgd_outer_grad(ctx, theta, local, scratch), 12 * WP),
        "fgd_mix mean -> [P]": (lambda: fgd.fgd_mix(ctx, mean, theta, xvec, out_is_vector=True), 4 * WP + 4 * P),
        "fgd_mix Mix2 kind -> [K,P]": (lambda: fgd.fgd_mix(ctx, m2, theta, scratch), 8 * WP),
        "fgd_consensus_distance": (lambda: fgd.fgd_consensus_distance(ctx, theta, cd), 4 * WP),
        "fgd_outer_step x=[P], with consensus": (lambda: fgd.fgd_outer_step(ctx, m2, None, xvec, True, local, theta, mom, theta, 0.7, 0.9, cd), 20 * WP + 4 * P),
        "fgd_outer_step x=[P], no consensus": (lambda: fgd.fgd_outer_step(ctx, m2, None, xvec, True, local, theta, mom, theta, 0.7, 0.9, None), 20 * WP + 4 * P),
        "fgd_outer_step Mix1 mean fused": (lambda: fgd.fgd_outer_step(ctx, m2, mean, None, False, local, theta, mom, theta, 0.7, 0.9, cd), 20 * WP),
        "fgd_outer_step x=[K,P]": (lambda: fgd.fgd_outer_step(ctx, m2, None, scratch, False, local, theta, mom, theta, 0.7, 0.9, cd), 24 * WP),
    }
    if cfg["mix1"][0] not in ("mean", "dense"):
        cases["fgd_outer_step Mix1 gossip fused"] = (lambda: fgd.fgd_outer_step(ctx, m2, m1, None, False, local, theta, mom, theta, 0.7, 0.9, cd), 20 * WP)
    out = {"workload": cfg["name"], "peak_gbs": peak[0], "peak_kind": peak[1], "kernels": {}}
    for name, (fn, nbytes) in cases.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        gbs = nbytes / (ms * 1e-3) / 1e9
        out["kernels"][name] = {"ms": round(ms, 4), "algorithmic_gb": round(nbytes / 1e9, 2), "gbs": round(gbs, 1),
                                "frac": round(gbs / peak[0], 3)}
    return out


def sweep_table(torch, fgd, gen, dev, peak, tensor_bytes=4_000_000_000, reps=10,
                Ks=(2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 16, 17, 20, 24, 28, 32, 40, 48, 56, 63, 64), standalone=False):
    """Fused outer step (in place, consensus sums on) across worker counts at a fixed tensor size:
    Mix2 = ring / hypercube (powers of two) / dense Sinkhorn with x one value per column, and the
    fully fused ring-ring and matching-matching (pairwise gossip for both mixes, App. A) rounds.  GB/s = algorithmic bytes (20 K P + 4 P, or 20 K P fused) / time."""
    out = {"peak_gbs": peak[0], "peak_kind": peak[1], "tensor_bytes": tensor_bytes, "unit": "GB/s", "rows": {}}
    for K in Ks:
        P = tensor_bytes // 4 // K // 128 * 128
        tp = torch.empty((K, P), dtype=torch.float32, device=dev).normal_(0.0, 0.02)
        tl = tp + 1e-3 * torch.randn_like(tp)
        v = torch.zeros_like(tp)
        x = tp.mean(0).contiguous()
        cd = torch.zeros(K, dtype=torch.float64, device=dev)
        ctx = fgd.Context(K, P, device=dev.index or 0)
        ring = fgd.MixDesc.ring(K)
        if standalone:      # the stand-alone calls: 8 / 4 + 4/K / 4 algorithmic bytes per worker-parameter
            out_t, xv, row = torch.empty_like(tp), torch.empty(P, dtype=torch.float32, device=dev), {}
            mean = fgd.MixDesc.mean(K)
            for name, f, nbytes in (("fgd_mix ring -> [K,P]", lambda: fgd.fgd_mix(ctx, ring, tp, out_t), 8 * K * P),
                                    ("fgd_mix matching -> [K,P]", lambda: fgd.fgd_mix(ctx, fgd.MixDesc.random_matching(K, 0, 0, 1), tp, out_t), 8 * K * P),
                                    ("fgd_mix mean -> [P]", lambda: fgd.fgd_mix(ctx, mean, tp, xv, out_is_vector=True), 4 * K * P + 4 * P),
                                    ("fgd_consensus_distance", lambda: fgd.fgd_consensus_distance(ctx, tp, cd), 4 * K * P)):
                for _ in range(3):
                    f()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(reps):
                    f()
                b.record()
                torch.cuda.synchronize()
                row[name] = round(nbytes / (a.elapsed_time(b) / reps * 1e-3) / 1e9)
            out["rows"][str(K)] = row
            del tp, tl, v, x, out_t, xv
            continue
        cases = {"ring": (ring, None), "dense": (fgd.MixDesc.dense(gen.sinkhorn_W(0, K)), None), "ring+ring fused": (ring, ring),
                 "matching+matching fused": (fgd.MixDesc.random_matching(K, 0, 0, 2), fgd.MixDesc.random_matching(K, 0, 0, 1))}
        if K & (K - 1) == 0 and K > 1:
            cases["hypercube"] = (fgd.MixDesc.hypercube(K), None)
        row = {}
        for name, (m2, m1) in cases.items():
            f = ((lambda: fgd.fgd_outer_step(ctx, m2, m1, None, False, tl, tp, v, tp, 0.7, 0.9, cd)) if m1 is not None
                 else (lambda: fgd.fgd_outer_step(ctx, m2, None, x, True, tl, tp, v, tp, 0.7, 0.9, cd)))
            for _ in range(3):
                f()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                f()
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / reps
            nbytes = 20 * K * P + (0 if m1 is not None else 4 * P)
            row[name] = round(nbytes / (ms * 1e-3) / 1e9)
        out["rows"][str(K)] = row
        del tp, tl, v, x
    return out


def js_table(torch, fgd, dev, peak, K=8, U=4096, V=128256, k=100, reps=5):
    """JS metric on synthetic logits shaped like a Llama-3 vocabulary: K workers, U token positions.
    Algorithmic bytes = one read of the averaged model's logits (U V 4) plus the gathered entries."""
    g = torch.Generator(device=dev)
    g.manual_seed(0)
    avg = torch.randn((U, V), device=dev, generator=g) * 2.0
    work = torch.empty((K, U, V), device=dev)
    for m in range(K):
        work[m] = avg + 0.3 * torch.randn((U, V), device=dev, generator=g)
    idx = torch.empty((U, k), dtype=torch.int32, device=dev)
    d = torch.empty((K, U), dtype=torch.float64, device=dev)
    cdw = torch.empty(K, dtype=torch.float64, device=dev)
    for _ in range(2):
        fgd.fgd_js_distance(work, avg, idx, d, cdw, top_k=k)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fgd.fgd_js_distance(work, avg, idx, d, cdw, top_k=k)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    nbytes = U * V * 4 + (K + 1) * U * k * 32      # one read of the averaged logits + one 32-byte sector per gathered entry
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"metric": "js_token_positions_per_s", "value": U / (ms * 1e-3), "ms": ms, "K": K, "U": U, "V": V, "top_k": k,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak[0], "unit": "GB/s", "frac": gbs / peak[0],
                         "algorithmic_bytes": nbytes, "peak_kind": f"of {peak[1]}", "traffic": None,
                         "kernel": "js_select_stream_kernel (+ js_distance_kernel, js_mean_kernel: the whole call is timed)"},
            "cd_js": float(cdw.mean())}


def copy_bandwidth(torch, dev, n=1 << 30, reps=10):
    """torch b.copy_(a) over 2^30 bf16 elements, read + write bytes, best of `reps` (GB/s)."""
    try:
        a = torch.empty(n, dtype=torch.bfloat16, device=dev)
        b = torch.empty_like(a)
    except Exception:
        return None
    best = None
    for _ in range(reps + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        b.copy_(a)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        best = ms if best is None else min(best, ms)
    return 2 * n * 2 / (best * 1e-3) / 1e9


def overlap_model(torch, fgd, inputs_gpu, drv, cfg, theta, local, sig, seed, dense_W, reps=3):
    """Algorithm 1's overlap on one GPU: Mix1 on the side stream while a stand-in compute kernel
    (the seeded drift generator) produces theta_local on the main stream.  Reports each alone
    and both together; on one GPU they share HBM, so this models the dependency structure."""
    dev = theta.device
    main = torch.cuda.current_stream(dev)
    m1 = mix_desc(fgd, cfg["mix1"], cfg, 0, seed, 1, dense_W)

    def timed(fn):
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(main)
            fn()
            b.record(main)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return min(ts)

    def mix1_only():
        drv.launch_mix1(m1, theta)
        main.wait_event(drv._pending[0])

    def standin_only():
        inputs_gpu.local_steps(local, theta, sig, seed, 1)

    def both():
        drv.launch_mix1(m1, theta)
        inputs_gpu.local_steps(local, theta, sig, seed, 1)
        main.wait_event(drv._pending[0])

    out = {"mix1_alone_ms": timed(mix1_only), "standin_compute_alone_ms": timed(standin_only),
           "overlapped_ms": timed(both)}
    drv._pending = None
    return out


def latency_leg(torch, fgd, drv, cfg, theta, local, mom, seed, dense_W, dev, reps=1000):
    """L2-resident configuration: the fused outer step is launch- and latency-bound, not an HBM
    number.  Times `reps` single launches (x given, consensus sums on) back to back with the working
    set hot in L2, and again with a 512 MB write between launches that evicts it."""
    K, P = cfg["K"], cfg["P"]
    main = torch.cuda.current_stream(dev)
    m2 = mix_desc(fgd, cfg["mix2"], cfg, 0, seed, 2, dense_W)
    x = torch.zeros(P, dtype=torch.float32, device=dev)
    cd = torch.zeros(K, dtype=torch.float64, device=dev)
    flush = torch.empty(128 << 20, dtype=torch.float32, device=dev)
    out = {"reps": reps, "unit": "us", "call": "fgd_outer_step, x given as [P], with consensus sums"}
    for name, do_flush in (("l2_hot", False), ("l2_flushed", True)):
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for i in range(-10, reps):
            if do_flush:
                flush.zero_()
            if i >= 0:
                pairs[i][0].record(main)
            fgd.fgd_outer_step(drv.ctx, m2, None, x, True, local, theta, mom, theta, 0.7, 0.9, cd)
            if i >= 0:
                pairs[i][1].record(main)
        torch.cuda.synchronize()
        us = sorted(a.elapsed_time(b) * 1e3 for a, b in pairs)
        out[name] = {"median": us[len(us) // 2], "best": us[0], "p95": us[int(0.95 * len(us))]}
    return out


def e2e_leg(torch, dist, fgd, drv, cfg, theta, local, mom, cd_log, seed, dense_W, world, dev, steps=3, n_chunks=16):
    """Same round through the C-ABI call that takes theta_local from HOST memory
    (fgd_outer_step_from_host: pinned host matrix, copied in column chunks that overlap the fused
    step of the previous chunk) and returns the consensus sums to the host; both transfers are
    inside the timed region, every step."""
    K, P = cfg["K"], cfg["P"]
    host_local = torch.empty((K, P), dtype=torch.float32, pin_memory=True)
    host_local.copy_(local)
    main = torch.cuda.current_stream(dev)

    def one(r):
        m1 = mix_desc(fgd, cfg["mix1"], cfg, r, seed, 1, dense_W)
        m2 = mix_desc(fgd, cfg["mix2"], cfg, r, seed, 2, dense_W)
        drv.launch_mix1(m1, theta)                       # side stream: overlaps the first chunk's copy
        ev, x, is_vec = drv._pending
        drv._pending = None
        main.wait_event(ev)
        fgd.fgd_outer_step_from_host(drv.ctx, m2, None, x, is_vec, host_local, local, theta, mom, theta, 0.7, 0.9,
                                     want_cd=True, n_chunks=n_chunks)   # returns once the sums are on the host
        drv.side.wait_event(main.record_event())          # x may be overwritten by the next round's Mix1 only now

    one(0)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(main)
    for r in range(steps):
        one(1 + r)
    b.record(main)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b)
    ms, units = aggregate(dist if world > 1 else None, ms, K * P, dev)
    return {"value": units / (ms / steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": K * P * 4,
            "d2h_bytes_per_step": K * 8 * min(n_chunks, (P + 1023) // 1024), "steps": steps, "ms_per_step": ms / steps,
            "call": f"fgd_outer_step_from_host, {n_chunks} column chunks"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
